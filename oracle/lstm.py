"""One LSTM layer with a projection, unrolled over time, in the mixed-precision recipe, on the CPU.

TEST INFRASTRUCTURE ONLY (see mpo.c).  The layer is the recurrent layer of the paper's language
model (section 4.5: 8192 cells projected to 1024): per time step

  [x_t ; r_{t-1}] . Wg^T + b  ->  gates  ->  c_t, h_t          (mpo_lstm_cell_fwd)
  r_t = rn16(h_t . Wp^T)                                          (FP32 accumulate, FP16 store)

and the backward pass walks the steps in reverse with scaled FP16 gradients (section 3.2):

  drtot_t = dr_ext_t + (recurrent part of dxr_{t+1})              (binary32 add, FP16 store)
  dh_t    = drtot_t . Wp
  dG_t, dc_{t-1} = cell backward(dh_t, dc_t, stored values)
  dxr_t   = dG_t . Wg           (left I columns: gradient wrt x_t; right P: wrt r_{t-1})
  dWg = sum_t dG_t^T . xr_t ,  dWp = sum_t drtot_t^T . h_t   (one product over all T*B rows each,
        so the sum over time is accumulated in binary32 before the single rounding to FP16)
  db  = column sums of dG over all T*B rows (binary32), rounded to FP16

Readings where the paper is silent: gate order and formulas as in mpo.c; cell state and gate
activations stored in FP16; bias kept as an FP16 working copy like the weights; no peepholes.
"""
from __future__ import annotations

import numpy as np

from . import mpo


class OracleLSTM:
    def __init__(self, T, B, I, H, P):
        self.T, self.B, self.I, self.H, self.P = T, B, I, H, P

    def forward(self, x, r0, c0, Wg, bias16, Wp):
        """x [T,B,I], r0 [B,P], c0 [B,H], Wg [4H,I+P], bias16 [4H], Wp [P,H]; all FP16 bit patterns."""
        T, B, I, H, P = self.T, self.B, self.I, self.H, self.P
        self.Wg, self.Wp = mpo._u16(Wg), mpo._u16(Wp)
        self.xr = np.zeros((T + 1, B, I + P), dtype=np.uint16)
        self.c = np.zeros((T + 1, B, H), dtype=np.uint16)
        self.h = np.zeros((T, B, H), dtype=np.uint16)
        self.acts = np.zeros((T, B, 4 * H), dtype=np.uint16)
        self.xr[:T, :, :I] = mpo._u16(x)
        self.xr[0, :, I:] = mpo._u16(r0)
        self.c[0] = mpo._u16(c0)
        for t in range(T):
            self.acts[t], self.c[t + 1], self.h[t] = mpo.lstm_cell_fwd(self.xr[t], self.Wg, bias16, self.c[t])
            self.xr[t + 1, :, I:] = mpo.gemm_f16(mpo.OP_FWD, self.h[t], self.Wp)
        return self.xr[1:, :, I:]          # r_t for t = 0..T-1

    def backward(self, dr_ext):
        """dr_ext [T,B,P]: scaled gradient wrt r_t from above.  Returns dx [T,B,I]; leaves dWg, dWp,
        db16 (and the per-step tensors) on the object."""
        T, B, I, H, P = self.T, self.B, self.I, self.H, self.P
        dr_ext = mpo._u16(dr_ext)
        self.dxr = np.zeros((T, B, I + P), dtype=np.uint16)
        self.drtot = np.zeros((T, B, P), dtype=np.uint16)
        self.dh = np.zeros((T, B, H), dtype=np.uint16)
        self.dG = np.zeros((T, B, 4 * H), dtype=np.uint16)
        self.dc = np.zeros((T + 1, B, H), dtype=np.uint16)     # dc[t]: gradient wrt c_{t-1} carried to step t-1
        for t in range(T - 1, -1, -1):
            if t == T - 1:
                self.drtot[t] = dr_ext[t]
            else:
                self.drtot[t] = mpo.add_f16(dr_ext[t], self.dxr[t + 1][:, I:])
            self.dh[t] = mpo.gemm_f16(mpo.OP_DGRAD, self.drtot[t], self.Wp)
            self.dG[t], self.dc[t] = mpo.lstm_cell_bwd(self.dh[t], None if t == T - 1 else self.dc[t + 1], self.acts[t],
                                                       self.c[t], self.c[t + 1])
            self.dxr[t] = mpo.gemm_f16(mpo.OP_DGRAD, self.dG[t], self.Wg)
        self.dWg = mpo.gemm_f16(mpo.OP_WGRAD, self.dG.reshape(T * B, 4 * H), self.xr[:T].reshape(T * B, I + P))
        self.dWp = mpo.gemm_f16(mpo.OP_WGRAD, self.drtot.reshape(T * B, P), self.h.reshape(T * B, H))
        self.db16, self.db32 = mpo.bias_grad(self.dG.reshape(T * B, 4 * H))
        return self.dxr[:, :, :I]


class OracleLSTMTrainer:
    """The LSTM layer trained in the mixed-precision recipe (sections 3.1, 3.2; the paper's
    language model, section 4.5, uses S = 128 and Adagrad): FP32 masters of Wg, Wp and the bias,
    FP16 working copies, and per iteration

      forward from zero state -> softmax cross-entropy over r_t as logits (mean over all T*B rows,
      logit gradient times S) -> backward through time -> inspect the unscaled weight and bias
      gradients for inf/NaN -> skip, or the optimizer step on the masters and re-round the copies
      -> optional dynamic scale (same schedule as OracleMLP).

    Readings where the paper is silent: the layer's projected output is used directly as the
    logits of the loss; recurrent input and cell state start at zero every iteration; the three
    parameter tensors share one optimizer (one clipping norm over all of them)."""

    def __init__(self, T, B, I, H, P, S, kind, lr, mu=0.0, b2=0.0, eps=0.0, wd=0.0, clip=0.0):
        self.net = OracleLSTM(T, B, I, H, P)
        self.T, self.B, self.I, self.H, self.P = T, B, I, H, P
        self.S = np.float32(S)
        self.kind, self.lr, self.mu = int(kind), np.float32(lr), np.float32(mu)
        self.b2, self.eps, self.wd, self.clip = np.float32(b2), np.float32(eps), np.float32(wd), float(clip)
        self.b1t, self.b2t = np.float32(1.0), np.float32(1.0)
        self.dynamic = None
        self.clean_steps = 0
        self.last_coef = np.float32(1.0)
        self.names = ("Wg", "Wp", "bias")

    def set_params(self, Wg, bias, Wp):
        K = self.I + self.P
        self.w32 = dict(Wg=np.array(Wg, dtype=np.float32).reshape(4 * self.H, K).copy(),
                        Wp=np.array(Wp, dtype=np.float32).reshape(self.P, self.H).copy(),
                        bias=np.array(bias, dtype=np.float32).reshape(4 * self.H).copy())
        self.w16 = {k: mpo.f2h(v) for k, v in self.w32.items()}
        self.s1 = {k: np.zeros_like(v) for k, v in self.w32.items()}
        self.s2 = {k: np.zeros_like(v) for k, v in self.w32.items()}
        self.g16 = {k: np.zeros(v.shape, dtype=np.uint16) for k, v in self.w32.items()}

    def set_dynamic_scale(self, growth_interval, min_scale, max_scale, backoff=0.5, growth=2.0):
        self.dynamic = (int(growth_interval), np.float32(backoff), np.float32(growth), np.float32(min_scale),
                        np.float32(max_scale))
        self.clean_steps = 0
        self.S = np.float32(min(max(self.S, np.float32(min_scale)), np.float32(max_scale)))

    def forward_backward(self, x16, labels):
        T, B, P, H = self.T, self.B, self.P, self.H
        r = self.net.forward(x16, np.zeros((B, P), dtype=np.uint16), np.zeros((B, H), dtype=np.uint16),
                             self.w16["Wg"], self.w16["bias"], self.w16["Wp"])
        self.logits = np.ascontiguousarray(r).reshape(T * B, P)
        dz, _, loss, bad = mpo.softmax_ce(self.logits, labels, self.S)
        self.dr_ext = dz.reshape(T, B, P)
        self.net.backward(self.dr_ext)
        self.g16 = dict(Wg=self.net.dWg, Wp=self.net.dWp, bias=self.net.db16)
        self.loss = loss
        return loss

    def step(self):
        inv = np.float32(1.0) / self.S
        overflow = 0
        for k in self.names:
            overflow |= mpo.grad_nonfinite(self.g16[k], inv)
        if not overflow:
            if self.clip > 0.0:
                total = sum(mpo.grad_sqnorm(self.g16[k], inv) for k in self.names)
                self.last_coef = mpo.clip_coef(total, self.clip)
            if self.kind == mpo.OPT_ADAM:
                self.b1t = np.float32(self.b1t * self.mu)
                self.b2t = np.float32(self.b2t * self.b2)
            bc1, bc2 = np.float32(1.0) - self.b1t, np.float32(1.0) - self.b2t
            for k in self.names:
                g = np.ascontiguousarray(self.g16[k]).reshape(-1)
                w, h = self.w32[k].reshape(-1), self.w16[k].reshape(-1)
                use_s1 = self.kind != mpo.OPT_SGD or float(self.mu) != 0.0
                s1 = self.s1[k].reshape(-1) if use_s1 else None
                s2 = self.s2[k].reshape(-1) if self.kind == mpo.OPT_ADAM else None
                if self.clip > 0.0:
                    mpo.update_apply_clip(self.kind, g, w, s1, s2, h, inv, self.last_coef, self.lr, self.mu, self.b2,
                                          self.eps, self.wd, bc1, bc2)
                else:
                    mpo.update_apply_opt(self.kind, g, w, s1, s2, h, inv, self.lr, self.mu, self.b2, self.eps, self.wd,
                                         bc1, bc2)
        if self.dynamic is not None:
            interval, backoff, growth, smin, smax = self.dynamic
            if overflow:
                self.S = np.float32(max(np.float32(self.S * backoff), smin))
                self.clean_steps = 0
            else:
                self.clean_steps += 1
                if self.clean_steps >= interval:
                    self.S = np.float32(min(np.float32(self.S * growth), smax))
                    self.clean_steps = 0
        return 1 if overflow else 0

    def train_step(self, x16, labels):
        loss = self.forward_backward(x16, labels)
        return loss, self.step()
