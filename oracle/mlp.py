"""One mixed-precision training iteration of an MLP, step by step, on the CPU.

TEST INFRASTRUCTURE ONLY (see mpo.c).  The sequence follows the iteration the
paper describes for a layer (section 3.1, figure 1 caption; section 3.2):

  master FP32 -> round to FP16 working copy -> forward GEMMs (FP32 accumulate,
  FP16 store, ReLU) -> softmax cross-entropy with the gradient multiplied by S
  -> backward GEMMs (weight gradients and activation gradients, FP16) ->
  unscale by 1/S while inspecting for inf/NaN -> skip, or FP32 SGD(+momentum)
  on the master copy and re-round the FP16 copy.

Dynamic loss scaling (the paper's closing section only says the factor could be raised or
lowered by inspecting the weight gradients for overflow while skipping overflowing updates):
after an overflowing step S <- max(S * backoff, min); after `growth_interval` consecutive
clean steps S <- min(S * growth, max); either event restarts the count.

Readings where the paper is silent: no bias; mean loss over the batch; momentum
form v <- mu*v + g, w <- w - lr*v with v in FP32 starting at zero; a skipped step
leaves master, momentum and FP16 weights untouched; the ReLU derivative is taken
from the stored FP16 activation; the first layer's input gradient is not formed.
"""
from __future__ import annotations

import numpy as np

from . import mpo


class OracleMLP:
    def __init__(self, layers, S, lr, momentum=0.0):
        """layers: list of (in_features, out_features, relu)."""
        self.layers = [(int(i), int(o), bool(r)) for (i, o, r) in layers]
        for a, b in zip(self.layers[:-1], self.layers[1:]):
            assert a[1] == b[0]
        assert not self.layers[-1][2]
        self.S = np.float32(S)
        self.lr = np.float32(lr)
        self.mu = np.float32(momentum)
        self.use_momentum = float(momentum) != 0.0
        self.w32 = [None] * len(self.layers)
        self.w16 = [None] * len(self.layers)
        self.v = [np.zeros((o, i), dtype=np.float32) for (i, o, _) in self.layers]
        self.g16 = [np.zeros((o, i), dtype=np.uint16) for (i, o, _) in self.layers]
        # optimizer: kind 0 SGD(+momentum) by default; set_optimizer switches (state s1/s2 start at zero)
        self.opt = dict(kind=mpo.OPT_SGD, b2=np.float32(0.0), eps=np.float32(0.0), wd=np.float32(0.0), clip=0.0)
        self.last_coef = np.float32(1.0)
        self.s2 = [np.zeros((o, i), dtype=np.float32) for (i, o, _) in self.layers]
        self.b1t = np.float32(1.0)     # running products beta1^t, beta2^t over applied steps (Adam)
        self.b2t = np.float32(1.0)
        self.dynamic = None    # (growth_interval, backoff, growth, min_scale, max_scale) or None
        self.clean_steps = 0
        self.acts = None       # [a_0 .. a_L], uint16
        self.dz = None         # dz_l for l = 1..L (index l-1), uint16
        self.loss = None

    # -- section 3.1: FP32 master copy, FP16 working copy by rounding
    def set_master(self, l, w):
        i, o, _ = self.layers[l]
        w = np.ascontiguousarray(w, dtype=np.float32).reshape(o, i).copy()
        self.w32[l] = w
        self.w16[l] = mpo.f2h(w)

    def get_master(self, l):
        return self.w32[l].copy()

    # -- section 3.3: a_l = rn16(act(a_{l-1} . w16_l^T)), FP32 accumulate
    def forward(self, x16):
        a = mpo._u16(np.ascontiguousarray(x16))
        self.acts = [a]
        for l, (_, _, relu) in enumerate(self.layers):
            a = mpo.gemm_f16(mpo.OP_FWD, a, self.w16[l], relu=relu)
            self.acts.append(a)
        return self.acts[-1]

    # -- section 3.2: scaled backward pass
    def backward_scaled(self, labels):
        L = len(self.layers)
        dz, _, loss, bad = mpo.softmax_ce(self.acts[L], labels, self.S)
        self.loss = loss
        self.dz = [None] * L
        self.dz[L - 1] = dz
        for l in range(L - 1, -1, -1):
            # weight gradient: gW_l[j,k] = rn16(sum_i dz_l[i,j] * a_{l-1}[i,k])
            self.g16[l] = mpo.gemm_f16(mpo.OP_WGRAD, self.dz[l], self.acts[l])
            if l > 0:
                # activation gradient with the ReLU mask of the stored activation
                self.dz[l - 1] = mpo.gemm_f16(mpo.OP_DGRAD, self.dz[l], self.w16[l],
                                              mask=self.acts[l] if self.layers[l - 1][2] else None)
        return loss

    def set_optimizer(self, kind, lr, mu=0.0, b2=0.0, eps=0.0, wd=0.0, clip=0.0):
        """kind: mpo.OPT_*; mu is the momentum (SGD, Nesterov) or beta1 (Adam); clip: global-norm
        bound on the unscaled gradients (0 = off)."""
        self.opt = dict(kind=int(kind), b2=np.float32(b2), eps=np.float32(eps), wd=np.float32(wd), clip=float(clip))
        self.lr = np.float32(lr)
        self.mu = np.float32(mu)
        self.use_momentum = (kind == mpo.OPT_SGD and float(mu) != 0.0) or kind != mpo.OPT_SGD

    def set_dynamic_scale(self, growth_interval, min_scale, max_scale, backoff=0.5, growth=2.0):
        self.dynamic = (int(growth_interval), np.float32(backoff), np.float32(growth), np.float32(min_scale),
                        np.float32(max_scale))
        self.clean_steps = 0
        self.S = np.float32(min(max(self.S, np.float32(min_scale)), np.float32(max_scale)))

    # -- sections 3.1, 3.2: unscale, inspect, skip or update
    def step(self):
        inv = np.float32(1.0) / self.S
        overflow = 0
        for g in self.g16:
            overflow |= mpo.grad_nonfinite(g, inv)
        if not overflow:
            kind = self.opt["kind"]
            clip = self.opt["clip"]
            if clip > 0.0:      # section 3.2: clipping acts on the unscaled gradients of all layers together
                total = sum(mpo.grad_sqnorm(g, inv) for g in self.g16)
                self.last_coef = mpo.clip_coef(total, clip)
            if kind == mpo.OPT_SGD and float(self.opt["wd"]) == 0.0 and clip <= 0.0:
                for l in range(len(self.layers)):
                    mpo.update_apply(self.g16[l], self.w32[l], self.v[l], self.w16[l], inv, self.lr, self.mu,
                                     self.use_momentum)
            else:
                if kind == mpo.OPT_ADAM:       # bias corrections use the products including this step
                    self.b1t = np.float32(self.b1t * self.mu)
                    self.b2t = np.float32(self.b2t * self.opt["b2"])
                bc1 = np.float32(1.0) - self.b1t
                bc2 = np.float32(1.0) - self.b2t
                for l in range(len(self.layers)):
                    s1 = self.v[l] if (kind != mpo.OPT_SGD or self.use_momentum) else None
                    s2 = self.s2[l] if kind == mpo.OPT_ADAM else None
                    if clip > 0.0:
                        mpo.update_apply_clip(kind, self.g16[l], self.w32[l], s1, s2, self.w16[l], inv, self.last_coef,
                                              self.lr, self.mu, self.opt["b2"], self.opt["eps"], self.opt["wd"], bc1, bc2)
                    else:
                        mpo.update_apply_opt(kind, self.g16[l], self.w32[l], s1, s2, self.w16[l], inv, self.lr, self.mu,
                                             self.opt["b2"], self.opt["eps"], self.opt["wd"], bc1, bc2)
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

    def set_grad(self, l, g16):
        i, o, _ = self.layers[l]
        self.g16[l] = np.ascontiguousarray(mpo._u16(g16)).reshape(o, i).copy()
