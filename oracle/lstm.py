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
