"""Data-parallel training of the MLP over R replicas, step by step, on the CPU.

TEST INFRASTRUCTURE ONLY (see mpo.c).  The paper's language model aggregates its batch over
4 GPUs (section 4.5) and gives no formulas for the exchange; the plain definition is used: every
replica runs the iteration of mlp.OracleMLP on its own part of the batch with identical FP16
weights; the update uses the mean of the replicas' gradients (mpo_dp_update_apply: FP32 sum in
replica order, times 1/(S*R)); an overflow on any replica skips the step on all of them
(section 3.2); all replicas end the step with the same FP16 weights and the same loss scale.
"""
from __future__ import annotations

import numpy as np

from . import mpo
from .mlp import OracleMLP


class OracleDataParallelMLP:
    def __init__(self, layers, S, lr, momentum, R):
        self.R = int(R)
        self.replicas = [OracleMLP(layers, S, lr, momentum) for _ in range(self.R)]

    def set_master(self, l, w):
        for r in self.replicas:
            r.set_master(l, w)

    def forward_backward(self, xs, labels):
        """xs[q], labels[q]: replica q's part of the batch.  Returns the replicas' mean losses."""
        out = []
        for r, x, y in zip(self.replicas, xs, labels):
            r.forward(x)
            out.append(r.backward_scaled(y))
        return out

    def set_grad(self, q, l, g16):
        self.replicas[q].set_grad(l, g16)

    def step(self):
        lead = self.replicas[0]
        inv = np.float32(1.0) / lead.S
        overflow = 0
        for r in self.replicas:
            for g in r.g16:
                overflow |= mpo.grad_nonfinite(g, inv)
        if not overflow:
            for l in range(len(lead.layers)):
                mpo.dp_update_apply([r.g16[l] for r in self.replicas], lead.w32[l], lead.v[l], lead.w16[l], lead.S,
                                    lead.lr, lead.mu, lead.use_momentum)
                for r in self.replicas[1:]:
                    r.w32[l][...] = lead.w32[l]
                    r.v[l][...] = lead.v[l]
                    r.w16[l][...] = lead.w16[l]
        if lead.dynamic is not None:
            interval, backoff, growth, smin, smax = lead.dynamic
            for r in self.replicas:
                if overflow:
                    r.S = np.float32(max(np.float32(r.S * backoff), smin))
                    r.clean_steps = 0
                else:
                    r.clean_steps += 1
                    if r.clean_steps >= interval:
                        r.S = np.float32(min(np.float32(r.S * growth), smax))
                        r.clean_steps = 0
        return 1 if overflow else 0
