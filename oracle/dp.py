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

    def set_optimizer(self, kind, lr, mu=0.0, b2=0.0, eps=0.0, wd=0.0, clip=0.0):
        """Any kind of mlp.OracleMLP.set_optimizer.  Clipping (section 3.2) bounds the global norm of
        the MEAN unscaled gradient over all layers - the gradient of the aggregated batch - so every
        replica applies the same coefficient."""
        for r in self.replicas:
            r.set_optimizer(kind, lr, mu, b2, eps, wd, clip=clip)

    def step(self):
        lead = self.replicas[0]
        inv = np.float32(1.0) / lead.S
        overflow = 0
        for r in self.replicas:
            for g in r.g16:
                overflow |= mpo.grad_nonfinite(g, inv)
        if not overflow:
            kind = lead.opt["kind"]
            clip = lead.opt["clip"]
            plain = kind == mpo.OPT_SGD and float(lead.opt["wd"]) == 0.0 and clip <= 0.0
            if clip > 0.0:
                total = sum(mpo.dp_grad_sqnorm([r.g16[l] for r in self.replicas], lead.S) for l in range(len(lead.layers)))
                coef = mpo.clip_coef(total, clip)
                for r in self.replicas:
                    r.last_coef = coef
            if kind == mpo.OPT_ADAM:       # bias corrections use the products including this step
                for r in self.replicas:
                    r.b1t = np.float32(r.b1t * r.mu)
                    r.b2t = np.float32(r.b2t * r.opt["b2"])
            bc1 = np.float32(1.0) - lead.b1t
            bc2 = np.float32(1.0) - lead.b2t
            for l in range(len(lead.layers)):
                gs = [r.g16[l] for r in self.replicas]
                if plain:
                    mpo.dp_update_apply(gs, lead.w32[l], lead.v[l], lead.w16[l], lead.S, lead.lr, lead.mu, lead.use_momentum)
                elif clip > 0.0:
                    s1 = lead.v[l] if (kind != mpo.OPT_SGD or lead.use_momentum) else None
                    s2 = lead.s2[l] if kind == mpo.OPT_ADAM else None
                    mpo.dp_update_apply_clip(kind, gs, lead.w32[l], s1, s2, lead.w16[l], lead.S, lead.last_coef, lead.lr,
                                             lead.mu, lead.opt["b2"], lead.opt["eps"], lead.opt["wd"], bc1, bc2)
                else:
                    s1 = lead.v[l] if (kind != mpo.OPT_SGD or lead.use_momentum) else None
                    s2 = lead.s2[l] if kind == mpo.OPT_ADAM else None
                    mpo.dp_update_apply_opt(kind, gs, lead.w32[l], s1, s2, lead.w16[l], lead.S, lead.lr, lead.mu,
                                            lead.opt["b2"], lead.opt["eps"], lead.opt["wd"], bc1, bc2)
                for r in self.replicas[1:]:
                    r.w32[l][...] = lead.w32[l]
                    r.v[l][...] = lead.v[l]
                    r.s2[l][...] = lead.s2[l]
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
