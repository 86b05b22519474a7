"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds NONE of the method's arithmetic: it only draws random numbers
(numpy PCG64) and casts them with numpy's own binary16 conversion, so that the
CUDA library and the CPU oracle can be handed identical bits.  Neither of those
two imports this module; their callers do.

The paper's experiments use datasets that are not available here (ILSVRC12,
VOC2007, WMT15, the 1-billion-word corpus, speech corpora).  The recipes below
stand in for them: they reproduce the layer shapes the paper quotes (the
bigLSTM gate/projection sizes of section 4.5) and the gradient-magnitude
structure it describes (section 3.2: most gradient exponents far below the FP16
normal range), with Gaussian activations and fan-in-scaled Gaussian weights.

Sub-streams are spawned from SeedSequence(seed) in the fixed order
weights-by-layer, inputs-by-step, labels-by-step.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np

# name -> (layers [(in, out, relu)], batch, S, lr, momentum, steps, seed)
MLP_CONFIGS = {
    # config 1: tiny MLP 256 -> 512 (ReLU) -> 10
    "tiny": dict(layers=[(256, 512, 1), (512, 10, 0)], batch=64, S=1024.0, lr=0.01, momentum=0.0,
                 steps=10, seed=0, head_scale=1.0),
    # config 2a: 4-layer width-1024 MLP whose head weights are scaled by 2^-16
    "scale_sweep": dict(layers=[(1024, 1024, 1)] * 3 + [(1024, 10, 0)], batch=256, S=1.0, lr=0.01,
                        momentum=0.0, steps=20, seed=1, head_scale=2.0 ** -16),
    # reduced twin of config 2a (same structure, width and batch / 4) for the CPU suite
    "scale_sweep_twin": dict(layers=[(256, 256, 1)] * 3 + [(256, 10, 0)], batch=64, S=1.0, lr=0.01,
                             momentum=0.0, steps=20, seed=1, head_scale=2.0 ** -16),
    # config 5: 8 square 12288 layers (ReLU) + 12288 -> 32000 head
    "large": dict(layers=[(12288, 12288, 1)] * 8 + [(12288, 32000, 0)], batch=4096, S=8192.0, lr=0.01,
                  momentum=0.9, steps=5, seed=4, head_scale=1.0),
    # reduced twin of config 5 (width and batch / 16)
    "large_twin": dict(layers=[(768, 768, 1)] * 8 + [(768, 2000, 0)], batch=256, S=8192.0, lr=0.01,
                       momentum=0.9, steps=5, seed=4, head_scale=1.0),
}

SCALE_SWEEP = (1.0, 2.0 ** 8, 2.0 ** 16, 2.0 ** 24)

# config 3: isolated GEMM shapes (M, N, K)
GEMM_SWEEP = [(1024, 1024, 1024), (2048, 2048, 2048), (4096, 4096, 4096), (8192, 8192, 8192),
              (8192, 16384, 4096), (8192, 4096, 16384)]
# config 4: bigLSTM-shaped products (section 4.5: 8192 cells, projection to 1024)
LSTM_GATE = (2048, 4 * 8192, 2048)
LSTM_PROJ = (2048, 1024, 8192)


def _streams(seed: int, n: int):
    return [np.random.default_rng(s) for s in np.random.SeedSequence(seed).spawn(n)]


def normal_f16(rng, shape, scale=1.0) -> np.ndarray:
    """N(0, scale^2) drawn in float64, cast to float32, then to float16 (numpy casts)."""
    x = rng.standard_normal(shape) * scale
    return x.astype(np.float32).astype(np.float16)


def normal_f16_fast(seed_seq, shape, scale=1.0, threads=8) -> np.ndarray:
    """Same distribution for multi-gigabyte tensors: float32 draws on several threads,
    one spawned stream per row block (the result depends on `threads`)."""
    rows = shape[0]
    out = np.empty(shape, dtype=np.float16)
    seqs = seed_seq.spawn(threads)
    bounds = np.linspace(0, rows, threads + 1).astype(np.int64)

    def work(t):
        r0, r1 = int(bounds[t]), int(bounds[t + 1])
        rng = np.random.default_rng(seqs[t])
        step = max(1, (1 << 24) // max(1, int(np.prod(shape[1:]))))
        for r in range(r0, r1, step):
            e = min(r1, r + step)
            blk = rng.standard_normal((e - r,) + tuple(shape[1:]), dtype=np.float32)
            blk *= np.float32(scale)
            out[r:e] = blk.astype(np.float16)

    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(work, range(threads)))
    return out


def mlp_masters(cfg, fast=False):
    """FP32 master weights N(0, 1/fan_in), made FP16-representable at t = 0."""
    L = len(cfg["layers"])
    seqs = np.random.SeedSequence(cfg["seed"]).spawn(L + 2 * cfg["steps"])
    out = []
    for l, (fin, fout, _) in enumerate(cfg["layers"]):
        scale = fin ** -0.5
        if l == L - 1:
            scale *= cfg["head_scale"]
        if fast:
            w16 = normal_f16_fast(seqs[l], (fout, fin), scale)
        else:
            w16 = normal_f16(np.random.default_rng(seqs[l]), (fout, fin), scale)
        out.append(w16.astype(np.float32))
    return out


def mlp_batches(cfg, steps=None):
    """(X float16 [steps, B, in], labels int32 [steps, B]); step t uses batch t."""
    L = len(cfg["layers"])
    T = cfg["steps"]
    seqs = np.random.SeedSequence(cfg["seed"]).spawn(L + 2 * T)
    n = T if steps is None else min(steps, T)
    fin = cfg["layers"][0][0]
    C = cfg["layers"][-1][1]
    B = cfg["batch"]
    X = np.empty((n, B, fin), dtype=np.float16)
    Y = np.empty((n, B), dtype=np.int32)
    for t in range(n):
        rx = np.random.default_rng(seqs[L + t])
        ry = np.random.default_rng(seqs[L + T + t])
        if B * fin > (1 << 25):
            X[t] = rx.standard_normal((B, fin), dtype=np.float32).astype(np.float16)
        else:
            X[t] = normal_f16(rx, (B, fin))
        Y[t] = ry.integers(0, C, size=B, dtype=np.int32)
    return X, Y


def loguniform_grads(n, S, seed=1):
    """Config 2b: 'true' gradients with random sign and magnitude 2^U, U ~ Uniform(-40, -10),
    formed in float32, multiplied by S (a power of two) and cast to float16 by numpy."""
    rng = np.random.default_rng(np.random.SeedSequence(seed).spawn(1)[0])
    U = rng.uniform(-40.0, -10.0, size=n)
    sign = np.where(rng.integers(0, 2, size=n) == 0, 1.0, -1.0)
    g = (sign * np.exp2(U)).astype(np.float32)
    return (g * np.float32(S)).astype(np.float16)


def gemm_operands(op, M, N, K, seed=2, scale_a=None, scale_b=None, fast=False):
    """Stored operands of one product.  op 0: A[M,K], B[N,K]; op 1: A[M,K], B[K,N];
    op 2: A[K,M], B[K,N].  Default scale: both N(0,1)/sqrt(K)."""
    sa = K ** -0.5 if scale_a is None else scale_a
    sb = K ** -0.5 if scale_b is None else scale_b
    shape_a = (K, M) if op == 2 else (M, K)
    shape_b = (N, K) if op == 0 else (K, N)
    seqs = np.random.SeedSequence([seed, op, M, N, K]).spawn(2)
    if fast:
        return normal_f16_fast(seqs[0], shape_a, sa), normal_f16_fast(seqs[1], shape_b, sb)
    return (normal_f16(np.random.default_rng(seqs[0]), shape_a, sa),
            normal_f16(np.random.default_rng(seqs[1]), shape_b, sb))


# LSTM layer with projection (the recurrent layer of the language model of section 4.5: 8192 cells
# projected to 1024, input width 1024; the batch of 1024 there is spread over 4 GPUs with 20
# unrolled steps).  "small" spans several tiles with ragged edges and finishes on the CPU in
# seconds; "biglstm" is the paper's layer with 2048 rows per step.
LSTM_CONFIGS = {
    "small": dict(T=4, B=200, I=64, H=160, P=96, S=1024.0, seed=71),
    "medium": dict(T=3, B=384, I=256, H=1024, P=256, S=1024.0, seed=72),
    "biglstm": dict(T=20, B=2048, I=1024, H=8192, P=1024, S=1024.0, seed=73),
}


def lstm_tensors(cfg, fast=False):
    """Seeded FP16 tensors of one LSTM layer: x [T,B,I] ~ N(0,1); Wg [4H,I+P] and Wp [P,H] ~
    N(0, 1/fan_in) with gate-interleaved rows (row 4j+q: gate q of cell j); bias16 [4H] ~ N(0, 0.1)
    with +1 on the forget gates (the usual initialisation); r0 [B,P], c0 [B,H] ~ N(0, 0.25);
    dr_ext [T,B,P] ~ S * N(0, 1/B) (a mean-loss gradient scaled by the loss scale)."""
    T, B, I, H, P, S = cfg["T"], cfg["B"], cfg["I"], cfg["H"], cfg["P"], cfg["S"]
    ss = np.random.SeedSequence(cfg["seed"]).spawn(7)
    gen = (lambda q, shape, scale: normal_f16_fast(ss[q], shape, scale)) if fast else \
          (lambda q, shape, scale: normal_f16(np.random.default_rng(ss[q]), shape, scale))
    x = gen(0, (T, B, I), 1.0)
    Wg = gen(1, (4 * H, I + P), 1.0 / np.sqrt(I + P))
    Wp = gen(2, (P, H), 1.0 / np.sqrt(H))
    bias = gen(3, (4 * H,), 0.1).astype(np.float32)
    bias[1::4] += 1.0
    bias16 = bias.astype(np.float16)
    r0 = gen(4, (B, P), 0.5)
    c0 = gen(5, (B, H), 0.5)
    dr_ext = gen(6, (T, B, P), S / B)
    return dict(x=x, Wg=Wg, Wp=Wp, bias16=bias16, r0=r0, c0=c0, dr_ext=dr_ext)
