"""Pins for the CPU oracle: each oracle function is checked against something that is
not the oracle (numpy's binary16 casts, Python's struct 'e', exact rationals, closed
forms, finite differences in float64, values the paper states)."""
import math
import os
import struct
from concurrent.futures import ThreadPoolExecutor
from fractions import Fraction

import numpy as np
import pytest

from oracle import mpo
from oracle.mlp import OracleMLP
from paper_1710_03740_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_limits():
    out = {}
    for line in open(os.path.join(GOLDEN, "fp16_limits.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        out[k] = int(v)
    return out


def f32(x):
    return float(np.float32(x))


def bits32(x):
    return struct.unpack("<I", struct.pack("<f", x))[0]


# ----------------------------------------------------------------- binary16

def test_fp16_limits_from_paper():
    """Paper section 3.2: largest FP16 value 65504, normal exponents [-14, 15];
    section 3.1: 2^-24 is the smallest magnitude, 10 mantissa bits."""
    g = _golden_limits()
    L = mpo.lib()
    assert L.mpo_f2h(float(g["max_finite"])) == 0x7BFF
    assert L.mpo_h2f(0x7BFF) == float(g["max_finite"])
    assert L.mpo_f2h(65519.9) == 0x7BFF          # still rounds down to 65504
    assert L.mpo_f2h(65520.0) == 0x7C00          # first value that becomes inf
    assert L.mpo_f2h(-65520.0) == 0xFC00
    tiny = 2.0 ** g["min_subnormal_log2"]
    assert L.mpo_f2h(tiny) == 0x0001 and L.mpo_h2f(0x0001) == tiny
    assert L.mpo_f2h(2.0 ** -25) == 0x0000       # tie to even -> zero
    assert L.mpo_f2h(f32(2.0 ** -25 * (1 + 2.0 ** -23))) == 0x0001
    assert L.mpo_f2h(0.75 * 2.0 ** -24) == 0x0001
    assert L.mpo_f2h(0.49 * 2.0 ** -24) == 0x0000
    assert L.mpo_f2h(-(2.0 ** -26)) == 0x8000    # sign of zero kept
    assert L.mpo_f2h(2.0 ** g["min_normal_exponent"]) == 0x0400
    assert L.mpo_h2f(0x7BFF) < 2.0 ** (g["max_normal_exponent"] + 1)
    assert L.mpo_h2f(0x7800) == 2.0 ** g["max_normal_exponent"]
    # 10 fraction bits: 1 + 2^-10 is representable, 1 + 2^-11 ties to 1
    assert L.mpo_f2h(1.0 + 2.0 ** -g["fraction_bits"]) == 0x3C01
    assert L.mpo_f2h(1.0 + 2.0 ** -(g["fraction_bits"] + 1)) == 0x3C00
    assert L.mpo_f2h(float("inf")) == 0x7C00
    h = L.mpo_f2h(float("nan"))
    assert (h & 0x7C00) == 0x7C00 and (h & 0x3FF) != 0


def test_h2f_all_patterns_vs_numpy_and_struct():
    allh = np.arange(65536, dtype=np.uint16)
    got = mpo.h2f(allh)
    ref = allh.view(np.float16).astype(np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))
    # Python's struct 'e' is a second independent binary16 decoder
    for h in list(range(0, 65536, 37)) + [0x0001, 0x03FF, 0x0400, 0x7BFF, 0x8001, 0xFBFF]:
        v = struct.unpack("<e", struct.pack("<H", h))[0]
        if math.isnan(v):
            assert math.isnan(float(got[h]))
        else:
            assert float(got[h]) == v
    # round trip
    back = mpo.f2h(got)
    assert np.array_equal(back[~nan], allh[~nan])


def _check_chunk(first, count):
    got = mpo.f2h_bits_range(first, count)
    x = np.arange(first, first + count, dtype=np.uint32).view(np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    return bool(np.array_equal(got, ref))


def test_f2h_exhaustive_band_vs_numpy():
    """Every binary32 pattern with 2^-27 <= |x| < 2^17 (all patterns whose result is
    neither a plain zero nor a plain infinity), both signs, against numpy's cast."""
    lo, hi = 0x32000000, 0x48000000       # 2^-27 .. 2^17
    chunk = 1 << 24
    jobs = []
    for sign in (0, 0x80000000):
        for first in range(lo, hi, chunk):
            jobs.append((first | sign, chunk))
    with ThreadPoolExecutor(8) as ex:
        ok = list(ex.map(lambda j: _check_chunk(*j), jobs))
    assert all(ok)


def test_f2h_outside_band():
    """Below 2^-27 every value is a signed zero, from 2^17 to inf every value is a signed
    infinity, above inf every pattern is a NaN; checked on all patterns."""
    step = 1 << 26
    for sign, sbit in ((0, 0), (0x80000000, 0x8000)):
        for first in range(0, 0x32000000, step):
            n = min(step, 0x32000000 - first)
            assert np.all(mpo.f2h_bits_range(first | sign, n) == sbit)
        for first in range(0x48000000, 0x7F800001, step):
            n = min(step, 0x7F800001 - first)
            assert np.all(mpo.f2h_bits_range(first | sign, n) == (sbit | 0x7C00))
        for first in range(0x7F800001, 0x80000000, step):
            n = min(step, 0x80000000 - first)
            h = mpo.f2h_bits_range(first | sign, n)
            assert np.all((h & 0x7C00) == 0x7C00) and np.all((h & 0x3FF) != 0)
            assert np.all((h & 0x8000) == sbit)


def test_f2h_vs_struct_e_sample():
    rng = np.random.default_rng(7)
    xs = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-9, 5, 2000),
                         [65504.0, 65519.0, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -26, 1e-8]]).astype(np.float32)
    got = mpo.f2h(xs)
    for x, h in zip(xs, got):
        assert int(h) == struct.unpack("<H", struct.pack("<e", float(x)))[0]


def test_product_of_two_halfs_is_exact_in_binary32():
    """Every product of two binary16 values is exact in binary32, so fused and unfused
    accumulation agree in the GEMM."""
    pats = []
    for e in range(0, 31):
        for m in (0, 1, 0x155, 0x2AA, 0x3FE, 0x3FF):
            pats.append((e << 10) | m)
    pats = np.array(sorted(set(pats)), dtype=np.uint16)
    a = pats.view(np.float16).astype(np.float32)
    p32 = a[:, None] * a[None, :]
    p64 = a.astype(np.float64)[:, None] * a.astype(np.float64)[None, :]
    assert np.array_equal(p32.astype(np.float64), p64)


# --------------------------------------------------------------------- GEMM

def _frac_of_half(h):
    return Fraction(float(np.uint16(h).view(np.float16)))


def _rn16_rational(q: Fraction) -> int:
    """Exact rational -> binary16 bits, round to nearest even (test-local)."""
    if q == 0:
        return 0
    s = 0x8000 if q < 0 else 0
    a = abs(q)
    e = -14
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    quantum = Fraction(2) ** (e - 10)
    n = a / quantum
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    val = fl * quantum
    if val >= 65520:
        return s | 0x7C00
    return s | int(np.float16(float(val)).view(np.uint16))


def _stored(op, Aop, Bop):
    """Aop[M,K], Bop[K,N] logical -> stored arrays for `op`."""
    A = Aop.T.copy() if op == 2 else Aop.copy()
    B = Bop.T.copy() if op == 0 else Bop.copy()
    return A, B


@pytest.mark.parametrize("op", [0, 1, 2])
def test_gemm_bruteforce_exact_small_integers(op):
    """Operands are small integers times 2^-3: every partial sum fits 24 bits, so the
    binary32 accumulation is exact and the oracle must equal the exactly rounded sum."""
    rng = np.random.default_rng(100 + op)
    for (M, N, K) in [(1, 1, 1), (3, 4, 16), (4, 2, 7), (2, 3, 13)]:
        Aop = (rng.integers(-8, 9, (M, K)) / 8.0).astype(np.float16)
        Bop = (rng.integers(-8, 9, (K, N)) * 4.0).astype(np.float16)
        A, B = _stored(op, Aop, Bop)
        C = mpo.gemm_f16(op, A, B)
        for m in range(M):
            for n in range(N):
                q = sum(Fraction(float(Aop[m, k])) * Fraction(float(Bop[k, n])) for k in range(K))
                assert int(C[m, n]) == _rn16_rational(q), (op, M, N, K, m, n)


@pytest.mark.parametrize("op", [0, 1, 2])
def test_gemm_bruteforce_random_halfs_within_bound(op):
    """Random halfs including subnormals: result must be the rounding of a value within
    the a-priori summation bound K*2^-24*sum|a*b| of the exact rational sum; the exact
    side channel must equal the rational sum to double precision."""
    rng = np.random.default_rng(200 + op)
    M, N, K = 4, 4, 16
    for trial in range(6):
        scale = [1.0, 1e-3, 2.0 ** -18, 50.0, 1e-6, 1.0][trial]
        Aop = (rng.standard_normal((M, K)) * scale).astype(np.float16)
        Bop = (rng.standard_normal((K, N))).astype(np.float16)
        A, B = _stored(op, Aop, Bop)
        C, ex, ab = mpo.gemm_f16(op, A, B, want_exact=True)
        for m in range(M):
            for n in range(N):
                terms = [Fraction(float(Aop[m, k])) * Fraction(float(Bop[k, n])) for k in range(K)]
                q = sum(terms)
                absq = sum(abs(t) for t in terms)
                assert abs(Fraction(ex[m, n]) - q) <= absq * Fraction(1, 2 ** 45)
                assert abs(Fraction(ab[m, n]) - absq) <= absq * Fraction(1, 2 ** 45)
                bound = absq * K / 2 ** 24
                lo, hi = _rn16_rational(q - bound), _rn16_rational(q + bound)
                v = float(np.uint16(C[m, n]).view(np.float16))
                vlo = float(np.uint16(lo).view(np.float16))
                vhi = float(np.uint16(hi).view(np.float16))
                assert vlo <= v <= vhi, (op, trial, m, n)
        # element entry point agrees with the full product
        h, e1, a1 = mpo.gemm_f16_element(op, A, B, 2, 3)
        assert h == int(C[2, 3]) and e1 == ex[2, 3] and a1 == ab[2, 3]


def test_gemm_variants_are_transposes_of_forward():
    rng = np.random.default_rng(5)
    M, N, K = 5, 7, 33
    Aop = rng.standard_normal((M, K)).astype(np.float16)
    Bop = rng.standard_normal((K, N)).astype(np.float16)
    outs = []
    for op in (0, 1, 2):
        A, B = _stored(op, Aop, Bop)
        outs.append(mpo.gemm_f16(op, A, B))
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    # against float64 matmul rounded once (sums this short: at most 1 ulp16 apart)
    ref = (Aop.astype(np.float64) @ Bop.astype(np.float64)).astype(np.float16)
    d = np.abs(outs[0].view(np.float16).astype(np.float64) - ref.astype(np.float64))
    assert np.all(d <= np.abs(ref.astype(np.float64)) * 2.0 ** -9 + 1e-7)


def test_gemm_leading_dimensions_and_row_slab():
    rng = np.random.default_rng(6)
    big = rng.standard_normal((16, 40)).astype(np.float16)
    A = big[:9, :24]              # lda = 40
    Bfull = rng.standard_normal((11, 64)).astype(np.float16)
    B = Bfull[:, :24]
    C = mpo.gemm_f16(0, A, B)
    C2 = mpo.gemm_f16(0, np.ascontiguousarray(A), np.ascontiguousarray(B))
    assert np.array_equal(C, C2)
    C3 = mpo.gemm_f16(0, A, B, rows=(3, 6))
    assert np.array_equal(C3[3:6], C[3:6]) and not C3[:3].any() and not C3[6:].any()


def test_accumulation_is_fp32_not_fp16():
    """Section 3.3: partial products accumulate in FP32.  1 + 4095 * 2^-12 needs more than
    11 bits while summing: an FP16 accumulator would stay at 1.0."""
    K = 4096
    x = np.ones((1, K), dtype=np.float16)
    w = np.full((1, K), 2.0 ** -12, dtype=np.float16)
    w[0, 0] = 1.0
    C = mpo.gemm_f16(0, x, w)
    assert C[0, 0] == np.float16(2.0).view(np.uint16)
    # overflow happens on the store: the FP32 sum 65520 is finite, its FP16 rounding is inf
    K = 65520
    ones = np.ones((1, K), dtype=np.float16)
    C, ex, _ = mpo.gemm_f16(0, ones, ones, want_exact=True)
    assert ex[0, 0] == 65520.0 and C[0, 0] == 0x7C00
    C = mpo.gemm_f16(0, ones[:, :65519], ones[:, :65519])
    assert C[0, 0] == 0x7BFF


def test_relu_and_mask_edge_cases():
    # sums: negative, zero from cancellation, NaN, positive
    A = np.array([[1.0, -2.0], [1.0, -1.0], [np.nan, 1.0], [3.0, 1.0]], dtype=np.float16)
    B = np.array([[1.0, 1.0]], dtype=np.float16)       # N=1, K=2
    C = mpo.gemm_f16(0, A, B, relu=True)
    assert C[0, 0] == 0x0000                            # -1 -> +0
    assert C[1, 0] == 0x0000
    assert (C[2, 0] & 0x7C00) == 0x7C00 and (C[2, 0] & 0x3FF)   # NaN propagates
    assert C[3, 0] == np.float16(4.0).view(np.uint16)
    # mask from a stored activation: > 0 keeps, 0 / -0 / negative / NaN give +0
    mask = np.array([[1.0], [0.0], [-0.0], [np.nan]], dtype=np.float16)
    A2 = np.array([[1.0, 1.0]] * 4, dtype=np.float16)
    C = mpo.gemm_f16(0, A2, B, mask=mask)
    assert C[0, 0] == np.float16(2.0).view(np.uint16) and not C[1:, 0].any()


@pytest.mark.parametrize("op", [0, 1, 2])
def test_power_of_two_scaling_is_exact_in_gemm(op):
    """Section 3.2: scaling by the chain rule; for a power of two nothing changes but the
    exponent while values stay in range."""
    A, B = inputs.gemm_operands(op, 24, 40, 64, seed=9, scale_a=1.0, scale_b=1.0)
    C1 = mpo.gemm_f16(op, A, B).view(np.float16).astype(np.float32)
    A2 = (A.astype(np.float32) * 2.0 ** -6).astype(np.float16)
    C2 = mpo.gemm_f16(op, A2, B).view(np.float16).astype(np.float32)
    normal = np.abs(C2) >= 2.0 ** -14
    assert normal.mean() > 0.9
    assert np.array_equal(C1[normal] * np.float32(2.0 ** -6), C2[normal])


# --------------------------------------------------------------- softmax-CE

def test_softmax_uniform_logits_closed_form():
    B, C, S = 8, 10, 1024.0
    z = np.zeros((B, C), dtype=np.float16)
    y = np.arange(B, dtype=np.int32) % C
    dz, rl, loss, bad = mpo.softmax_ce(z, y, S)
    assert bad == 0
    assert abs(loss - math.log(C)) < 1e-6
    exp_off = np.float16(np.float32(S / B) * np.float32(1.0 / C))
    exp_on = np.float16(np.float32(S / B) * (np.float32(1.0 / C) - np.float32(1.0)))
    d = dz.view(np.float16)
    for i in range(B):
        for j in range(C):
            want = exp_on if j == y[i] else exp_off
            assert abs(float(d[i, j]) - float(want)) <= abs(float(want)) * 2.0 ** -10


def test_softmax_vs_float64_and_invariants():
    rng = np.random.default_rng(3)
    B, C, S = 32, 57, 256.0
    z = (rng.standard_normal((B, C)) * 3).astype(np.float16)
    y = rng.integers(0, C, B).astype(np.int32)
    dz, rl, loss, _ = mpo.softmax_ce(z, y, S)
    z64 = z.astype(np.float64)
    m = z64.max(1, keepdims=True)
    p = np.exp(z64 - m)
    p /= p.sum(1, keepdims=True)
    ref_rl = -np.log(p[np.arange(B), y])
    assert np.allclose(rl, ref_rl, rtol=1e-5, atol=1e-6)
    assert abs(loss - ref_rl.mean()) <= 1e-5 * abs(ref_rl.mean())
    onehot = np.zeros((B, C))
    onehot[np.arange(B), y] = 1
    ref_dz = (p - onehot) * (S / B)
    got = dz.view(np.float16).astype(np.float64)
    assert np.all(np.abs(got - ref_dz) <= np.abs(ref_dz) * 2.0 ** -10 + 2.0 ** -24)
    # rows of the gradient sum to ~0 (sum_j p_j = 1)
    assert np.all(np.abs(got.sum(1)) <= C * (S / B) * 2.0 ** -10)
    # shift invariance for an exactly representable shift
    zs = (np.round(z.astype(np.float32) * 4) / 4).astype(np.float16)      # multiples of 1/4
    dz_a, _, loss_a, _ = mpo.softmax_ce(zs, y, S)
    dz_b, _, loss_b, _ = mpo.softmax_ce((zs.astype(np.float32) + 16.0).astype(np.float16), y, S)
    assert np.array_equal(dz_a, dz_b) and abs(loss_a - loss_b) <= 4e-6 * max(1.0, abs(loss_a))


def test_softmax_dominant_logit_needs_loss_scale():
    """z_y = 40 and the rest 0: the off-label probabilities are e^-40 ~ 2^-57.7, below
    anything FP16 holds unless S lifts them (section 3.2)."""
    C = 10
    z = np.zeros((1, C), dtype=np.float16)
    z[0, 3] = 40.0
    y = np.array([3], dtype=np.int32)
    dz, rl, loss, _ = mpo.softmax_ce(z, y, 1.0)
    # true loss (C-1)e^-40 ~ 4e-17 is far below FP32 resolution at m = 40: FP32 gives ~0
    assert abs(loss - (C - 1) * math.exp(-40)) <= 40 * 2.0 ** -23
    assert not dz.any() or np.all(dz.view(np.float16) == 0)
    dz2, _, _, _ = mpo.softmax_ce(z, y, 2.0 ** 48)
    off = dz2.view(np.float16)[0, 0]
    assert abs(float(off) - math.exp(-40) * 2.0 ** 48) <= math.exp(-40) * 2.0 ** 48 * 2.0 ** -9


def test_softmax_bad_label_and_ld():
    z = np.zeros((3, 16), dtype=np.float16)[:, :5]           # ldz = 16
    y = np.array([0, 7, -1], dtype=np.int32)
    dz, rl, loss, bad = mpo.softmax_ce(z, y, 1.0)
    assert bad == 2 and not dz[1].any() and not dz[2].any() and rl[1] == 0 and rl[2] == 0
    assert abs(loss - math.log(5) / 3) < 1e-6


# ------------------------------------------------------- master-weight pass

def _one_weight(w, g16, lr, S=1.0, mu=0.0, steps=1):
    net = OracleMLP([(1, 1, 0)], S, lr, mu)
    net.set_master(0, np.array([[w]], dtype=np.float32))
    hist = []
    for _ in range(steps):
        net.set_grad(0, np.array([[g16]], dtype=np.float16))
        fl = net.step()
        hist.append((fl, float(net.w32[0][0, 0]), int(net.w16[0][0, 0])))
    return hist


def test_master_copy_keeps_updates_fp16_drops():
    """Section 3.1: an update 2^-12 relative to the weight is absorbed by an FP16 weight;
    the FP32 master keeps it and the FP16 copy moves once enough has accumulated."""
    h = _one_weight(1.0, 2.0 ** -11, 0.5, steps=2)
    assert h[0] == (0, 1.0 - 2.0 ** -12, 0x3C00)       # tie to even: FP16 copy still 1.0
    assert h[1] == (0, 1.0 - 2.0 ** -11, 0x3BFF)
    # FP16-only weight: 1.0 - 2^-12 rounds back to 1.0 every time
    assert np.float16(np.float32(1.0) - np.float32(2.0 ** -12)) == np.float16(1.0)
    g = _golden_limits()
    assert 2 ** (g["fraction_bits"] + 1) == g["absorb_ratio"]
    # ratio sweep: update = w * 2^-j
    for j, moved in ((10, True), (11, True), (12, False), (13, False)):
        w16_after = np.float16(np.float32(1.0) + np.float32(2.0 ** -j))
        # 2^-11 is the exact tie: from 1.0 (even) it is lost, from 1+2^-10 (odd) rounding recovers it
        if j == 11:
            assert w16_after == np.float16(1.0)
            assert np.float16(np.float32(1.0 + 2.0 ** -10) + np.float32(2.0 ** -11)) > np.float16(1.0 + 2.0 ** -10)
        else:
            assert (w16_after != np.float16(1.0)) == moved
        hist = _one_weight(1.0, 2.0 ** -j, -1.0)
        assert hist[0][1] == 1.0 + 2.0 ** -j           # the master always keeps it


def test_master_copy_keeps_updates_below_fp16_range():
    """Section 3.1: lr*g below 2^-24 cannot be held in FP16 at all."""
    h = _one_weight(0.0, 2.0 ** -20, 2.0 ** -6, steps=3)
    assert [x[1] for x in h] == [-(2.0 ** -26), -(2.0 ** -25), -3 * 2.0 ** -26]
    assert [x[2] for x in h] == [0x8000, 0x8000, 0x8001]
    assert mpo.lib().mpo_f2h(2.0 ** -26) == 0


def test_update_rounds_each_operation_separately():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "fma_pairs.txt")) if not l.startswith("#")]
    assert len(rows) >= 20
    for kind, x, c, g, sep, fused in rows:
        x, c, g = (struct.unpack("<f", struct.pack("<I", int(v, 16)))[0] for v in (x, c, g))
        g16 = np.array([g], dtype=np.float16)
        assert float(g16[0]) == g
        w32 = np.array([x if kind == "sub" else 0.0], dtype=np.float32)
        v = np.array([0.0 if kind == "sub" else x], dtype=np.float32)
        w16 = np.zeros(1, dtype=np.uint16)
        if kind == "sub":
            mpo.update_apply(g16, w32, None, w16, 1.0, c, 0.0, False)
            assert bits32(float(w32[0])) == int(sep, 16) != int(fused, 16)
        else:
            mpo.update_apply(g16, w32, v, w16, 1.0, 0.0, c, True)
            assert bits32(float(v[0])) == int(sep, 16) != int(fused, 16)


@pytest.mark.parametrize("use_momentum", [False, True])
def test_update_vs_numpy_float32_ops(use_momentum):
    """numpy float32 array arithmetic rounds every operation separately."""
    rng = np.random.default_rng(11)
    n = 1 << 20
    w = rng.standard_normal(n).astype(np.float32)
    v = (rng.standard_normal(n) * 0.1).astype(np.float32)
    g16 = (rng.standard_normal(n) * 37.0).astype(np.float16)
    S, lr, mu = np.float32(128.0), np.float32(0.01), np.float32(0.9)
    inv = np.float32(1.0) / S
    g = g16.astype(np.float32) * inv
    if use_momentum:
        v_ref = mu * v + g
        w_ref = w - lr * v_ref
    else:
        v_ref = v.copy()
        w_ref = w - lr * g
    w16 = np.zeros(n, dtype=np.uint16)
    w2, v2 = w.copy(), v.copy()
    mpo.update_apply(g16, w2, v2, w16, inv, lr, mu, use_momentum)
    assert np.array_equal(w2.view(np.uint32), w_ref.view(np.uint32))
    assert np.array_equal(v2.view(np.uint32), v_ref.view(np.uint32))
    assert np.array_equal(w16, w_ref.astype(np.float16).view(np.uint16))


@pytest.mark.parametrize("kind", [0, 1, 2, 3])
@pytest.mark.parametrize("wd", [0.0, 1e-2])
def test_optimizer_variants_vs_numpy_float32_ops(kind, wd):
    """Nesterov / Adagrad / Adam / weight decay on the master copy (optimizers the paper's
    experiments use, sections 4.3, 4.5, 4.6; section 3.2: decay acts on the unscaled gradient):
    numpy float32 array arithmetic rounds every operation separately, in the same order."""
    rng = np.random.default_rng(40 + kind)
    n = 1 << 18
    w = rng.standard_normal(n).astype(np.float32)
    s1 = (np.abs(rng.standard_normal(n)) * 0.1).astype(np.float32)
    s2 = (np.abs(rng.standard_normal(n)) * 0.01).astype(np.float32)
    if kind in (0, 1):
        s1 = (rng.standard_normal(n) * 0.1).astype(np.float32)
    g16 = (rng.standard_normal(n) * 37.0).astype(np.float16)
    f = np.float32
    S, lr, mu, b2, eps, wdf = f(128.0), f(0.01), f(0.9), f(0.999), f(1e-8), f(wd)
    bc1, bc2 = f(1.0) - f(0.9) ** 3, f(1.0) - f(0.999) ** 3
    inv = f(1.0) / S
    g = g16.astype(np.float32) * inv
    if wd:
        g = g + wdf * w
    s1r, s2r = s1.copy(), s2.copy()
    if kind == 0:
        s1r = mu * s1 + g
        u = lr * s1r
    elif kind == 1:
        s1r = mu * s1 + g
        u = lr * (g + mu * s1r)
    elif kind == 2:
        s1r = s1 + g * g
        u = lr * (g / (np.sqrt(s1r) + eps))
    else:
        s1r = mu * s1 + (f(1.0) - mu) * g
        s2r = b2 * s2 + (f(1.0) - b2) * (g * g)
        u = lr * ((s1r / bc1) / (np.sqrt(s2r / bc2) + eps))
    w_ref = w - u
    w2, a1, a2 = w.copy(), s1.copy(), s2.copy()
    h = np.zeros(n, dtype=np.uint16)
    mpo.update_apply_opt(kind, g16, w2, a1, a2 if kind == 3 else None, h, inv, lr, mu, b2, eps, wdf, bc1, bc2)
    assert np.array_equal(w2.view(np.uint32), w_ref.view(np.uint32))
    assert np.array_equal(a1.view(np.uint32), s1r.astype(np.float32).view(np.uint32))
    if kind == 3:
        assert np.array_equal(a2.view(np.uint32), s2r.astype(np.float32).view(np.uint32))
    assert np.array_equal(h, w_ref.astype(np.float16).view(np.uint16))
    if kind == 0 and not wd:     # the generic entry point agrees with the SGD+momentum one
        w3, v3, h3 = w.copy(), s1.copy(), np.zeros(n, dtype=np.uint16)
        mpo.update_apply(g16, w3, v3, h3, inv, lr, mu, True)
        assert w3.tobytes() == w2.tobytes() and v3.tobytes() == a1.tobytes() and h3.tobytes() == h.tobytes()


def test_optimizer_first_step_closed_forms():
    """From zero state: Adam's bias-corrected first update is lr*g/(|g|+eps), Adagrad's is the
    same expression, Nesterov's is lr*(1+mu)*g, and decay adds wd*w to the unscaled gradient."""
    g16 = np.array([0.5, -2.0, 3.0, -0.125], dtype=np.float16)
    g = g16.astype(np.float64)
    lr, eps = 0.01, 1e-8
    for kind, want in ((3, lr * g / (np.abs(g) + eps)), (2, lr * g / (np.abs(g) + eps)), (1, lr * 1.9 * g)):
        net = OracleMLP([(4, 1, 0)], 1.0, lr, 0.0)
        net.set_master(0, np.zeros((1, 4), dtype=np.float32))
        net.set_optimizer(kind, lr, mu=0.9, b2=0.999, eps=eps)
        net.set_grad(0, g16.reshape(1, 4))
        assert net.step() == 0
        assert np.allclose(-net.w32[0][0].astype(np.float64), want, rtol=2e-6, atol=0)
    net = OracleMLP([(4, 1, 0)], 1.0, lr, 0.0)
    w0 = np.array([[1.0, -2.0, 4.0, 8.0]], dtype=np.float32)
    net.set_master(0, w0)
    net.set_optimizer(0, lr, wd=0.5)
    net.set_grad(0, g16.reshape(1, 4))
    net.step()
    assert np.allclose(net.w32[0][0].astype(np.float64), w0[0] - lr * (g + 0.5 * w0[0]), rtol=1e-6)
    # Adam's bias correction uses the number of APPLIED steps: a skipped step does not advance it
    net = OracleMLP([(4, 1, 0)], 1.0, lr, 0.0)
    net.set_master(0, np.zeros((1, 4), dtype=np.float32))
    net.set_optimizer(3, lr, mu=0.9, b2=0.999, eps=eps)
    bad = g16.copy()
    bad[0] = np.inf
    net.set_grad(0, bad.reshape(1, 4))
    assert net.step() == 1 and float(net.b1t) == 1.0 and not net.w32[0].any()
    net.set_grad(0, g16.reshape(1, 4))
    assert net.step() == 0
    assert np.allclose(-net.w32[0][0].astype(np.float64), lr * g / (np.abs(g) + eps), rtol=2e-6)


def test_global_norm_clipping_closed_forms():
    """Section 3.2: clipping acts on the unscaled gradients.  Known norm (3-4-5 triangle spread
    over two layers), coefficient min(1, clip/norm), update equal to numpy float32 arithmetic,
    and independence from the loss scale."""
    f = np.float32
    for S in (1.0, 256.0):
        net = OracleMLP([(2, 1, 1), (1, 1, 0)], S, 0.5, 0.0)
        net.set_master(0, np.array([[1.0, 2.0]], dtype=np.float32))
        net.set_master(1, np.array([[3.0]], dtype=np.float32))
        net.set_optimizer(0, 0.5, clip=2.5)
        net.set_grad(0, (np.array([[3.0, 0.0]]) * S).astype(np.float16))
        net.set_grad(1, (np.array([[4.0]]) * S).astype(np.float16))
        assert net.step() == 0
        coef = f(2.5 / (5.0 + 1e-6))
        assert float(net.last_coef) == float(coef)
        assert float(net.w32[0][0, 0]) == float(f(1.0) - f(0.5) * (f(3.0) * coef))
        assert float(net.w32[0][0, 1]) == 2.0
        assert float(net.w32[1][0, 0]) == float(f(3.0) - f(0.5) * (f(4.0) * coef))
    # a bound that binary32 cannot hold (0.3): the optimizer's parameter is a binary32 number, so the
    # quotient is formed from float32(0.3); with the 3-4-5 gradient the two readings give different
    # binary32 coefficients (0x3D75C28D from the rounded bound, one code lower from the double 0.3)
    net = OracleMLP([(2, 1, 0)], 1.0, 0.5, 0.0)
    net.set_master(0, np.zeros((1, 2), dtype=np.float32))
    net.set_optimizer(0, 0.5, clip=0.3)
    net.set_grad(0, np.array([[3.0, 4.0]], dtype=np.float16))
    net.step()
    want = f(float(f(0.3)) / (5.0 + 1e-6))
    other = f(0.3 / (5.0 + 1e-6))
    assert want.view(np.uint32) == 0x3D75C28D and other.view(np.uint32) == 0x3D75C28C
    assert np.float32(net.last_coef).view(np.uint32) == 0x3D75C28D
    assert np.float32(mpo.clip_coef(25.0, 0.3)).view(np.uint32) == 0x3D75C28D
    assert float(net.w32[0][0, 0]) == float(f(0.0) - f(0.5) * (f(3.0) * want))
    # a norm under the bound leaves the gradient alone (coefficient exactly 1)
    net = OracleMLP([(2, 1, 0)], 1.0, 0.5, 0.0)
    net.set_master(0, np.zeros((1, 2), dtype=np.float32))
    net.set_optimizer(0, 0.5, clip=10.0)
    net.set_grad(0, np.array([[3.0, 4.0]], dtype=np.float16))
    net.step()
    assert float(net.last_coef) == 1.0 and net.w32[0].tolist() == [[-1.5, -2.0]]
    # the sum of squares against numpy float64 on random data, and the generic step against numpy
    rng = np.random.default_rng(77)
    n = 1 << 16
    g16 = (rng.standard_normal(n) * 20).astype(np.float16)
    inv = f(1.0) / f(64.0)
    ref = float(((g16.astype(np.float32) * inv).astype(np.float64) ** 2).sum())
    got = mpo.grad_sqnorm(g16, inv)
    assert abs(got - ref) <= 1e-12 * ref
    coef = mpo.clip_coef(got, 1.0)
    w = rng.standard_normal(n).astype(np.float32)
    v = (rng.standard_normal(n) * 0.1).astype(np.float32)
    g = (g16.astype(np.float32) * inv) * coef
    g = g + f(1e-2) * w
    v_ref = f(0.9) * v + g
    w_ref = w - f(0.01) * (g + f(0.9) * v_ref)
    w2, v2, h = w.copy(), v.copy(), np.zeros(n, dtype=np.uint16)
    mpo.update_apply_clip(1, g16, w2, v2, None, h, inv, coef, f(0.01), f(0.9), wd=f(1e-2))
    assert np.array_equal(w2.view(np.uint32), w_ref.view(np.uint32)) and np.array_equal(v2.view(np.uint32), v_ref.view(np.uint32))


def test_overflow_detect_and_skip():
    """Section 3.2: an inf/NaN in any weight gradient skips the update."""
    layers = [(8, 6, 1), (6, 4, 0)]
    rng = np.random.default_rng(2)
    for bad in (np.inf, -np.inf, np.nan):
        for where in (0, 1):
            net = OracleMLP(layers, 4.0, 0.1, 0.9)
            for l, (i, o, _) in enumerate(layers):
                net.set_master(l, rng.standard_normal((o, i)).astype(np.float32))
                net.set_grad(l, rng.standard_normal((o, i)).astype(np.float16))
            assert net.step() == 0                       # finite: updates
            before = [(a.copy(), b.copy(), c.copy()) for a, b, c in zip(net.w32, net.v, net.w16)]
            g = net.g16[where].view(np.float16).copy()
            g[-1, -1] = bad
            net.set_grad(where, g)
            assert net.step() == 1
            for (a, b, c), a2, b2, c2 in zip(before, net.w32, net.v, net.w16):
                assert a.tobytes() == a2.tobytes() and b.tobytes() == b2.tobytes() and c.tobytes() == c2.tobytes()
    # the largest finite FP16 gradient is not an overflow
    assert mpo.grad_nonfinite(np.array([65504.0, -65504.0], dtype=np.float16), 1.0) == 0
    assert mpo.grad_nonfinite(np.array([1.0, np.inf], dtype=np.float16), 1.0 / 1024) == 1


def test_loguniform_gradient_survival_fractions():
    """Section 3.2 / 3.1: magnitudes 2^U, U ~ U(-40,-10); after multiplying by S the
    fraction that is non-zero in FP16 is the share of U above -25 - log2 S."""
    n = 1 << 22
    for S, frac in ((1.0, 15 / 30), (2.0 ** 8, 23 / 30), (2.0 ** 16, 1.0), (2.0 ** 24, 1.0)):
        g = inputs.loguniform_grads(n, S)
        nz = float((g != 0).mean())
        assert abs(nz - frac) < 4e-3, (S, nz, frac)
        assert np.isfinite(g.astype(np.float32)).all()
        inv = np.float32(1.0) / np.float32(S)
        assert mpo.grad_nonfinite(g, inv) == 0
    assert float(np.abs(inputs.loguniform_grads(n, 2.0 ** 24).astype(np.float32)).max()) <= 2.0 ** 14


# -------------------------------------------------------------- whole MLP

def _mlp_float64_loss(ws, x, y):
    a = x
    for l, w in enumerate(ws):
        a = a @ w.T
        if l < len(ws) - 1:
            a = np.maximum(a, 0.0)
    m = a.max(1, keepdims=True)
    lse = m[:, 0] + np.log(np.exp(a - m).sum(1))
    return float((lse - a[np.arange(len(y)), y]).mean())


def test_backward_matches_finite_differences():
    """The oracle's weight gradients (FP16, scaled) against central differences of a
    float64 forward pass written with numpy only."""
    rng = np.random.default_rng(21)
    layers = [(12, 16, 1), (16, 9, 1), (9, 5, 0)]
    B, S = 8, 256.0
    net = OracleMLP(layers, S, 0.0)
    ws = []
    for l, (i, o, _) in enumerate(layers):
        w = (rng.standard_normal((o, i)) * i ** -0.5).astype(np.float16).astype(np.float32)
        net.set_master(l, w)
        ws.append(w.astype(np.float64))
    x = rng.standard_normal((B, 12)).astype(np.float16)
    y = rng.integers(0, 5, B).astype(np.int32)
    net.forward(x)
    loss = net.backward_scaled(y)
    x64 = x.astype(np.float64)
    assert abs(loss - _mlp_float64_loss(ws, x64, y)) < 5e-3
    h = 1e-5
    for l in range(len(layers)):
        g = net.g16[l].view(np.float16).astype(np.float64) / S
        num = np.zeros_like(g)
        for idx in np.ndindex(*g.shape):
            wp = [w.copy() for w in ws]
            wp[l][idx] += h
            wm = [w.copy() for w in ws]
            wm[l][idx] -= h
            num[idx] = (_mlp_float64_loss(wp, x64, y) - _mlp_float64_loss(wm, x64, y)) / (2 * h)
        scale = np.abs(num).max()
        assert np.all(np.abs(g - num) <= 0.02 * scale + 1e-6), (l, np.abs(g - num).max(), scale)


def _run(cfg, S, steps, masters=None, head_shrink=1.0):
    cfg = dict(cfg)
    net = OracleMLP(cfg["layers"], S, cfg["lr"], cfg["momentum"])
    ms = inputs.mlp_masters(cfg) if masters is None else masters
    for l, w in enumerate(ms):
        if l == len(ms) - 1 and head_shrink != 1.0:
            w = (w * np.float32(head_shrink)).astype(np.float16).astype(np.float32)
        net.set_master(l, w)
    X, Y = inputs.mlp_batches(cfg, steps)
    flags, losses, grads = [], [], []
    for t in range(steps):
        net.forward(X[t])
        losses.append(net.backward_scaled(Y[t]))
        grads.append([g.copy() for g in net.g16])
        flags.append(net.step())
    return net, flags, losses, grads


def test_power_of_two_loss_scale_is_exact_end_to_end():
    """Section 3.2: with every gradient FP16-normal at S=1, training at S=1 and S=2^10 gives
    bit-identical unscaled gradients and masters.  Shrinking the head so gradients leave
    the normal range breaks the identity exactly on elements that lost bits at S=1."""
    cfg = dict(layers=[(32, 48, 1), (48, 6, 0)], batch=4, lr=0.05, momentum=0.0, steps=3, seed=33,
               head_scale=1.0)
    n1, f1, l1, g1 = _run(cfg, 1.0, 3)
    n2, f2, l2, g2 = _run(cfg, 2.0 ** 10, 3)
    assert f1 == [0, 0, 0] and f2 == [0, 0, 0]
    g1f = [g.view(np.float16).astype(np.float32) for g in g1[0]]
    g2f = [g.view(np.float16).astype(np.float32) for g in g2[0]]
    identical_everywhere = all(np.array_equal(a * np.float32(1024.0), b) for a, b in zip(g1f, g2f))
    if identical_everywhere:
        for a, b in zip(n1.w32, n2.w32):
            assert a.tobytes() == b.tobytes()
        assert l1 == l2
    else:
        # elements that differ must be ones whose S=1 value is subnormal/zero in FP16
        for a, b in zip(g1f, g2f):
            diff = (a * np.float32(1024.0)) != b
            assert np.all(np.abs(a[diff]) < 2.0 ** -14)
    # shrink the head: hidden-layer gradients underflow at S=1 but not at S=2^10
    n3, _, _, g3 = _run(cfg, 1.0, 1, head_shrink=2.0 ** -12)
    n4, _, _, g4 = _run(cfg, 2.0 ** 10, 1, head_shrink=2.0 ** -12)
    a = g3[0][0].view(np.float16).astype(np.float32)
    b = g4[0][0].view(np.float16).astype(np.float32)
    diff = (a * np.float32(1024.0)) != b
    assert diff.any()
    assert np.all(np.abs(a[diff]) < 2.0 ** -14)         # only values outside the normal range lost bits
    assert np.array_equal((a * np.float32(1024.0))[~diff], b[~diff])


def test_scale_sweep_first_step_structure():
    """Config 2a, first step: at S=1 the activation gradients below the head are all under
    2^-25 and round to zero, so layers 1-3 receive all-zero weight gradients and their
    masters do not move; at S=2^16 they are non-zero; at S=2^24 the head overflows."""
    cfg = inputs.MLP_CONFIGS["scale_sweep"]
    masters = inputs.mlp_masters(cfg)
    res = {}
    for S in (1.0, 2.0 ** 16, 2.0 ** 24):
        net, flags, losses, grads = _run(cfg, S, 1, masters=masters)
        res[S] = (net, flags, losses, grads[0])
        assert abs(losses[0] - math.log(10)) < 1e-2
    net1, f1, _, g1 = res[1.0]
    assert f1 == [0]
    for l in range(3):
        assert not g1[l].any()
        assert net1.w32[l].tobytes() == masters[l].tobytes()
    assert (g1[3] != 0).mean() > 0.9
    # float64 view of the true activation gradient under the head (numpy only)
    X, Y = inputs.mlp_batches(cfg, 1)
    a = X[0].astype(np.float64)
    for l in range(3):
        a = np.maximum(a @ masters[l].astype(np.float64).T, 0)
    z = a @ masters[3].astype(np.float64).T
    p = np.exp(z - z.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    p[np.arange(len(Y[0])), Y[0]] -= 1
    dz3 = (p / len(Y[0])) @ masters[3].astype(np.float64)
    assert np.abs(dz3).max() < 2.0 ** -25
    _, f16, _, g16 = res[2.0 ** 16]
    assert f16 == [0]
    for l in range(3):
        assert (g16[l] != 0).mean() > 0.5
    net24, f24, _, g24 = res[2.0 ** 24]
    assert f24 == [1]
    gh = g24[3].view(np.float16)
    assert (~np.isfinite(gh.astype(np.float32))).mean() > 0.05
    for l in range(4):
        assert net24.w32[l].tobytes() == masters[l].tobytes()


def test_overflowing_scale_skips_every_step_twin():
    """Section 3.2: S=2^24 overflows on each of the 20 steps; the master never moves."""
    cfg = inputs.MLP_CONFIGS["scale_sweep_twin"]
    masters = inputs.mlp_masters(cfg)
    net, flags, losses, _ = _run(cfg, 2.0 ** 24, cfg["steps"], masters=masters)
    assert flags == [1] * 20
    for l in range(4):
        assert net.w32[l].tobytes() == masters[l].tobytes()
        assert not net.v[l].any()
    net, flags, losses, _ = _run(cfg, 2.0 ** 16, cfg["steps"], masters=masters)
    assert flags == [0] * 20
    assert losses[-1] < losses[0]


def test_dynamic_scale_schedule_hand_trace():
    """Dynamic loss scaling (paper section 5: raise or lower the factor by inspecting the weight
    gradients for overflow, skipping overflowing updates).  One weight, injected gradients: the
    scale after each step is worked out by hand for interval 3, bounds [2, 64], start 16."""
    net = OracleMLP([(1, 1, 0)], 16.0, 0.5, 0.0)
    net.set_master(0, np.array([[1.0]], dtype=np.float32))
    net.set_dynamic_scale(3, 2.0, 64.0)
    inf, ok = np.float16(np.inf), np.float16(16.0)          # 16/S is the unscaled gradient
    seq = [ok, ok, ok, ok, inf, ok, ok, inf, inf, inf, inf, ok, ok, ok, ok, ok, ok, ok, ok, ok]
    # S used by each step:    16  16  16  32  32   16  16  16   8    4    2   2   2   2   4   4   4   8   8   8
    want_S_after = [16, 16, 32, 32, 16, 16, 16, 8, 4, 2, 2, 2, 2, 4, 4, 4, 8, 8, 8, 16]
    want_flag = [0, 0, 0, 0, 1, 0, 0, 1, 1, 1, 1, 0, 0, 0, 0, 0, 0, 0, 0, 0]
    w = 1.0
    for t, g in enumerate(seq):
        S_used = float(net.S)
        net.set_grad(0, np.array([[g]], dtype=np.float16))
        flag = net.step()
        assert flag == want_flag[t] and float(net.S) == want_S_after[t], (t, flag, float(net.S))
        if not flag:
            w = float(np.float32(w) - np.float32(0.5) * np.float32(16.0 / S_used))
        assert float(net.w32[0][0, 0]) == w                 # skipped steps leave the master alone
    # clamp at the upper bound
    net2 = OracleMLP([(1, 1, 0)], 32.0, 0.5, 0.0)
    net2.set_master(0, np.array([[1.0]], dtype=np.float32))
    net2.set_dynamic_scale(1, 2.0, 64.0)
    for want in (64, 64, 64):
        net2.set_grad(0, np.array([[1.0]], dtype=np.float16))
        net2.step()
        assert float(net2.S) == want


def test_dynamic_scale_recovers_from_an_overflowing_start():
    """Twin of the scale-sweep network started at S = 2^24 (overflows, section 3.2): the scale
    backs off until steps go through, no skipped step moves the master, and from then on the
    run is bit-identical to a constant-scale run started at the settled scale from the same
    masters (power-of-two scales only change exponents)."""
    cfg = dict(inputs.MLP_CONFIGS["scale_sweep_twin"])
    masters = inputs.mlp_masters(cfg)
    X, Y = inputs.mlp_batches(cfg, 12)
    net = OracleMLP(cfg["layers"], 2.0 ** 24, cfg["lr"], cfg["momentum"])
    for l, w in enumerate(masters):
        net.set_master(l, w)
    net.set_dynamic_scale(1000, 1.0, 2.0 ** 24)
    flags, scales = [], []
    for t in range(12):
        net.forward(X[t])
        net.backward_scaled(Y[t])
        scales.append(float(net.S))
        flags.append(net.step())
    n_skip = flags.index(0)
    assert n_skip >= 1 and flags[:n_skip] == [1] * n_skip and flags[n_skip:] == [0] * (12 - n_skip)
    assert scales[:n_skip + 1] == [2.0 ** (24 - i) for i in range(n_skip + 1)]
    ref = OracleMLP(cfg["layers"], scales[n_skip], cfg["lr"], cfg["momentum"])
    for l, w in enumerate(masters):
        ref.set_master(l, w)
    for t in range(n_skip, 12):
        ref.forward(X[t])
        ref.backward_scaled(Y[t])
        assert ref.step() == 0
    for l in range(len(masters)):
        assert ref.w32[l].tobytes() == net.w32[l].tobytes()


def test_tiny_config_trains():
    cfg = inputs.MLP_CONFIGS["tiny"]
    net, flags, losses, _ = _run(cfg, cfg["S"], cfg["steps"])
    assert flags == [0] * 10
    assert all(np.isfinite(losses))
    assert 1.5 < losses[0] < 4.0
