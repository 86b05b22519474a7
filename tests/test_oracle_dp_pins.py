"""Pins for the oracle's data-parallel step (section 4.5: a batch aggregated over several GPUs):
cases whose result is fixed by arithmetic that can be done by hand or by an already pinned routine."""
import numpy as np

from oracle import mpo
from paper_1710_03740_b200 import inputs


def _state(n, seed):
    rng = np.random.default_rng(seed)
    w32 = rng.standard_normal(n).astype(np.float32)
    v = (0.1 * rng.standard_normal(n)).astype(np.float32)
    return w32, v


def test_one_replica_is_the_plain_update():
    # R = 1: the sum has one term and 1/(S*1) = 1/S, so the step is the single-GPU update
    n = 4099
    g = inputs.loguniform_grads(n, 1024.0, seed=11).view(np.uint16)
    w32, v = _state(n, 1)
    wa, va, ha = w32.copy(), v.copy(), np.zeros(n, np.uint16)
    wb, vb, hb = w32.copy(), v.copy(), np.zeros(n, np.uint16)
    S = 1024.0
    mpo.dp_update_apply([g], wa, va, ha, S, 0.05, 0.9, True)
    mpo.update_apply(g, wb, vb, hb, np.float32(1.0) / np.float32(S), 0.05, 0.9, True)
    assert np.array_equal(wa.view(np.uint32), wb.view(np.uint32))
    assert np.array_equal(va.view(np.uint32), vb.view(np.uint32))
    assert np.array_equal(ha, hb)


def test_identical_replicas_power_of_two_equal_single_replica():
    # R = 4 copies of the same gradient, S a power of two: the binary32 sum is exactly 4*g and
    # 1/(4*S) is exact, so s * inv_SR == g * (1/S) exactly and the step equals the one-replica step
    n = 2048 + 5
    g = inputs.loguniform_grads(n, 256.0, seed=5).view(np.uint16)
    w32, v = _state(n, 2)
    wa, va, ha = w32.copy(), v.copy(), np.zeros(n, np.uint16)
    wb, vb, hb = w32.copy(), v.copy(), np.zeros(n, np.uint16)
    mpo.dp_update_apply([g, g.copy(), g.copy(), g.copy()], wa, va, ha, 256.0, 0.01, 0.5, True)
    mpo.update_apply(g, wb, vb, hb, np.float32(1.0 / 256.0), 0.01, 0.5, True)
    assert np.array_equal(wa.view(np.uint32), wb.view(np.uint32))
    assert np.array_equal(va.view(np.uint32), vb.view(np.uint32))
    assert np.array_equal(ha, hb)


def test_mean_of_small_integers_is_exact():
    # integer gradients, S = 1, R = 4, lr = 1, no momentum: every operation is exact, so
    # w - mean(g) must come out exactly (computed here in float64)
    rng = np.random.default_rng(3)
    n, R = 1000, 4
    gs = [rng.integers(-64, 65, n).astype(np.float16) for _ in range(R)]
    w0 = rng.integers(-1000, 1000, n).astype(np.float32)
    w, h = w0.copy(), np.zeros(n, np.uint16)
    mpo.dp_update_apply([g.view(np.uint16) for g in gs], w, None, h, 1.0, 1.0, 0.0, False)
    want = w0.astype(np.float64) - sum(g.astype(np.float64) for g in gs) / R
    assert np.array_equal(w.astype(np.float64), want)
    assert np.array_equal(h, want.astype(np.float16).view(np.uint16))


def test_sum_runs_in_ascending_replica_order_in_binary32():
    # replicas hold (65504, 2^-24, -65504): in ascending order the tiny term is absorbed by the
    # first addition (2^-24 is far below half an ulp of 65504 in binary32) and the sum is exactly 0;
    # any order that adds the two large terms first would leave 2^-24.  With S = 1, lr = 3 (so that
    # lr * g / 3 is visible), w0 = 0: ascending order leaves w = 0, another order gives -2^-24.
    big = np.array([65504.0], np.float16).view(np.uint16)
    tiny = np.array([0x0001], np.uint16)
    neg = np.array([-65504.0], np.float16).view(np.uint16)
    w, h = np.zeros(1, np.float32), np.zeros(1, np.uint16)
    mpo.dp_update_apply([big, tiny, neg], w, None, h, 1.0, 3.0, 0.0, False)
    assert w[0] == 0.0 and h[0] == 0
    w2, h2 = np.zeros(1, np.float32), np.zeros(1, np.uint16)
    mpo.dp_update_apply([big, neg, tiny], w2, None, h2, 1.0, 3.0, 0.0, False)
    # 1/(1*3) in binary32 times 2^-24 times 3 rounds back to 2^-24 (one ulp of slack allowed)
    assert abs(float(w2[0]) + 2.0 ** -24) <= 2.0 ** -47


def test_sum_is_not_rounded_to_binary16():
    # two replicas with 40000 each: the sum 80000 exceeds the binary16 range but is a legal binary32
    # intermediate; with S = 2 the unscaled mean is 20000 and w = 0 - 1 * 20000
    g = np.array([40000.0], np.float16).view(np.uint16)
    gval = float(g.view(np.float16)[0])     # 40000 is representable exactly in binary16
    assert gval == 40000.0
    w, h = np.zeros(1, np.float32), np.zeros(1, np.uint16)
    mpo.dp_update_apply([g, g.copy()], w, None, h, 2.0, 1.0, 0.0, False)
    assert w[0] == -20000.0
    assert h[0] == np.array([-20000.0], np.float16).view(np.uint16)[0]


def test_inverse_scale_is_one_division_of_the_binary32_product():
    assert mpo.dp_inv_scale(128.0, 4) == np.float32(1.0 / 512.0)
    # 3 replicas: 1/(S*3) is not exact; the value is the binary32 quotient, not a double rounded twice
    x = mpo.dp_inv_scale(1.0, 3)
    assert x == np.float32(1.0) / np.float32(3.0)


# ---- the replicated MLP iteration


def _mlp_setup(R, layers, S=128.0, lr=0.1, mu=0.9, seed=0):
    from oracle.dp import OracleDataParallelMLP
    from oracle.mlp import OracleMLP
    rng = np.random.default_rng(seed)
    dp, one = OracleDataParallelMLP(layers, S, lr, mu, R), OracleMLP(layers, S, lr, mu)
    for l, (i, o, _) in enumerate(layers):
        w = (rng.standard_normal((o, i)) * i ** -0.5).astype(np.float32)
        dp.set_master(l, w)
        one.set_master(l, w)
    return dp, one, rng


def test_mlp_one_replica_is_the_single_gpu_iteration():
    layers = [(16, 32, 1), (32, 10, 0)]
    dp, one, rng = _mlp_setup(1, layers)
    for t in range(3):
        x = rng.standard_normal((8, 16)).astype(np.float16)
        y = rng.integers(0, 10, 8).astype(np.int32)
        la = dp.forward_backward([x], [y])[0]
        one.forward(x)
        lb = one.backward_scaled(y)
        assert la == lb and dp.step() == one.step()
        for l in range(2):
            assert np.array_equal(dp.replicas[0].w32[l].view(np.uint32), one.w32[l].view(np.uint32))
            assert np.array_equal(dp.replicas[0].w16[l], one.w16[l])


def test_mlp_replicas_fed_the_same_batch_equal_one_replica():
    # R = 2 replicas see the same rows: both gradients are identical, their FP32 sum is exactly 2g,
    # and 1/(2S) is exact for S a power of two, so the run equals the single replica bit for bit
    layers = [(16, 24, 1), (24, 5, 0)]
    dp, one, rng = _mlp_setup(2, layers, S=64.0)
    for t in range(3):
        x = rng.standard_normal((8, 16)).astype(np.float16)
        y = rng.integers(0, 5, 8).astype(np.int32)
        dp.forward_backward([x, x.copy()], [y, y.copy()])
        one.forward(x)
        one.backward_scaled(y)
        assert dp.step() == one.step() == 0
        for q in range(2):
            for l in range(2):
                assert np.array_equal(dp.replicas[q].w32[l].view(np.uint32), one.w32[l].view(np.uint32))
                assert np.array_equal(dp.replicas[q].w16[l], one.w16[l])


def test_mlp_two_halves_approximate_the_full_batch_step():
    # mean of the half-batch mean gradients = full-batch mean gradient in exact arithmetic; with FP16
    # gradient storage the two runs differ by rounding only (a "sum instead of mean" mistake would
    # double the step, a dropped replica would change it by tens of percent)
    layers = [(32, 48, 1), (48, 10, 0)]
    dp, one, rng = _mlp_setup(2, layers, S=256.0, lr=0.5, mu=0.0)
    x = rng.standard_normal((64, 32)).astype(np.float16)
    y = rng.integers(0, 10, 64).astype(np.int32)
    w_before = [w.copy() for w in one.w32]
    dp.forward_backward([x[:32], x[32:]], [y[:32], y[32:]])
    one.forward(x)
    one.backward_scaled(y)
    assert dp.step() == one.step() == 0
    for l in range(2):
        da = dp.replicas[0].w32[l].astype(np.float64) - w_before[l]
        db = one.w32[l].astype(np.float64) - w_before[l]
        assert np.linalg.norm(da - db) <= 2e-2 * np.linalg.norm(db)
        assert np.array_equal(dp.replicas[0].w16[l], dp.replicas[1].w16[l])


def test_mlp_overflow_on_one_replica_skips_all_and_halves_every_scale():
    layers = [(8, 8, 0)]
    dp, _, rng = _mlp_setup(2, layers, S=1024.0)
    for r in dp.replicas:
        r.set_dynamic_scale(2, 1.0, 65536.0)
    before = [r.w32[0].copy() for r in dp.replicas]
    g = (rng.standard_normal((8, 8))).astype(np.float16)
    bad = g.copy()
    bad[2, 3] = np.float16(np.inf)
    dp.set_grad(0, 0, g.view(np.uint16))
    dp.set_grad(1, 0, bad.view(np.uint16))
    assert dp.step() == 1
    for q, r in enumerate(dp.replicas):
        assert np.array_equal(r.w32[0], before[q]) and r.S == np.float32(512.0)
    dp.set_grad(1, 0, g.view(np.uint16))
    assert dp.step() == 0 and dp.step() == 0        # two clean steps: the scale doubles again
    assert all(r.S == np.float32(1024.0) for r in dp.replicas)


# ---- other optimizers in the data-parallel step


import pytest


@pytest.mark.parametrize("kind", [mpo.OPT_SGD, mpo.OPT_NESTEROV, mpo.OPT_ADAGRAD, mpo.OPT_ADAM])
@pytest.mark.parametrize("wd", [0.0, 0.01])
def test_opt_one_replica_is_the_single_gpu_step(kind, wd):
    # R = 1: the sum has one term and 1/(S*1) = 1/S: the step is update_apply_opt (pinned elsewhere)
    n, S = 3001, 512.0
    g = inputs.loguniform_grads(n, S, seed=21).view(np.uint16)
    rng = np.random.default_rng(kind)
    w = rng.standard_normal(n).astype(np.float32)
    s1 = np.abs(0.1 * rng.standard_normal(n)).astype(np.float32)
    s2 = np.abs(0.01 * rng.standard_normal(n)).astype(np.float32)
    a = [w.copy(), s1.copy(), s2.copy(), np.zeros(n, np.uint16)]
    b = [w.copy(), s1.copy(), s2.copy(), np.zeros(n, np.uint16)]
    args = dict(b2=0.999, eps=1e-8, wd=wd, bc1=0.19, bc2=0.002)
    mpo.dp_update_apply_opt(kind, [g], a[0], a[1], a[2], a[3], S, 0.01, 0.9, **args)
    mpo.update_apply_opt(kind, g, b[0], b[1], b[2], b[3], np.float32(1.0) / np.float32(S), 0.01, 0.9, **args)
    for x, y in zip(a, b):
        assert np.array_equal(x.view(np.uint8), y.view(np.uint8))


@pytest.mark.parametrize("kind", [mpo.OPT_NESTEROV, mpo.OPT_ADAGRAD, mpo.OPT_ADAM])
def test_opt_identical_replicas_power_of_two_equal_single_replica(kind):
    # four copies of one gradient, S a power of two: s * 1/(4S) == g * 1/S exactly
    n, S = 2053, 128.0
    g = inputs.loguniform_grads(n, S, seed=22).view(np.uint16)
    rng = np.random.default_rng(kind + 10)
    w = rng.standard_normal(n).astype(np.float32)
    s1 = np.abs(0.1 * rng.standard_normal(n)).astype(np.float32)
    s2 = np.abs(0.01 * rng.standard_normal(n)).astype(np.float32)
    a = [w.copy(), s1.copy(), s2.copy(), np.zeros(n, np.uint16)]
    b = [w.copy(), s1.copy(), s2.copy(), np.zeros(n, np.uint16)]
    args = dict(b2=0.99, eps=1e-6, wd=0.0, bc1=0.1, bc2=0.01)
    mpo.dp_update_apply_opt(kind, [g, g.copy(), g.copy(), g.copy()], a[0], a[1], a[2], a[3], S, 0.02, 0.9, **args)
    mpo.update_apply_opt(kind, g, b[0], b[1], b[2], b[3], np.float32(1.0 / S), 0.02, 0.9, **args)
    for x, y in zip(a, b):
        assert np.array_equal(x.view(np.uint8), y.view(np.uint8))


def test_opt_adagrad_mean_of_integers_by_hand():
    # two replicas, gradients 3 and 5 (mean 4), S = 1, accumulator 9 -> 25, sqrt 5, eps 0:
    # w = 10 - 2 * 4 / 5 = 8.4 (rounded to binary32 as the oracle's operations do)
    g0 = np.array([3.0], np.float16).view(np.uint16)
    g1 = np.array([5.0], np.float16).view(np.uint16)
    w, s1, h = np.array([10.0], np.float32), np.array([9.0], np.float32), np.zeros(1, np.uint16)
    mpo.dp_update_apply_opt(mpo.OPT_ADAGRAD, [g0, g1], w, s1, None, h, 1.0, 2.0, 0.0, eps=0.0)
    assert s1[0] == 25.0
    assert w[0] == np.float32(10.0) - np.float32(2.0) * (np.float32(4.0) / np.float32(5.0))
    assert abs(float(w[0]) - 8.4) < 1e-6


@pytest.mark.parametrize("kind", [mpo.OPT_NESTEROV, mpo.OPT_ADAGRAD, mpo.OPT_ADAM])
def test_mlp_optimizer_replicas_fed_the_same_batch_equal_one_replica(kind):
    layers = [(16, 24, 1), (24, 5, 0)]
    dp, one, rng = _mlp_setup(2, layers, S=64.0)
    dp.set_optimizer(kind, 0.01, 0.9, b2=0.999, eps=1e-8, wd=0.001)
    one.set_optimizer(kind, 0.01, 0.9, b2=0.999, eps=1e-8, wd=0.001)
    for t in range(3):
        x = rng.standard_normal((8, 16)).astype(np.float16)
        y = rng.integers(0, 5, 8).astype(np.int32)
        dp.forward_backward([x, x.copy()], [y, y.copy()])
        one.forward(x)
        one.backward_scaled(y)
        assert dp.step() == one.step() == 0
        for q in range(2):
            for l in range(2):
                assert np.array_equal(dp.replicas[q].w32[l].view(np.uint32), one.w32[l].view(np.uint32))
                assert np.array_equal(dp.replicas[q].w16[l], one.w16[l])


def test_clip_one_replica_is_the_single_gpu_clip_and_identical_replicas_too():
    # R = 1: norm and update are those of the pinned single-GPU clipping; four identical replicas with
    # a power-of-two S have the same mean gradient bit for bit, hence the same norm and the same step
    n, S = 4099, 256.0
    g = inputs.loguniform_grads(n, S, seed=31).view(np.uint16)
    inv = np.float32(1.0) / np.float32(S)
    assert mpo.dp_grad_sqnorm([g], S) == mpo.grad_sqnorm(g, inv)
    assert mpo.dp_grad_sqnorm([g, g.copy(), g.copy(), g.copy()], S) == mpo.grad_sqnorm(g, inv)
    coef = mpo.clip_coef(mpo.grad_sqnorm(g, inv), 1e-4)
    assert 0.0 < float(coef) < 1.0
    rng = np.random.default_rng(3)
    w = rng.standard_normal(n).astype(np.float32)
    s1 = np.abs(0.1 * rng.standard_normal(n)).astype(np.float32)
    a = [w.copy(), s1.copy(), np.zeros(n, np.uint16)]
    b = [w.copy(), s1.copy(), np.zeros(n, np.uint16)]
    c = [w.copy(), s1.copy(), np.zeros(n, np.uint16)]
    mpo.dp_update_apply_clip(mpo.OPT_ADAGRAD, [g], a[0], a[1], None, a[2], S, coef, 0.05, 0.0, eps=1e-6)
    mpo.update_apply_clip(mpo.OPT_ADAGRAD, g, b[0], b[1], None, b[2], inv, coef, 0.05, 0.0, eps=1e-6)
    mpo.dp_update_apply_clip(mpo.OPT_ADAGRAD, [g, g.copy(), g.copy(), g.copy()], c[0], c[1], None, c[2], S, coef, 0.05, 0.0, eps=1e-6)
    for x, y, z in zip(a, b, c):
        assert np.array_equal(x.view(np.uint8), y.view(np.uint8)) and np.array_equal(x.view(np.uint8), z.view(np.uint8))


def test_clip_norm_is_taken_over_the_mean_gradient_by_hand():
    # two replicas with gradients (6, 0) and (0, 8), S = 1: the mean is (3, 4), norm 5 - not the
    # norm of either replica's gradient (6, 8) nor of their sum (10); bound 2.5 halves the step
    g0 = np.array([6.0, 0.0], np.float16).view(np.uint16)
    g1 = np.array([0.0, 8.0], np.float16).view(np.uint16)
    assert mpo.dp_grad_sqnorm([g0, g1], 1.0) == 25.0
    coef = mpo.clip_coef(25.0, 2.5)
    assert float(coef) == float(np.float32(2.5 / (5.0 + 1e-6)))
    w, h = np.zeros(2, np.float32), np.zeros(2, np.uint16)
    mpo.dp_update_apply_clip(mpo.OPT_SGD, [g0, g1], w, None, None, h, 1.0, coef, 1.0, 0.0)
    assert w[0] == -(np.float32(3.0) * coef) and w[1] == -(np.float32(4.0) * coef)


def test_mlp_clipped_replicas_fed_the_same_batch_equal_one_clipped_replica():
    layers = [(16, 24, 1), (24, 5, 0)]
    dp, one, rng = _mlp_setup(2, layers, S=64.0)
    dp.set_optimizer(mpo.OPT_SGD, 0.05, 0.9, clip=0.05)
    one.set_optimizer(mpo.OPT_SGD, 0.05, 0.9, clip=0.05)
    clipped = False
    for t in range(3):
        x = rng.standard_normal((8, 16)).astype(np.float16)
        y = rng.integers(0, 5, 8).astype(np.int32)
        dp.forward_backward([x, x.copy()], [y, y.copy()])
        one.forward(x)
        one.backward_scaled(y)
        assert dp.step() == one.step() == 0
        assert float(dp.replicas[0].last_coef) == float(one.last_coef)
        clipped |= float(one.last_coef) < 1.0
        for q in range(2):
            for l in range(2):
                assert np.array_equal(dp.replicas[q].w32[l].view(np.uint32), one.w32[l].view(np.uint32))
    assert clipped
