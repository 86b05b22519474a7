"""Parity of the master-weight pass with the oracle: bit-exact (paper sections 3.1, 3.2)."""
import numpy as np
import pytest

from oracle import mpo
from paper_1710_03740_b200 import inputs
from gpu_util import dev, host_u16, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _binding():
    from paper_1710_03740_b200 import binding
    return binding


@pytest.mark.parametrize("n", [0, 1, 7, 8, 1000, 4096 + 3, (1 << 20) + 5])
def test_recast_matches_oracle(n):
    b = _binding()
    rng = np.random.default_rng(n)
    w = (rng.standard_normal(n) * 10.0 ** rng.integers(-9, 6, n)).astype(np.float32)
    if n >= 8:
        w[:8] = [65504.0, 65519.9, 65520.0, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -26, -2.0 ** -26, np.inf]
    wd = dev(np.concatenate([w, np.zeros(1, np.float32)]))      # never an empty (null) buffer
    out = torch.zeros(n + 1, dtype=torch.int16, device="cuda")
    b.mpt_recast(wd, out, n)
    torch.cuda.synchronize()
    assert np.array_equal(host_u16(out)[:n], mpo.f2h(w))


def _run_update(n, use_momentum, S, lr, mu, g16, w, v, misalign=0, detect=True):
    b = _binding()
    pad = misalign
    gd = torch.zeros(n + 8, dtype=torch.int16, device="cuda")
    wd = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    vd = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    hd = torch.zeros(n + 8, dtype=torch.int16, device="cuda")
    gd[pad:pad + n] = dev(g16.view(np.uint16))
    wd[pad:pad + n] = dev(w)
    vd[pad:pad + n] = dev(v)
    flags = torch.zeros(2, dtype=torch.int32, device="cuda")
    inv = float(np.float32(1.0) / np.float32(S))
    b.mpt_update_flat(gd[pad:], wd[pad:], vd[pad:] if use_momentum else None, hd[pad:], n, inv, lr, mu,
                      use_momentum, detect, flags)
    torch.cuda.synchronize()
    return (wd[pad:pad + n].cpu().numpy(), vd[pad:pad + n].cpu().numpy(), host_u16(hd[pad:pad + n]),
            flags.cpu().numpy())


@pytest.mark.parametrize("use_momentum", [False, True])
@pytest.mark.parametrize("n,misalign", [(1, 0), (13, 0), (8 * 256 * 3 + 5, 0), ((1 << 21) + 11, 0), (5000, 1)])
def test_update_bit_exact(use_momentum, n, misalign):
    rng = np.random.default_rng(n + 17 * use_momentum)
    S, lr, mu = 512.0, 0.01, 0.9
    g16 = (rng.standard_normal(n) * 40.0).astype(np.float16)
    w = rng.standard_normal(n).astype(np.float32)
    v = (rng.standard_normal(n) * 0.1).astype(np.float32)
    if n > 100:
        g16[:6] = np.array([65504.0, -65504.0, 2.0 ** -24, -2.0 ** -24, 0.0, 6e-5], dtype=np.float16)
    w_ref, v_ref = w.copy(), v.copy()
    h_ref = np.zeros(n, dtype=np.uint16)
    inv = np.float32(1.0) / np.float32(S)
    assert mpo.grad_nonfinite(g16, inv) == 0
    mpo.update_apply(g16, w_ref, v_ref, h_ref, inv, np.float32(lr), np.float32(mu), use_momentum)
    w_g, v_g, h_g, flags = _run_update(n, use_momentum, S, lr, mu, g16, w, v, misalign)
    assert flags.tolist() == [0, 0]
    assert np.array_equal(w_g.view(np.uint32), w_ref.view(np.uint32))
    if use_momentum:
        assert np.array_equal(v_g.view(np.uint32), v_ref.view(np.uint32))
    else:
        assert np.array_equal(v_g.view(np.uint32), v.view(np.uint32))
    assert np.array_equal(h_g, h_ref)


def test_update_golden_fma_pairs():
    """Operands for which a fused multiply-add would change the last bit."""
    import os
    import struct
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "fma_pairs.txt"))
            if not l.startswith("#")]
    for kind, x, c, g, sep, fused in rows:
        x, c, g = (struct.unpack("<f", struct.pack("<I", int(t, 16)))[0] for t in (x, c, g))
        g16 = np.array([g] * 9, dtype=np.float16)
        if kind == "sub":
            w_g, _, _, _ = _run_update(9, False, 1.0, c, 0.0, g16, np.full(9, x, np.float32), np.zeros(9, np.float32))
            assert all(int(t) == int(sep, 16) for t in w_g.view(np.uint32))
        else:
            _, v_g, _, _ = _run_update(9, True, 1.0, 0.0, c, g16, np.zeros(9, np.float32), np.full(9, x, np.float32))
            assert all(int(t) == int(sep, 16) for t in v_g.view(np.uint32))


@pytest.mark.parametrize("bad", [np.inf, -np.inf, np.nan])
@pytest.mark.parametrize("pos", [0, 4097, -1])
def test_overflow_skips_everything(bad, pos):
    n = 10007
    rng = np.random.default_rng(3)
    g16 = rng.standard_normal(n).astype(np.float16)
    g16[pos] = bad
    w = rng.standard_normal(n).astype(np.float32)
    v = rng.standard_normal(n).astype(np.float32)
    assert mpo.grad_nonfinite(g16, 1.0) == 1
    w_g, v_g, h_g, flags = _run_update(n, True, 1.0, 0.1, 0.9, g16, w, v)
    assert flags[0] == 1
    assert w_g.tobytes() == w.tobytes() and v_g.tobytes() == v.tobytes() and not h_g.any()


def test_nonfinite_flag_matches_oracle_on_loguniform():
    b = _binding()
    n = 1 << 22
    for S in inputs.SCALE_SWEEP:
        g = inputs.loguniform_grads(n, S)
        inv = float(np.float32(1.0) / np.float32(S))
        flag = torch.zeros(1, dtype=torch.int32, device="cuda")
        b.mpt_grad_nonfinite(dev(g.view(np.uint16)), n, inv, flag)
        torch.cuda.synchronize()
        assert int(flag.item()) == mpo.grad_nonfinite(g, inv) == 0
    g = inputs.loguniform_grads(n, 1.0)
    g[-3] = np.inf
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.mpt_grad_nonfinite(dev(g.view(np.uint16)), n, 1.0, flag)
    assert int(flag.item()) == 1


def test_update_loguniform_config_2b_bit_exact():
    """Config 2b: 2^24 log-uniform gradients on a 4096x4096 layer, every scale of the sweep."""
    n = 1 << 24
    rng = np.random.default_rng(5)
    w = (rng.standard_normal(n) / 64).astype(np.float32)
    for S in inputs.SCALE_SWEEP:
        g16 = inputs.loguniform_grads(n, S)
        inv = np.float32(1.0) / np.float32(S)
        w_ref = w.copy()
        h_ref = np.zeros(n, dtype=np.uint16)
        mpo.update_apply(g16, w_ref, None, h_ref, inv, np.float32(0.01), np.float32(0.0), False)
        w_g, _, h_g, flags = _run_update(n, False, S, 0.01, 0.0, g16, w, np.zeros(1, np.float32).repeat(n))
        assert flags.tolist() == [0, 0]
        assert np.array_equal(w_g.view(np.uint32), w_ref.view(np.uint32))
        assert np.array_equal(h_g, h_ref)


@pytest.mark.parametrize("kind", [0, 1, 2, 3])
@pytest.mark.parametrize("wd", [0.0, 1e-2])
@pytest.mark.parametrize("n,misalign", [(8 * 256 * 5 + 3, 0), (4097, 1)])
def test_optimizer_variants_bit_exact(kind, wd, n, misalign):
    """Nesterov, Adagrad, Adam and weight decay on the master pass: bit for bit with the oracle."""
    b = _binding()
    if kind == 0 and wd == 0.0:
        pytest.skip("plain SGD(+momentum) is covered above")
    rng = np.random.default_rng(50 + kind)
    f = np.float32
    S, lr, mu, b2, eps = 256.0, 0.01, 0.9, 0.999, 1e-8
    g16 = (rng.standard_normal(n) * 30.0).astype(np.float16)
    w = rng.standard_normal(n).astype(np.float32)
    s1 = (np.abs(rng.standard_normal(n)) * 0.1).astype(np.float32)
    s2 = (np.abs(rng.standard_normal(n)) * 0.01).astype(np.float32)
    b1t, b2t = f(f(0.9) * f(0.9)), f(f(0.999) * f(0.999))                 # second applied step
    inv = f(1.0) / f(S)
    w_ref, a_ref, c_ref = w.copy(), s1.copy(), s2.copy()
    h_ref = np.zeros(n, dtype=np.uint16)
    mpo.update_apply_opt(kind, g16, w_ref, a_ref, c_ref if kind == 3 else None, h_ref, inv, f(lr), f(mu), f(b2), f(eps),
                         f(wd), f(1.0) - b1t, f(1.0) - b2t)
    pad = misalign
    gd = torch.zeros(n + 8, dtype=torch.int16, device="cuda")
    wd_ = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    ad = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    cd = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    hd = torch.zeros(n + 8, dtype=torch.int16, device="cuda")
    gd[pad:pad + n] = dev(g16.view(np.uint16)); wd_[pad:pad + n] = dev(w); ad[pad:pad + n] = dev(s1); cd[pad:pad + n] = dev(s2)
    flags = torch.zeros(2, dtype=torch.int32, device="cuda")
    opt = b.Optimizer(kind, lr, mu, b2, eps, wd)
    b.mpt_update_flat_opt(opt, gd[pad:], wd_[pad:], ad[pad:], cd[pad:] if kind == 3 else None, hd[pad:], n, float(inv),
                          float(b1t), float(b2t), True, flags)
    torch.cuda.synchronize()
    assert flags.tolist() == [0, 0]
    assert np.array_equal(wd_[pad:pad + n].cpu().numpy().view(np.uint32), w_ref.view(np.uint32))
    assert np.array_equal(ad[pad:pad + n].cpu().numpy().view(np.uint32), a_ref.view(np.uint32))
    if kind == 3:
        assert np.array_equal(cd[pad:pad + n].cpu().numpy().view(np.uint32), c_ref.view(np.uint32))
    assert np.array_equal(host_u16(hd[pad:pad + n]), h_ref)


@pytest.mark.parametrize("kind", [0, 1, 2, 3])
@pytest.mark.parametrize("n,misalign", [(1 << 20, 0), (300007, 0), (4099, 3), (5, 0)])
def test_clipped_update_bit_exact(kind, n, misalign):
    """Global-norm clipping in the stateless pass: the coefficient (double-precision norm over a
    fixed partition, rounded to FP32) equals the oracle's, and the update with it is bit-exact;
    unaligned arrays take the scalar path of both kernels."""
    from paper_1710_03740_b200 import binding as b
    f = np.float32
    rng = np.random.default_rng(1000 + n + kind)
    S, lr, clip = 1024.0, 0.01, 0.5
    g16 = (rng.standard_normal(n) * 30).astype(np.float16)
    w = rng.standard_normal(n).astype(np.float32)
    s1 = (np.abs(rng.standard_normal(n)) * 0.01).astype(np.float32)
    s2 = (np.abs(rng.standard_normal(n)) * 0.01).astype(np.float32)
    inv = f(1.0) / f(S)
    coef = mpo.clip_coef(mpo.grad_sqnorm(g16, inv), clip)
    assert coef < 1.0 or n == 5
    w_ref, a_ref, c_ref, h_ref = w.copy(), s1.copy(), s2.copy(), np.zeros(n, dtype=np.uint16)
    b1t, b2t = f(0.9), f(0.999)
    mpo.update_apply_clip(kind, g16, w_ref, a_ref, c_ref if kind == 3 else None, h_ref, inv, coef, f(lr), f(0.9), f(0.999),
                          f(1e-8), f(1e-3), f(1.0) - b1t, f(1.0) - b2t)
    pad = misalign
    gd = torch.zeros(n + 8, dtype=torch.int16, device="cuda")
    wd_ = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    ad = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    cd = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    hd = torch.zeros(n + 8, dtype=torch.int16, device="cuda")
    gd[pad:pad + n] = dev(g16.view(np.uint16)); wd_[pad:pad + n] = dev(w); ad[pad:pad + n] = dev(s1); cd[pad:pad + n] = dev(s2)
    flags = torch.zeros(2, dtype=torch.int32, device="cuda")
    scratch = torch.zeros(b.CLIP_SCRATCH_BYTES // 4, dtype=torch.float32, device="cuda")
    opt = b.Optimizer(kind, lr, 0.9, 0.999, 1e-8, 1e-3, clip)
    for _ in range(2):          # the second call checks that the result does not depend on leftover scratch
        wd_[pad:pad + n] = dev(w); ad[pad:pad + n] = dev(s1); cd[pad:pad + n] = dev(s2)
        b.mpt_update_flat_opt(opt, gd[pad:], wd_[pad:], ad[pad:], cd[pad:] if kind == 3 else None, hd[pad:], n, float(inv),
                              float(b1t), float(b2t), True, flags, clip_scratch=scratch)
        torch.cuda.synchronize()
        assert flags.tolist() == [0, 0]
        got = scratch[:2].cpu().numpy()
        assert got[0] == coef
        ref_norm = np.sqrt(((g16.astype(np.float32) * inv).astype(np.float64) ** 2).sum())
        assert abs(float(got[1]) - ref_norm) <= 1e-6 * ref_norm
        assert np.array_equal(wd_[pad:pad + n].cpu().numpy().view(np.uint32), w_ref.view(np.uint32))
        assert np.array_equal(ad[pad:pad + n].cpu().numpy().view(np.uint32), a_ref.view(np.uint32))
        assert np.array_equal(host_u16(hd[pad:pad + n]), h_ref)
    with pytest.raises(b.MptError):     # clipping without the scratch is refused
        b.mpt_update_flat_opt(opt, gd[pad:], wd_[pad:], ad[pad:], cd[pad:], hd[pad:], n, float(inv), 0.9, 0.999, True, flags)
