"""Parity at the full sizes of the isolated-GEMM sweep, the bigLSTM-shaped products and the
large-MLP step, in the launch configuration the benchmark times.  The oracle cannot run these
products in full, so sampled outputs are recomputed one by one (random elements, corners,
tile-boundary neighbours, whole rows), the softmax is recomputed in full and the master update
is compared bit for bit layer by layer.  Inside the MLP step every kernel is checked against
the oracle applied to the inputs that kernel read on the device."""
import numpy as np
import pytest

from oracle import mpo
from paper_1710_03740_b200 import inputs
from parity import gemm_accept
from gpu_util import dev, host_u16, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _host_ram_gb():
    import psutil
    return psutil.virtual_memory().available / 2 ** 30


def _sample_positions(M, N, rng, n_random=768):
    pos = {(0, 0), (0, N - 1), (M - 1, 0), (M - 1, N - 1)}
    for m in (127, 128, M // 2 - 1, M // 2):           # neighbours of 128-row tile edges
        for n in (255, 256, N // 2 - 1, N // 2):       # neighbours of 256-column tile edges
            if m < M and n < N:
                pos.add((m, n))
    ms = rng.integers(0, M, n_random)
    ns = rng.integers(0, N, n_random)
    pos.update(zip(ms.tolist(), ns.tolist()))
    return sorted(pos)


def _check_sampled(op, A, B, got, K, relu=False, mask=None, seed=0, full_rows=1, n_random=768):
    """got: full GPU output (uint16 [M,N]); A, B: the stored operands it was computed from."""
    M, N = got.shape
    rng = np.random.default_rng(seed)
    pos = _sample_positions(M, N, rng, n_random)
    g = np.empty(len(pos), dtype=np.uint16)
    r = np.empty(len(pos), dtype=np.uint16)
    ab = np.empty(len(pos))
    ex = np.empty(len(pos))
    for i, (m, n) in enumerate(pos):
        h, ex[i], a = mpo.gemm_f16_element(op, A, B, m, n, relu=relu)
        if mask is not None and not (np.float32(mask[m, n:n + 1].view(np.float16)[0]) > 0):
            h = 0
        g[i], r[i], ab[i] = got[m, n], h, a
    ok, stats = gemm_accept(g, r, K=K, absdot=ab, exact=ex)
    assert ok.all(), (op, got.shape, K, stats, [pos[i] for i in np.flatnonzero(~ok)[:8]])
    assert stats["max_ulp"] <= 2 or stats["by_abs_only"] + stats["by_rel_only"] > 0
    for row in rng.integers(0, M, full_rows).tolist():
        A1 = A[:, row:row + 1] if op == 2 else A[row:row + 1]          # the one output row's operand
        ref, exr, abr = mpo.gemm_f16(op, A1, B, relu=relu, mask=None if mask is None else mask[row:row + 1],
                                     want_exact=True)
        ok, st = gemm_accept(got[row], ref[0], K=K, absdot=abr[0], exact=exr[0])
        assert ok.all(), (op, "row", row, st)
    return stats


def _run(op, A, B, M, N, K, flags=0):
    from paper_1710_03740_b200 import binding as b
    Ad, Bd = dev(A.view(np.uint16)), dev(B.view(np.uint16))
    Cd = torch.empty((M, N), dtype=torch.int16, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    b.mpt_gemm_f16(op, M, N, K, Ad, A.shape[1], Bd, B.shape[1], Cd, N, flags, None, 0, None, status)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0
    return host_u16(Cd)


# 1024^3 and 2048^3 are compared element by element in test_gpu_gemm.py (test_tc_gemm_parity and
# test_sweep_2048_cubed_in_full_every_kernel); the larger shapes are sampled here
SHAPES = inputs.GEMM_SWEEP[2:] + [inputs.LSTM_GATE, inputs.LSTM_PROJ]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_gemm_sweep_and_lstm_shapes_sampled(M, N, K):
    if _host_ram_gb() < 16:
        pytest.skip("not enough host memory for full-size operands")
    lstm = (M, N, K) in (inputs.LSTM_GATE, inputs.LSTM_PROJ)
    for op in (0, 1, 2):
        # bigLSTM-shaped: activations N(0,1), weights N(0,1/K); sweep: both N(0,1)/sqrt(K)
        A, B = inputs.gemm_operands(op, M, N, K, seed=3 if lstm else 2, fast=True,
                                    scale_a=1.0 if lstm else None)
        got = _run(op, A, B, M, N, K)
        _check_sampled(op, A, B, got, K, seed=op)
        del A, B, got


@pytest.mark.parametrize("n", [2048 * 32768 + 8192 * 1024])
def test_lstm_sized_update_bit_exact_in_full(n):
    """Config-4-sized master pass (2 layers x (gate + projection) = 150,994,944 parameters, momentum
    0.9, S = 512): the whole arena, bit for bit.  Gradients have the magnitude structure of scaled
    weight gradients (Gaussian times S, a band of tiny values, FP16 extremes)."""
    from paper_1710_03740_b200 import binding as b
    n = 2 * n
    if _host_ram_gb() < 12:
        pytest.skip("not enough host memory")
    S, lr, mu = 512.0, 0.01, 0.9
    seqs = np.random.SeedSequence(3).spawn(3)
    g16 = inputs.normal_f16_fast(seqs[0], (n // 1024, 1024), 40.0).reshape(-1)
    g16[:4] = np.array([65504.0, -65504.0, 6e-8, 0.0], dtype=np.float16)
    g16[4::97] = (g16[4::97].astype(np.float32) * 2.0 ** -16).astype(np.float16)
    w = inputs.normal_f16_fast(seqs[1], (n // 1024, 1024), 0.02).reshape(-1).astype(np.float32)
    v = (inputs.normal_f16_fast(seqs[2], (n // 1024, 1024), 0.5).reshape(-1).astype(np.float32)) * np.float32(1.0009765625)
    gd, wd, vd = dev(g16.view(np.uint16)), dev(w), dev(v)
    hd = torch.zeros(n, dtype=torch.int16, device="cuda")
    flags = torch.zeros(2, dtype=torch.int32, device="cuda")
    inv = np.float32(1.0) / np.float32(S)
    for it in range(2):                                       # two consecutive steps on the same state
        b.mpt_update_flat(gd, wd, vd, hd, n, float(inv), lr, mu, True, True, flags)
        torch.cuda.synchronize()
        assert flags.tolist() == [0, 0]
        h_ref = np.zeros(n, dtype=np.uint16)
        assert mpo.grad_nonfinite(g16, inv) == 0
        mpo.update_apply(g16, w, v, h_ref, inv, np.float32(lr), np.float32(mu), True)
        assert np.array_equal(wd.cpu().numpy().view(np.uint32), w.view(np.uint32))
        assert np.array_equal(vd.cpu().numpy().view(np.uint32), v.view(np.uint32))
        assert np.array_equal(host_u16(hd), h_ref)


def test_large_mlp_all_steps_teacher_forced():
    """All five iterations of the large-MLP configuration (8 x 12288^2 + 12288 -> 32000, batch
    4096, S = 8192, momentum 0.9) exactly as the benchmark launches them.  Every iteration: each
    product on sampled outputs from the operands the device read, the softmax in full, the master
    pass bit for bit over all 1.6 G parameters from the state the previous iteration left (so the
    momentum buffer is non-zero from the second iteration on).  Iterations 3 to 5 sample fewer
    product outputs to bound the run time."""
    from paper_1710_03740_b200 import binding as b
    if _host_ram_gb() < 48:
        pytest.skip("not enough host memory for the full-size check")
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * 2 ** 30:
        pytest.skip("not enough device memory")
    cfg = inputs.MLP_CONFIGS["large"]
    L = len(cfg["layers"])
    steps = cfg["steps"]
    assert steps == 5
    net = b.Context(cfg["layers"], cfg["S"], cfg["lr"], cfg["momentum"], cfg["batch"])
    seqs = np.random.SeedSequence(cfg["seed"]).spawn(L + 2 * cfg["steps"])
    w16_host, w32_host, v_host = [], [], []
    for l, (fin, fout, _) in enumerate(cfg["layers"]):
        w = inputs.normal_f16_fast(seqs[l], (fout, fin), fin ** -0.5, threads=16)
        w32 = w.astype(np.float32)                           # masters are FP16-representable at t = 0
        net.set_master(l, w32)
        w16_host.append(w.view(np.uint16))
        w32_host.append(w32)
        v_host.append(np.zeros_like(w32))
    X, Y = inputs.mlp_batches(cfg, steps)
    B = cfg["batch"]
    inv = np.float32(1.0) / np.float32(cfg["S"])
    losses = []
    for t in range(steps):
        n_random = 768 if t < 2 else 96
        x16 = X[t].view(np.uint16)
        x_dev, y_dev = dev(x16), dev(Y[t])      # must stay alive until the backward pass has run
        net.forward(x_dev)
        loss = net.backward_scaled(y_dev)
        losses.append(loss)

        # forward products, layer by layer, from the activations the device actually consumed
        a_prev = x16
        acts = []
        for l, (fin, fout, relu) in enumerate(cfg["layers"]):
            assert np.array_equal(net.get_tensor(b.T_W16, l), w16_host[l]), (t, l)
            a = net.get_tensor(b.T_ACT16, l)
            _check_sampled(0, a_prev, w16_host[l], a, fin, relu=bool(relu), seed=100 * t + 10 + l,
                           full_rows=1, n_random=n_random)
            acts.append(a)
            a_prev = a
        # softmax cross-entropy in full
        dz_ref, _, loss_ref, bad = mpo.softmax_ce(acts[-1], Y[t], cfg["S"])
        dzL = net.get_tensor(b.T_DACT16, L - 1)
        ok, stats = gemm_accept(dzL, dz_ref)
        assert bad == 0 and ok.all(), (t, stats)
        assert abs(loss - loss_ref) <= (32000 * 2.0 ** -24 + 1e-5) * abs(loss_ref)
        del dz_ref
        # backward products
        dz = dzL
        grads = [None] * L
        for l in range(L - 1, -1, -1):
            fin, fout, _ = cfg["layers"][l]
            a_in = acts[l - 1] if l else x16
            g = net.get_tensor(b.T_GRAD16, l)
            _check_sampled(2, dz, a_in, g, B, seed=100 * t + 30 + l, full_rows=1, n_random=n_random)
            grads[l] = g
            if l > 0:
                dprev = net.get_tensor(b.T_DACT16, l - 1)
                mask = acts[l - 1] if cfg["layers"][l - 1][2] else None
                _check_sampled(1, dz, w16_host[l], dprev, fout, mask=mask, seed=100 * t + 50 + l,
                               full_rows=1, n_random=n_random)
                dz = dprev
        del acts, dz, dzL
        # master pass: bit-exact, layer by layer, from the state the previous iteration left
        flag_ref = 0
        for g in grads:
            flag_ref |= mpo.grad_nonfinite(g, inv)
        flag = net.step()
        assert flag == flag_ref == 0
        for l in range(L):
            w, v = w32_host[l], v_host[l]
            if t > 0:
                assert v.any()                                # the momentum buffer carries state by now
            h = np.zeros(w.shape, dtype=np.uint16)
            mpo.update_apply(grads[l], w, v, h, inv, np.float32(cfg["lr"]), np.float32(cfg["momentum"]), True)
            assert np.array_equal(net.get_master(l).view(np.uint32), w.view(np.uint32)), (t, l)
            assert np.array_equal(net.get_tensor(b.T_MOMENTUM32, l).view(np.uint32), v.view(np.uint32)), (t, l)
            assert np.array_equal(net.get_tensor(b.T_W16, l), h), (t, l)
            w16_host[l] = h
            grads[l] = None
    assert all(np.isfinite(losses))
    net.close()
