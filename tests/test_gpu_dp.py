"""Data-parallel step (section 4.5: a batch aggregated over several GPUs) against the oracle,
bit for bit.  With one GPU the replicas are emulated: every replica's buffers live on the same
device and the per-replica calls run one after another (the kernel never waits on a peer, so the
order of the calls does not matter).  A second test runs two replicas as two PROCESSES that map
each other's buffers."""
import os
import socket

import numpy as np
import pytest

from oracle import mpo
from gpu_util import dev, host_u16, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _binding():
    from paper_1710_03740_b200 import binding
    return binding


def _inputs(n, R, seed):
    rng = np.random.default_rng(seed)
    gs = []
    for q in range(R):
        mag = np.exp2(rng.uniform(-20.0, 4.0, n))
        gs.append((mag * rng.choice([-1.0, 1.0], n)).astype(np.float32).astype(np.float16))
    w = rng.standard_normal(n).astype(np.float32)
    v = (0.1 * rng.standard_normal(n)).astype(np.float32)
    return gs, w, v


def _emulate(n, R, S, lr, mu, gs, w, v, flag_words=None, order=None):
    """Run the R per-replica calls on one device.  Returns (w32, v, [w16 per replica], [flags per replica])."""
    b = _binding()
    npad = n + 8
    g_dev = [torch.zeros(npad, dtype=torch.int16, device="cuda") for _ in range(R)]
    h_dev = [torch.full((npad,), 0x1234, dtype=torch.int16, device="cuda") for _ in range(R)]
    f_dev = [torch.zeros(2, dtype=torch.int32, device="cuda") for _ in range(R)]
    for q in range(R):
        if n:
            g_dev[q][:n] = dev(gs[q].view(np.uint16))
        if flag_words is not None:
            f_dev[q][0] = int(flag_words[q])
    w_full = torch.zeros(npad, dtype=torch.float32, device="cuda")
    v_full = torch.zeros(npad, dtype=torch.float32, device="cuda")
    if n:
        w_full[:n] = dev(w)
        v_full[:n] = dev(v)
    for q in (order if order is not None else range(R)):
        lo, hi = b.mpt_dp_shard(n, R, q)
        # the shard owner's state: here a slice of one array; lo is a multiple of 8, so it stays aligned
        b.mpt_dp_step_flat(g_dev, f_dev, h_dev, w_full[lo:], v_full[lo:] if mu != 0.0 else None, n, R, q, S, lr, mu, f_dev[q])
    torch.cuda.synchronize()
    return (w_full[:n].cpu().numpy(), v_full[:n].cpu().numpy(), [host_u16(h[:n]) for h in h_dev],
            [f.cpu().numpy() for f in f_dev], [host_u16(h[n:]) for h in h_dev])


def _oracle(n, R, S, lr, mu, gs, w, v):
    w32, vv, w16 = w.copy(), v.copy(), np.zeros(n, np.uint16)
    mpo.dp_update_apply([g.view(np.uint16) for g in gs], w32, vv if mu != 0.0 else None, w16, S, lr, mu, mu != 0.0)
    return w32, vv, w16


@pytest.mark.parametrize("mu", [0.0, 0.9])
@pytest.mark.parametrize("R", [1, 2, 3, 4, 8, 16])
@pytest.mark.parametrize("n", [5, 8 * 256 * 2 + 3, (1 << 20) + 13])
def test_dp_step_bit_exact(n, R, mu):
    S, lr = 1024.0, 0.05
    gs, w, v = _inputs(n, R, seed=n + 31 * R)
    w32, vv, w16s, flags, guard = _emulate(n, R, S, lr, mu, gs, w, v)
    rw, rv, rh = _oracle(n, R, S, lr, mu, gs, w, v)
    assert np.array_equal(w32.view(np.uint32), rw.view(np.uint32))
    if mu != 0.0:
        assert np.array_equal(vv.view(np.uint32), rv.view(np.uint32))
    else:
        assert np.array_equal(vv.view(np.uint32), v.view(np.uint32))       # untouched
    for q in range(R):
        assert np.array_equal(w16s[q], rh), "replica %d's FP16 weights" % q
        assert np.all(guard[q] == 0x1234)                                   # nothing written past n
        assert flags[q][0] == 0 and flags[q][1] == 0


def test_dp_order_of_calls_does_not_matter():
    n, R, S, lr, mu = 4099, 4, 256.0, 0.01, 0.5
    gs, w, v = _inputs(n, R, seed=9)
    a = _emulate(n, R, S, lr, mu, gs, w, v)
    b = _emulate(n, R, S, lr, mu, gs, w, v, order=[3, 1, 0, 2])
    assert np.array_equal(a[0].view(np.uint32), b[0].view(np.uint32))
    assert all(np.array_equal(x, y) for x, y in zip(a[2], b[2]))


@pytest.mark.parametrize("bad_replica", [0, 2])
def test_dp_skip_when_any_replica_overflowed(bad_replica):
    # section 3.2: an overflow anywhere skips the update everywhere; nothing but the flags changes
    n, R, S, lr, mu = 3000, 3, 1024.0, 0.05, 0.9
    gs, w, v = _inputs(n, R, seed=4)
    gs[bad_replica][17] = np.float16(np.inf)
    words = [0] * R
    words[bad_replica] = 1          # what that replica's weight-gradient epilogue reported
    w32, vv, w16s, flags, _ = _emulate(n, R, S, lr, mu, gs, w, v, flag_words=words)
    assert np.array_equal(w32.view(np.uint32), w.view(np.uint32))
    assert np.array_equal(vv.view(np.uint32), v.view(np.uint32))
    for q in range(R):
        assert np.all(w16s[q] == 0x1234)
        assert flags[q][0] != 0


def test_dp_kernel_reports_a_nonfinite_mean_it_meets():
    # a non-finite gradient that no replica flagged: the owner of that element sees it in flags[1]
    n, R = 2048, 2
    gs, w, v = _inputs(n, R, seed=6)
    gs[1][1500] = np.float16(np.nan)
    b = _binding()
    owner = [q for q in range(R) if b.mpt_dp_shard(n, R, q)[0] <= 1500 < b.mpt_dp_shard(n, R, q)[1]][0]
    _, _, _, flags, _ = _emulate(n, R, 8.0, 0.1, 0.0, gs, w, v)
    for q in range(R):
        assert flags[q][0] == 0
        assert (flags[q][1] != 0) == (q == owner)


def test_dp_empty_problem_and_bad_arguments():
    b = _binding()
    gs, w, v = _inputs(0, 2, seed=1)
    _emulate(0, 2, 4.0, 0.1, 0.9, gs, w, v)           # n = 0: launches only publish the (clear) decision
    t = torch.zeros(64, dtype=torch.int16, device="cuda")
    f = torch.zeros(2, dtype=torch.int32, device="cuda")
    w32 = torch.zeros(64, dtype=torch.float32, device="cuda")
    with pytest.raises(b.MptError):
        b.mpt_dp_step_flat([t, t], [f, f], [t, t], w32, None, 64, 2, 2, 1.0, 0.1, 0.0, f)      # rank out of range
    with pytest.raises(b.MptError):
        b.mpt_dp_step_flat([t[1:], t], [f, f], [t, t], w32, None, 32, 2, 0, 1.0, 0.1, 0.0, f)  # misaligned gradient
    with pytest.raises(b.MptError):
        b.mpt_dp_step_flat([t, t], [f, f], [t, t], w32, None, 64, 2, 0, 0.0, 0.1, 0.0, f)      # S must be positive
    with pytest.raises(b.MptError):
        b.mpt_dp_step_flat([t, t], [f, f], [t, t], w32, None, 64, 2, 0, 1.0, 0.1, 0.9, f)      # momentum without state


@pytest.mark.parametrize("wd", [0.0, 0.01])
@pytest.mark.parametrize("kind", [0, 1, 2, 3])
@pytest.mark.parametrize("R,n", [(2, 8 * 256 + 5), (3, 4099), (8, (1 << 18) + 3)])
def test_dp_step_other_optimizers_bit_exact(R, n, kind, wd):
    """Weight decay, Nesterov, Adagrad, Adam on the mean gradient (section 4.5 trains its
    multi-GPU language model with Adagrad), emulated replicas, against the oracle."""
    if kind == 0 and wd == 0.0:
        pytest.skip("plain SGD(+momentum) is covered above")
    b = _binding()
    S, lr, mu, b2, eps = 512.0, 0.01, 0.9, 0.999, 1e-8
    gs, w, _ = _inputs(n, R, seed=n + kind)
    rng = np.random.default_rng(kind + 7)
    s1 = np.abs(0.1 * rng.standard_normal(n)).astype(np.float32)
    s2 = np.abs(0.01 * rng.standard_normal(n)).astype(np.float32)
    b1t, b2t = np.float32(0.81), np.float32(0.998)
    opt = b.Optimizer(kind, lr, mu, b2, eps, wd, 0.0)
    npad = n + 8
    g_dev = [torch.zeros(npad, dtype=torch.int16, device="cuda") for _ in range(R)]
    h_dev = [torch.full((npad,), 0x1234, dtype=torch.int16, device="cuda") for _ in range(R)]
    f_dev = [torch.zeros(2, dtype=torch.int32, device="cuda") for _ in range(R)]
    for q in range(R):
        g_dev[q][:n] = dev(gs[q].view(np.uint16))
    full = [torch.zeros(npad, dtype=torch.float32, device="cuda") for _ in range(3)]
    for t, a in zip(full, (w, s1, s2)):
        t[:n] = dev(a)
    for q in range(R):
        lo, hi = b.mpt_dp_shard(n, R, q)
        b.mpt_dp_step_flat_opt(opt, g_dev, f_dev, h_dev, full[0][lo:], full[1][lo:], full[2][lo:] if kind == 3 else None,
                               n, R, q, S, float(b1t), float(b2t), f_dev[q])
    torch.cuda.synchronize()
    rw, r1, r2, rh = w.copy(), s1.copy(), s2.copy(), np.zeros(n, np.uint16)
    use_s1 = kind != 0 or mu != 0.0
    mpo.dp_update_apply_opt(kind, [g.view(np.uint16) for g in gs], rw, r1 if use_s1 else None, r2 if kind == 3 else None, rh,
                            S, lr, mu, b2, eps, wd, np.float32(1.0) - b1t, np.float32(1.0) - b2t)
    assert np.array_equal(full[0][:n].cpu().numpy().view(np.uint32), rw.view(np.uint32))
    assert np.array_equal(full[1][:n].cpu().numpy().view(np.uint32), r1.view(np.uint32))
    assert np.array_equal(full[2][:n].cpu().numpy().view(np.uint32), (r2 if kind == 3 else s2).view(np.uint32))
    for q in range(R):
        assert np.array_equal(host_u16(h_dev[q][:n]), rh)
        assert np.all(host_u16(h_dev[q][n:]) == 0x1234)
        assert f_dev[q].cpu().numpy().tolist() == [0, 0]


@pytest.mark.parametrize("kind,R,n", [(0, 2, 4099), (2, 4, (1 << 18) + 5), (3, 3, 70001), (1, 8, 12345)])
def test_dp_clipped_step_bit_exact(kind, R, n):
    """Global-norm clipping of the mean gradient: every emulated replica publishes its shard's sum
    of squares, then each forms the coefficient from all of them.  Norm within 1e-12 of the
    oracle's sequential double sum, coefficient the same FP32 bits on every replica and equal to
    the oracle's, update bit for bit."""
    b = _binding()
    S, lr, mu, b2, eps, wd, clip = 256.0, 0.01, 0.9, 0.999, 1e-8, 1e-3, 0.01
    opt = b.Optimizer(kind, lr, mu, b2, eps, wd, clip)
    gs, w, _ = _inputs(n, R, seed=n + R)
    rng = np.random.default_rng(kind)
    s1 = np.abs(0.1 * rng.standard_normal(n)).astype(np.float32)
    s2 = np.abs(0.01 * rng.standard_normal(n)).astype(np.float32)
    b1t, b2t = np.float32(0.81), np.float32(0.998)
    npad = n + 8
    g_dev = [torch.zeros(npad, dtype=torch.int16, device="cuda") for _ in range(R)]
    h_dev = [torch.full((npad,), 0x1234, dtype=torch.int16, device="cuda") for _ in range(R)]
    f_dev = [torch.zeros(2, dtype=torch.int32, device="cuda") for _ in range(R)]
    slots = [torch.full((1,), -1.0, dtype=torch.float64, device="cuda") for _ in range(R)]
    outs = [torch.zeros(2, dtype=torch.float32, device="cuda") for _ in range(R)]
    scratch = torch.zeros(b.DP_NORM_SCRATCH_BYTES // 8, dtype=torch.float64, device="cuda")
    for q in range(R):
        g_dev[q][:n] = dev(gs[q].view(np.uint16))
    full = [torch.zeros(npad, dtype=torch.float32, device="cuda") for _ in range(3)]
    for t, a_ in zip(full, (w, s1, s2)):
        t[:n] = dev(a_)
    for q in range(R):                                   # phase 1 on every replica
        b.mpt_dp_norm_flat(g_dev, n, R, q, S, scratch, slots[q])
    torch.cuda.synchronize()                             # "order the replicas"
    for q in range(R):                                   # phase 2
        lo, hi = b.mpt_dp_shard(n, R, q)
        b.mpt_dp_step_flat_opt(opt, g_dev, f_dev, h_dev, full[0][lo:], full[1][lo:], full[2][lo:] if kind == 3 else None,
                               n, R, q, S, float(b1t), float(b2t), f_dev[q], norm_peers=slots, clip_out=outs[q])
    torch.cuda.synchronize()
    glist = [g.view(np.uint16) for g in gs]
    total_ref = mpo.dp_grad_sqnorm(glist, S)
    total_dev = float(sum(float(x.item()) for x in slots))
    assert abs(total_dev - total_ref) <= 1e-12 * total_ref
    coef_ref = mpo.clip_coef(total_ref, clip)
    assert 0.0 < float(coef_ref) < 1.0                   # the bound bites in this test
    for q in range(R):
        c, nrm = outs[q].cpu().numpy()
        assert np.float32(c).view(np.uint32) == np.float32(coef_ref).view(np.uint32)
        assert abs(float(nrm) - np.sqrt(total_ref)) <= 1e-6 * np.sqrt(total_ref)
    rw, r1, r2, rh = w.copy(), s1.copy(), s2.copy(), np.zeros(n, np.uint16)
    use_s1 = kind != 0 or mu != 0.0
    mpo.dp_update_apply_clip(kind, glist, rw, r1 if use_s1 else None, r2 if kind == 3 else None, rh, S, coef_ref, lr, mu, b2, eps,
                             wd, np.float32(1.0) - b1t, np.float32(1.0) - b2t)
    assert np.array_equal(full[0][:n].cpu().numpy().view(np.uint32), rw.view(np.uint32))
    assert np.array_equal(full[1][:n].cpu().numpy().view(np.uint32), r1.view(np.uint32))
    assert np.array_equal(full[2][:n].cpu().numpy().view(np.uint32), (r2 if kind == 3 else s2).view(np.uint32))
    for q in range(R):
        assert np.array_equal(host_u16(h_dev[q][:n]), rh)
        assert np.all(host_u16(h_dev[q][n:]) == 0x1234)


def test_dp_step_opt_clipping_needs_the_norm_slots():
    b = _binding()
    t = torch.zeros(64, dtype=torch.int16, device="cuda")
    f = torch.zeros(2, dtype=torch.int32, device="cuda")
    w32 = torch.zeros(64, dtype=torch.float32, device="cuda")
    with pytest.raises(b.MptError):                      # clip_norm > 0 without norm_peers / clip_out
        b.mpt_dp_step_flat_opt(b.Optimizer(2, 0.1, 0.0, 0.0, 1e-8, 0.0, 1.0), [t, t], [f, f], [t, t], w32, w32, None, 64, 2, 0,
                               1.0, 1.0, 1.0, f)


# ---------------------------------------------------------------- two processes, mapped buffers


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _replica_main(rank, R, port, n, S, lr, mu, steps, out_dir):
    import datetime
    import torch as th
    import torch.distributed as dist
    from paper_1710_03740_b200 import binding as b
    th.cuda.set_device(0)
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=R,
                            timeout=datetime.timedelta(seconds=90))
    try:
        dp = b.DataParallelFlat(n, S, lr, mu)
        gs0, w, v = _inputs(n, R, seed=77)
        lo, hi = dp.lo, dp.hi
        if hi > lo:
            dp.w32[:hi - lo] = th.from_numpy(w[lo:hi]).cuda()
            dp.v[:hi - lo] = th.from_numpy(v[lo:hi]).cuda()
        skipped = []
        for t in range(steps):
            gs, _, _ = _inputs(n, R, seed=100 + t)
            dp.g16[:] = th.from_numpy(gs[rank].view(np.int16)).cuda()
            if t == 1 and rank == 1:
                dp.flags[0] = 1                     # this replica's backward overflowed in step 1
            skipped.append(dp.step())
        th.cuda.synchronize()
        np.savez(os.path.join(out_dir, "r%d.npz" % rank), w32=dp.w32[:max(hi - lo, 0)].cpu().numpy(),
                 v=dp.v[:max(hi - lo, 0)].cpu().numpy(), w16=dp.w16.cpu().numpy().view(np.uint16),
                 skipped=np.array(skipped), lo=lo, hi=hi)
        dp.close()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_dp_two_processes_mapped_buffers(tmp_path):
    """Two replicas as two processes on this GPU: each maps the other's gradient, weight and flag
    buffers through exported handles and runs its shard's kernel between host barriers.  Three
    steps, the second one skipped because one replica reported an overflow."""
    import torch.multiprocessing as mp
    R, n, S, lr, mu, steps = 2, 100003, 512.0, 0.05, 0.9, 3
    port = _free_port()
    mp.spawn(_replica_main, args=(R, port, n, S, lr, mu, steps, str(tmp_path)), nprocs=R, join=True)
    _, w, v = _inputs(n, R, seed=77)
    w16 = np.zeros(n, np.uint16)
    for t in range(steps):
        gs, _, _ = _inputs(n, R, seed=100 + t)
        if t == 1:
            continue
        mpo.dp_update_apply([g.view(np.uint16) for g in gs], w, v, w16, S, lr, mu, True)
    for q in range(R):
        z = np.load(os.path.join(str(tmp_path), "r%d.npz" % q))
        lo, hi = int(z["lo"]), int(z["hi"])
        assert list(z["skipped"]) == [False, True, False]
        assert np.array_equal(z["w32"].view(np.uint32), w[lo:hi].view(np.uint32))
        assert np.array_equal(z["v"].view(np.uint32), v[lo:hi].view(np.uint32))
        assert np.array_equal(z["w16"], w16), "replica %d holds all shards' FP16 weights" % q


# ---------------------------------------------------------------- MLP contexts as replicas

_MLP_LAYERS = [(64, 96, 1), (96, 10, 0)]
_MLP = dict(S=256.0, lr=0.05, mu=0.9, batch=32, inj_steps=3, e2e_steps=3)


def _mlp_masters():
    rng = np.random.default_rng(5)
    return [(rng.standard_normal((o, i)) * i ** -0.5).astype(np.float16).astype(np.float32) for (i, o, _) in _MLP_LAYERS]


def _mlp_injected_grad(t, q, l):
    i, o, _ = _MLP_LAYERS[l]
    rng = np.random.default_rng([t, q, l, 41])
    g = (rng.standard_normal((o, i)) * 8.0).astype(np.float16)
    if t == 1 and q == 1 and l == 0:
        g[3, 7] = np.float16(np.inf)            # replica 1 overflows in step 1: everybody skips
    return g


def _mlp_batch(t, q):
    rng = np.random.default_rng([t, q, 43])
    x = rng.standard_normal((_MLP["batch"], _MLP_LAYERS[0][0])).astype(np.float16)
    y = rng.integers(0, _MLP_LAYERS[-1][1], _MLP["batch"]).astype(np.int32)
    return x, y


def _mlp_replica_main(rank, R, port, out_dir, dynamic=False, opt_kind=0, clip=0.0, shard_state=False, overlap=False):
    import datetime
    import torch as th
    import torch.distributed as dist
    from paper_1710_03740_b200 import binding as b
    th.cuda.set_device(0)
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=R,
                            timeout=datetime.timedelta(seconds=90))
    try:
        opt = b.Optimizer(opt_kind, _MLP["lr"], _MLP["mu"], 0.999, 1e-8, 0.001, clip) if (opt_kind or clip) else None
        dp = b.DataParallelMLP(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], max_batch=_MLP["batch"], optimizer=opt,
                               shard_state=shard_state, overlap=overlap)
        L = len(_MLP_LAYERS)
        for l, w in enumerate(_mlp_masters()):
            dp.ctx.set_master(l, w)
        if dynamic:
            dp.ctx.set_dynamic_scale(True, growth_interval=2, min_scale=1.0, max_scale=65536.0)
        rec = {}
        for t in range(_MLP["inj_steps"]):
            for l in range(L):
                dp.ctx.set_grad(l, _mlp_injected_grad(t, rank, l).view(np.uint16))
            rec["inj_skip_%d" % t] = np.array(dp.step())
            rec["inj_scale_%d" % t] = np.array(dp.ctx.get_scale())
            for l in range(L):
                rec["inj_w16_%d_%d" % (t, l)] = dp.ctx.get_tensor(b.T_W16, l)
                rec["inj_w32_%d_%d" % (t, l)] = dp.ctx.get_master(l)
                rec["inj_v_%d_%d" % (t, l)] = dp.ctx.get_tensor(b.T_MOMENTUM32, l)
        for t in range(_MLP["e2e_steps"]):
            x, y = _mlp_batch(t, rank)
            dp.ctx.forward(th.from_numpy(x.view(np.int16)).cuda())
            if overlap and t % 2 == 0:
                # the pass is only enqueued: the exchange of the last layers runs while the first are still being
                # differentiated; the gradients are read back after the step (the step does not change them)
                yd = th.from_numpy(y).cuda()
                dp.ctx.backward_scaled(yd, want_loss=False)
                rec["e2e_skip_%d" % t] = np.array(dp.step())
                rec["e2e_loss_%d" % t] = np.array(np.nan)
                for l in range(L):
                    rec["e2e_g16_%d_%d" % (t, l)] = dp.ctx.get_tensor(b.T_GRAD16, l)
            else:
                rec["e2e_loss_%d" % t] = np.array(dp.ctx.backward_scaled(th.from_numpy(y).cuda()))
                for l in range(L):
                    rec["e2e_g16_%d_%d" % (t, l)] = dp.ctx.get_tensor(b.T_GRAD16, l)
                rec["e2e_skip_%d" % t] = np.array(dp.step())
            if clip > 0.0:
                rec["e2e_norm_coef_%d" % t] = np.array(dp.ctx.get_grad_norm(), dtype=np.float32)
            for l in range(L):
                rec["e2e_w16_%d_%d" % (t, l)] = dp.ctx.get_tensor(b.T_W16, l)
        rec["launches"] = np.array(dp.ctx.launch_count())
        rec["workspace_bytes"] = np.array(dp.ctx.workspace_bytes)
        rec["state_ranges"] = np.array([dp.ctx.state_range(l) for l in range(L)], dtype=np.int64)
        if opt_kind == 3:
            for l in range(L):
                rec["end_state2_%d" % l] = dp.ctx.get_tensor(b.T_STATE2_32, l)
        np.savez(os.path.join(out_dir, "m%d.npz" % rank), **rec)
        dp.close()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_dp_mlp_two_processes(tmp_path):
    """Two MLP contexts as two processes on this GPU, attached to each other's workspaces.
    Injected (seeded) gradients: FP16 weights of every replica, and the FP32 state inside each
    replica's shard, equal the oracle's data-parallel step bit for bit, including a skipped step.
    Then whole iterations: losses against the oracle's replicas, and the step against the oracle
    applied to the gradients each replica's backward produced."""
    import torch.multiprocessing as mp
    from oracle.dp import OracleDataParallelMLP
    R = 2
    mp.spawn(_mlp_replica_main, args=(R, _free_port(), str(tmp_path)), nprocs=R, join=True)
    rec = [np.load(os.path.join(str(tmp_path), "m%d.npz" % q)) for q in range(R)]
    L = len(_MLP_LAYERS)
    ora = OracleDataParallelMLP(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], R)
    for l, w in enumerate(_mlp_masters()):
        ora.set_master(l, w)
    for t in range(_MLP["inj_steps"]):
        for q in range(R):
            for l in range(L):
                ora.set_grad(q, l, _mlp_injected_grad(t, q, l).view(np.uint16))
        skipped = ora.step()
        assert skipped == (1 if t == 1 else 0)
        for l in range(L):
            want16, want32, wantv = ora.replicas[0].w16[l], ora.replicas[0].w32[l], ora.replicas[0].v[l]
            owned = np.zeros(want32.shape, bool)
            for q in range(R):
                assert bool(rec[q]["inj_skip_%d" % t]) == bool(skipped)
                assert np.array_equal(rec[q]["inj_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
                m = rec[q]["inj_w32_%d_%d" % (t, l)].reshape(want32.shape).view(np.uint32) == want32.view(np.uint32)
                m &= rec[q]["inj_v_%d_%d" % (t, l)].reshape(wantv.shape).view(np.uint32) == wantv.view(np.uint32)
                owned |= m
            assert owned.all(), "every element's FP32 state is current on the replica that owns it"
    for t in range(_MLP["e2e_steps"]):
        xs, ys = zip(*[_mlp_batch(t, q) for q in range(R)])
        losses = ora.forward_backward(list(xs), list(ys))
        for q in range(R):
            got = float(rec[q]["e2e_loss_%d" % t])
            assert abs(got - losses[q]) <= 1e-3 * abs(losses[q]), (t, q, got, losses[q])
            for l in range(L):
                ora.set_grad(q, l, rec[q]["e2e_g16_%d_%d" % (t, l)])       # the step is checked on the gradients it read
        skipped = ora.step()
        for q in range(R):
            assert bool(rec[q]["e2e_skip_%d" % t]) == bool(skipped)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["e2e_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
    assert all(int(r["launches"]) > 0 for r in rec)


@pytest.mark.timeout(300)
@pytest.mark.parametrize("kind", [0, 3])
def test_dp_mlp_two_processes_shard_only_state(tmp_path, kind):
    """The same two processes with contexts that keep FP32 master and optimizer state for their own
    shard only (mpt_create_dp; sections 3.1 and 4.5: 4 bytes per parameter and state, needed on one
    replica each).  FP16 weights of both replicas stay bit-exact with the oracle's replicas through the
    injected steps (one of them skipped) and whole iterations; each replica returns FP32 state for exactly
    its shard (NaN fill elsewhere), bit-exact there, and the shards cover every element; the workspace
    is smaller than an ordinary context's by the FP32 state of the other shard."""
    import torch.multiprocessing as mp
    from oracle.dp import OracleDataParallelMLP
    from paper_1710_03740_b200 import binding as b
    R = 2
    mp.spawn(_mlp_replica_main, args=(R, _free_port(), str(tmp_path), False, kind, 0.0, True), nprocs=R, join=True)
    rec = [np.load(os.path.join(str(tmp_path), "m%d.npz" % q)) for q in range(R)]
    L = len(_MLP_LAYERS)
    ora = OracleDataParallelMLP(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], R)
    if kind:
        ora.set_optimizer(kind, _MLP["lr"], _MLP["mu"], 0.999, 1e-8, 0.001)
    for l, w in enumerate(_mlp_masters()):
        ora.set_master(l, w)
    for t in range(_MLP["inj_steps"]):
        for q in range(R):
            for l in range(L):
                ora.set_grad(q, l, _mlp_injected_grad(t, q, l).view(np.uint16))
        skipped = ora.step()
        assert skipped == (1 if t == 1 else 0)
        for l in range(L):
            want16, want32 = ora.replicas[0].w16[l], ora.replicas[0].w32[l]
            wantv = ora.replicas[0].v[l]
            covered = np.zeros(want32.size, np.int32)
            for q in range(R):
                assert bool(rec[q]["inj_skip_%d" % t]) == bool(skipped)
                assert np.array_equal(rec[q]["inj_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
                first, count = (int(x) for x in rec[q]["state_ranges"][l])
                for name, want in (("inj_w32_%d_%d", want32), ("inj_v_%d_%d", wantv)):
                    got = rec[q][name % (t, l)].reshape(-1)
                    inside = np.zeros(got.size, bool)
                    inside[first:first + count] = True
                    assert np.isnan(got[~inside]).all(), "nothing is reported outside the shard"
                    assert np.array_equal(got[inside].view(np.uint32), want.reshape(-1)[inside].view(np.uint32)), (t, l, q, name)
                covered[first:first + count] += 1
            assert (covered == 1).all(), "every element's FP32 state lives on exactly one replica"
    for t in range(_MLP["e2e_steps"]):
        xs, ys = zip(*[_mlp_batch(t, q) for q in range(R)])
        losses = ora.forward_backward(list(xs), list(ys))
        for q in range(R):
            got = float(rec[q]["e2e_loss_%d" % t])
            assert abs(got - losses[q]) <= 1e-3 * abs(losses[q]), (t, q, got, losses[q])
            for l in range(L):
                ora.set_grad(q, l, rec[q]["e2e_g16_%d_%d" % (t, l)])
        skipped = ora.step()
        for q in range(R):
            assert bool(rec[q]["e2e_skip_%d" % t]) == bool(skipped)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["e2e_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
    if kind == 3:
        for l in range(L):
            want = ora.replicas[0].s2[l].reshape(-1)
            for q in range(R):
                first, count = (int(x) for x in rec[q]["state_ranges"][l])
                got = rec[q]["end_state2_%d" % l].reshape(-1)
                assert np.array_equal(got[first:first + count].view(np.uint32), want[first:first + count].view(np.uint32))
    # the workspace: same size on both replicas, smaller than an ordinary context's by the other shard's FP32 state
    opt = b.Optimizer(kind, _MLP["lr"], _MLP["mu"], 0.999, 1e-8, 0.001, 0.0) if kind else None
    full = b.Context(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], max_batch=_MLP["batch"], optimizer=opt)
    n = full.dp_layout().n
    n_states = 1 + (2 if kind == 3 else 1)
    assert int(rec[0]["workspace_bytes"]) == int(rec[1]["workspace_bytes"])
    saved = full.workspace_bytes - int(rec[0]["workspace_bytes"])
    assert abs(saved - n_states * 4 * (n - n // R)) <= n_states * (256 + 32 * R), (saved, n, n_states)
    full.close()


@pytest.mark.timeout(300)
@pytest.mark.parametrize("kind,shard_state,clip", [(0, False, 0.0), (2, True, 0.0), (2, False, 0.02)])
def test_dp_mlp_two_processes_overlapped_exchange(tmp_path, kind, shard_state, clip):
    """The exchange overlapped with the backward pass: per-layer interprocess events, the sums of each
    layer's gradients formed on a second stream as soon as that layer is complete on both replicas, the
    step from the sums once both passes are complete.  Same bits as the one-kernel exchange: FP16 weights
    of both replicas against the oracle's replicas through injected steps (one skipped) and whole
    iterations, half of them with the backward pass only enqueued when the exchange is issued.  With
    global-norm clipping the parts of the norm come from the sums and the coefficient has the oracle's bits."""
    import torch.multiprocessing as mp
    from oracle.dp import OracleDataParallelMLP
    R = 2
    mp.spawn(_mlp_replica_main, args=(R, _free_port(), str(tmp_path), False, kind, clip, shard_state, True), nprocs=R, join=True)
    rec = [np.load(os.path.join(str(tmp_path), "m%d.npz" % q)) for q in range(R)]
    L = len(_MLP_LAYERS)
    ora = OracleDataParallelMLP(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], R)
    if kind:
        ora.set_optimizer(kind, _MLP["lr"], _MLP["mu"], 0.999, 1e-8, 0.001, clip)
    for l, w in enumerate(_mlp_masters()):
        ora.set_master(l, w)
    for t in range(_MLP["inj_steps"]):
        for q in range(R):
            for l in range(L):
                ora.set_grad(q, l, _mlp_injected_grad(t, q, l).view(np.uint16))
        skipped = ora.step()
        assert skipped == (1 if t == 1 else 0)
        for l in range(L):
            want16, want32 = ora.replicas[0].w16[l], ora.replicas[0].w32[l]
            for q in range(R):
                assert bool(rec[q]["inj_skip_%d" % t]) == bool(skipped)
                assert np.array_equal(rec[q]["inj_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
                first, count = (int(x) for x in rec[q]["state_ranges"][l])
                if shard_state:
                    got = rec[q]["inj_w32_%d_%d" % (t, l)].reshape(-1)[first:first + count]
                    assert np.array_equal(got.view(np.uint32), want32.reshape(-1)[first:first + count].view(np.uint32))
    for t in range(_MLP["e2e_steps"]):
        xs, ys = zip(*[_mlp_batch(t, q) for q in range(R)])
        losses = ora.forward_backward(list(xs), list(ys))
        for q in range(R):
            got = float(rec[q]["e2e_loss_%d" % t])
            assert np.isnan(got) == (t % 2 == 0)
            if not np.isnan(got):
                assert abs(got - losses[q]) <= 1e-3 * abs(losses[q]), (t, q, got, losses[q])
            for l in range(L):
                ora.set_grad(q, l, rec[q]["e2e_g16_%d_%d" % (t, l)])
        skipped = ora.step()
        for q in range(R):
            assert bool(rec[q]["e2e_skip_%d" % t]) == bool(skipped)
            if clip > 0.0:
                coef = np.float32(ora.replicas[0].last_coef)
                assert np.float32(rec[q]["e2e_norm_coef_%d" % t][1]).view(np.uint32) == coef.view(np.uint32), (t, q)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["e2e_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)


def test_overlapped_exchange_error_paths():
    """The overlapped exchange needs an attached context, its events before the attach, and a call of
    mpt_dp_reduce_async; a context that is none of that says so and stays usable."""
    require_gpu()
    from paper_1710_03740_b200 import binding as b
    ctx = b.Context(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], max_batch=_MLP["batch"])
    with pytest.raises(b.MptError) as e:
        ctx.dp_reduce_async()
    assert e.value.code == -3
    handles = ctx.dp_overlap_events()
    assert len(handles) == (len(_MLP_LAYERS) + 1) * b.DP_HANDLE_BYTES and handles == ctx.dp_overlap_events()
    with pytest.raises(b.MptError) as e:
        ctx.dp_overlap_attach([handles, handles], 0)        # not attached to any replica
    assert e.value.code == -3
    for l, w in enumerate(_mlp_masters()):
        ctx.set_master(l, w)
    for l in range(len(_MLP_LAYERS)):
        ctx.set_grad(l, _mlp_injected_grad(0, 0, l).view(np.uint16))
    assert ctx.step() == 0                                   # the ordinary single-GPU step still works
    ctx.close()


def test_shard_only_context_refuses_what_it_cannot_do():
    """A context made by mpt_create_dp has no FP32 state outside its shard: it steps only while attached
    as that replica, and cannot be attached as another."""
    require_gpu()
    from paper_1710_03740_b200 import binding as b
    ctx = b.Context(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], max_batch=_MLP["batch"], shard=(2, 1))
    L = len(_MLP_LAYERS)
    for l, w in enumerate(_mlp_masters()):
        ctx.set_master(l, w)
        got = ctx.get_master(l).reshape(-1)
        first, count = ctx.state_range(l)
        assert np.array_equal(got[first:first + count], w.reshape(-1)[first:first + count])
        assert np.isnan(got[:first]).all() and np.isnan(got[first + count:]).all()
        with np.errstate(over="ignore"):
            assert np.array_equal(ctx.get_tensor(b.T_W16, l).reshape(-1), w.astype(np.float16).view(np.uint16).reshape(-1))
    total = sum(ctx.state_range(l)[1] for l in range(L))
    lo, hi = b.mpt_dp_shard(ctx.dp_layout().n, 2, 1)
    assert 0 < total <= hi - lo
    for l in range(L):
        ctx.set_grad(l, _mlp_injected_grad(0, 0, l).view(np.uint16))
    with pytest.raises(b.MptError) as e:
        ctx.step()
    assert e.value.code == -3          # MPT_ERR_STATE
    lay = ctx.dp_layout()
    base = ctx._ws_ptr
    tabs = [[base + off] * 2 for off in (lay.g16_offset, lay.flags_offset, lay.w16_offset)]
    with pytest.raises(b.MptError) as e:
        ctx.dp_attach(2, 0, *tabs)
    assert e.value.code == -1          # MPT_ERR_INVALID_ARG
    ctx.close()
    with pytest.raises(b.MptError):
        b.Context(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], max_batch=_MLP["batch"], shard=(1, 0))


@pytest.mark.timeout(300)
def test_dp_mlp_two_processes_dynamic_scale(tmp_path):
    """The same two attached contexts with dynamic loss scaling: the kernel reads S from device
    memory, every replica sees the OR-ed overflow word, so both halve S after the skipped step and
    double it after two clean ones - the oracle's replicas do the same, bit for bit."""
    import torch.multiprocessing as mp
    from oracle.dp import OracleDataParallelMLP
    R = 2
    mp.spawn(_mlp_replica_main, args=(R, _free_port(), str(tmp_path), True), nprocs=R, join=True)
    rec = [np.load(os.path.join(str(tmp_path), "m%d.npz" % q)) for q in range(R)]
    L = len(_MLP_LAYERS)
    ora = OracleDataParallelMLP(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], R)
    for l, w in enumerate(_mlp_masters()):
        ora.set_master(l, w)
    for r in ora.replicas:
        r.set_dynamic_scale(2, 1.0, 65536.0)
    scales = []
    for t in range(_MLP["inj_steps"]):
        for q in range(R):
            for l in range(L):
                ora.set_grad(q, l, _mlp_injected_grad(t, q, l).view(np.uint16))
        skipped = ora.step()
        scales.append(float(ora.replicas[0].S))
        for q in range(R):
            assert bool(rec[q]["inj_skip_%d" % t]) == bool(skipped)
            assert float(rec[q]["inj_scale_%d" % t]) == float(ora.replicas[q].S), (t, q)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["inj_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
    assert scales[1] == _MLP["S"] / 2          # the skipped step halved the scale everywhere
    for t in range(_MLP["e2e_steps"]):
        xs, ys = zip(*[_mlp_batch(t, q) for q in range(R)])
        losses = ora.forward_backward(list(xs), list(ys))
        for q in range(R):
            got = float(rec[q]["e2e_loss_%d" % t])
            assert abs(got - losses[q]) <= 1e-3 * abs(losses[q]), (t, q, got, losses[q])
            for l in range(L):
                ora.set_grad(q, l, rec[q]["e2e_g16_%d_%d" % (t, l)])
        skipped = ora.step()
        for q in range(R):
            assert bool(rec[q]["e2e_skip_%d" % t]) == bool(skipped)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["e2e_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)


@pytest.mark.timeout(300)
@pytest.mark.parametrize("kind", [2, 3])
def test_dp_mlp_two_processes_adagrad_adam(tmp_path, kind):
    """Two attached contexts stepping with Adagrad (the optimizer of the paper's multi-GPU language
    model, section 4.5) or Adam, with weight decay: FP16 weights of both replicas bit-exact against
    the oracle's replicas through a skipped step; Adam's running beta products stay in step."""
    import torch.multiprocessing as mp
    from oracle.dp import OracleDataParallelMLP
    R = 2
    mp.spawn(_mlp_replica_main, args=(R, _free_port(), str(tmp_path), False, kind), nprocs=R, join=True)
    rec = [np.load(os.path.join(str(tmp_path), "m%d.npz" % q)) for q in range(R)]
    L = len(_MLP_LAYERS)
    ora = OracleDataParallelMLP(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], R)
    ora.set_optimizer(kind, _MLP["lr"], _MLP["mu"], b2=0.999, eps=1e-8, wd=0.001)
    for l, w in enumerate(_mlp_masters()):
        ora.set_master(l, w)
    for t in range(_MLP["inj_steps"]):
        for q in range(R):
            for l in range(L):
                ora.set_grad(q, l, _mlp_injected_grad(t, q, l).view(np.uint16))
        skipped = ora.step()
        assert skipped == (1 if t == 1 else 0)
        for q in range(R):
            assert bool(rec[q]["inj_skip_%d" % t]) == bool(skipped)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["inj_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
    for t in range(_MLP["e2e_steps"]):
        xs, ys = zip(*[_mlp_batch(t, q) for q in range(R)])
        losses = ora.forward_backward(list(xs), list(ys))
        for q in range(R):
            got = float(rec[q]["e2e_loss_%d" % t])
            assert abs(got - losses[q]) <= 1e-3 * abs(losses[q]), (t, q, got, losses[q])
            for l in range(L):
                ora.set_grad(q, l, rec[q]["e2e_g16_%d_%d" % (t, l)])
        skipped = ora.step()
        for q in range(R):
            assert bool(rec[q]["e2e_skip_%d" % t]) == bool(skipped)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["e2e_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)


@pytest.mark.timeout(300)
def test_dp_mlp_two_processes_clipped(tmp_path):
    """Two attached contexts with global-norm clipping (section 3.2) of the mean gradient: every
    replica publishes its shard's part of the norm (mpt_dp_norm), the replicas are ordered, every
    replica forms the same coefficient in mpt_step.  Coefficient bits and FP16 weights of both
    replicas against the oracle's replicas, through a skipped step; and mpt_step without the norm
    call is refused."""
    import torch.multiprocessing as mp
    from oracle.dp import OracleDataParallelMLP
    R, kind, clip = 2, 2, 0.02
    mp.spawn(_mlp_replica_main, args=(R, _free_port(), str(tmp_path), False, kind, clip), nprocs=R, join=True)
    rec = [np.load(os.path.join(str(tmp_path), "m%d.npz" % q)) for q in range(R)]
    L = len(_MLP_LAYERS)
    ora = OracleDataParallelMLP(_MLP_LAYERS, _MLP["S"], _MLP["lr"], _MLP["mu"], R)
    ora.set_optimizer(kind, _MLP["lr"], _MLP["mu"], b2=0.999, eps=1e-8, wd=0.001, clip=clip)
    for l, w in enumerate(_mlp_masters()):
        ora.set_master(l, w)
    for t in range(_MLP["inj_steps"]):
        for q in range(R):
            for l in range(L):
                ora.set_grad(q, l, _mlp_injected_grad(t, q, l).view(np.uint16))
        skipped = ora.step()
        assert skipped == (1 if t == 1 else 0)
        for q in range(R):
            assert bool(rec[q]["inj_skip_%d" % t]) == bool(skipped)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["inj_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
    bit = False
    for t in range(_MLP["e2e_steps"]):
        xs, ys = zip(*[_mlp_batch(t, q) for q in range(R)])
        ora.forward_backward(list(xs), list(ys))
        for q in range(R):
            for l in range(L):
                ora.set_grad(q, l, rec[q]["e2e_g16_%d_%d" % (t, l)])
        skipped = ora.step()
        coef = np.float32(ora.replicas[0].last_coef)
        bit |= float(coef) < 1.0
        for q in range(R):
            assert bool(rec[q]["e2e_skip_%d" % t]) == bool(skipped)
            assert np.float32(rec[q]["e2e_norm_coef_%d" % t][1]).view(np.uint32) == coef.view(np.uint32), (t, q)
            for l in range(L):
                want16 = ora.replicas[0].w16[l]
                assert np.array_equal(rec[q]["e2e_w16_%d_%d" % (t, l)].reshape(want16.shape), want16), (t, l, q)
    assert bit                                           # the bound was active in at least one iteration
