"""Per-kernel timing through the C ABI (CUDA events, synthetic data): the isolated GEMM
sweep, the bigLSTM-shaped products, the master-update pass and the softmax cross-entropy.

    python -m paper_1710_03740_b200.kernel_bench gemm   [--shape MxNxK ...] [--op 0 1 2] [--iters 20]
    python -m paper_1710_03740_b200.kernel_bench update [--params N] [--momentum 0|1] [--iters 20]
    python -m paper_1710_03740_b200.kernel_bench softmax [--rows B] [--classes C] [--iters 20]
    python -m paper_1710_03740_b200.kernel_bench step    [--workload tiny|scale_sweep|large_twin] [--iters 50]

    python -m paper_1710_03740_b200.kernel_bench lstm    [--config biglstm] [--iters 20]
    python -m paper_1710_03740_b200.kernel_bench dp      [--params N] [--replicas R]

Prints one JSON line per case: best-of and back-to-back ("sustained") rates.  Working sets
are larger than the 126 MB L2 unless the shape itself is smaller; small cases say so.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as mpt
from . import inputs

OPS = {0: "fwd", 1: "dgrad", 2: "wgrad"}


def _time_graph(fn, iters):
    """Device time per call with the calls replayed from a CUDA graph (no host launch cost)."""
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(3):
            fn()
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(iters):
                fn()
        g.replay()
        side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        g.replay()
        e1.record(side)
        side.synchronize()
    return e0.elapsed_time(e1) / iters


def _time(fn, iters, warmup=5):
    """(best single launch, mean of `iters` back-to-back launches) in ms after `warmup` calls; the
    median of the individually timed launches is kept in _time.last_median."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    singles = []
    for _ in range(max(5, min(iters, 20))):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        singles.append(e0.elapsed_time(e1))
    singles.sort()
    _time.last_median = singles[len(singles) // 2]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return singles[0], e0.elapsed_time(e1) / iters


_time.last_median = None


def bench_gemm(M, N, K, op, iters, flags=mpt.GEMM_FORCE_TC, use_workspace=True):
    sa = (K, M) if op == 2 else (M, K)
    sb = (N, K) if op == 0 else (K, N)
    g = torch.Generator(device="cuda").manual_seed(2)
    A = (torch.randn(sa, device="cuda", generator=g) * K ** -0.5).half()
    B = (torch.randn(sb, device="cuda", generator=g) * K ** -0.5).half()
    C = torch.empty((M, N), dtype=torch.half, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    nws = mpt.mpt_gemm_workspace_bytes(op, M, N, K) if use_workspace else 0
    ws = torch.empty(max(nws, 16) // 4, dtype=torch.float32, device="cuda")      # split-K scratch, if the shape wants one
    fn = lambda: mpt.mpt_gemm_f16_ws(op, M, N, K, A, sa[1], B, sb[1], C, N, flags, None, 0, None, st,  # noqa: E731
                                     ws if nws else None)
    best, sus = _time(fn, iters)
    fl = 2.0 * M * N * K
    if sus < 0.2:       # short kernels: host launch cost hides the device time, so replay from a graph as well
        sus = min(sus, _time_graph(lambda: mpt.mpt_gemm_f16_ws(op, M, N, K, A, sa[1], B, sb[1], C, N, flags, None, 0, None,
                                                                st, ws if nws else None, torch.cuda.current_stream()),
                                   iters))
    out = {"kernel": "gemm", "op": OPS[op], "M": M, "N": N, "K": K, "best_ms": best, "median_ms": _time.last_median,
           "sustained_ms": sus,
           "best_tflops": fl / best / 1e9, "sustained_tflops": fl / sus / 1e9, "device_error": int(st[0]), "splitk_workspace_mb": nws / 1e6,
           "working_set_mb": (A.numel() + B.numel() + C.numel()) * 2 / 1e6}
    return out


def trace_gemm(M, N, K, op):
    """One launch of the CTA-pair kernel from the trace build (build.py --trace) after 30 warm-up
    launches: per cluster, the main loops' SM cycles per issued k-block (512 = the tensor pipe's
    full rate for a 256x256x64 block), the SM clock they ran at, and when the clusters finished."""
    import numpy as np
    sa = (K, M) if op == 2 else (M, K)
    sb = (N, K) if op == 0 else (K, N)
    g = torch.Generator(device="cuda").manual_seed(2)
    A = (torch.randn(sa, device="cuda", generator=g) * K ** -0.5).half()
    B = (torch.randn(sb, device="cuda", generator=g) * K ** -0.5).half()
    C = torch.empty((M, N), dtype=torch.half, device="cuda")
    st = torch.zeros(1024, dtype=torch.int32, device="cuda")
    nws = mpt.mpt_gemm_workspace_bytes(op, M, N, K)
    ws = torch.empty(max(nws, 16) // 4, dtype=torch.float32, device="cuda")
    run = lambda: mpt.mpt_gemm_f16_ws(op, M, N, K, A, sa[1], B, sb[1], C, N, mpt.GEMM_FORCE_PAIR, None, 0, None, st,  # noqa: E731
                                      ws if nws else None)
    for _ in range(30):
        run()
    torch.cuda.synchronize()
    st.zero_()
    run()
    torch.cuda.synchronize()
    t = st.cpu().numpy().view(np.uint32)[64:64 + 8 * 74].reshape(74, 8).astype(np.int64)
    t = t[t[:, 3] > 0]
    us = ((t[:, 1] - t[:, 0]) % (1 << 32)) / 1e3
    end = ((t[:, 1] - t[:, 0].min()) % (1 << 32)) / 1e3
    cyc, kb = t[:, 2], t[:, 3]
    return {"kernel": "gemm_trace", "op": OPS[op], "M": M, "N": N, "K": K, "clusters": int(len(t)),
            "units_per_cluster": [int(t[:, 4].min()), int(t[:, 4].max())],
            "cycles_per_kblock_median": float(np.median(cyc / kb)), "cycles_per_kblock_max": float((cyc / kb).max()),
            "sm_mhz_median": float(np.median(cyc / us)), "last_issue_us": [float(end.min()), float(end.max())],
            "device_error": int(st[0])}


def bench_update(n, momentum, iters):
    g = torch.Generator(device="cuda").manual_seed(3)
    g16 = (torch.randn(n, device="cuda", generator=g) * 37).half()
    w32 = torch.randn(n, device="cuda", generator=g)
    v = torch.zeros(n, device="cuda") if momentum else None
    w16 = torch.empty(n, dtype=torch.half, device="cuda")
    flags = torch.zeros(2, dtype=torch.int32, device="cuda")
    fn = lambda: mpt.mpt_update_flat(g16, w32, v, w16, n, 1.0 / 512, 1e-4, 0.9, momentum, False, flags)  # noqa: E731
    best, sus = _time(fn, iters)
    bpp = 20 if momentum else 12
    out = {"kernel": "update", "params": n, "momentum": bool(momentum), "bytes_per_param": bpp, "best_ms": best,
           "median_ms": _time.last_median, "sustained_ms": sus, "best_gbs": bpp * n / best / 1e6,
           "median_gbs": bpp * n / _time.last_median / 1e6, "sustained_gbs": bpp * n / sus / 1e6,
           "working_set_mb": bpp * n / 1e6, "flags": flags.tolist()}
    if bpp * n < 256e6:
        out["note"] = "working set below 256 MB: L2-resident, not an HBM claim"
    return out


def bench_update_opt(n, kind, wd, iters, clip=0.0):
    """Master pass with Nesterov (1), Adagrad (2) or Adam (3), optional weight decay and global-norm
    clipping (one more read of the FP16 gradients: +2 bytes per parameter)."""
    g = torch.Generator(device="cuda").manual_seed(3)
    g16 = (torch.randn(n, device="cuda", generator=g) * 37).half()
    w32 = torch.randn(n, device="cuda", generator=g)
    s1 = torch.zeros(n, device="cuda")
    s2 = torch.zeros(n, device="cuda") if kind == mpt.OPT_ADAM else None
    w16 = torch.empty(n, dtype=torch.half, device="cuda")
    flags = torch.zeros(2, dtype=torch.int32, device="cuda")
    opt = mpt.Optimizer(kind, 1e-4, 0.9, 0.999, 1e-8, wd, clip)
    scratch = torch.zeros(mpt.CLIP_SCRATCH_BYTES // 4, device="cuda") if clip > 0 else None
    fn = lambda: mpt.mpt_update_flat_opt(opt, g16, w32, s1, s2, w16, n, 1.0 / 512, 0.81, 0.998, False, flags,  # noqa: E731
                                         clip_scratch=scratch)
    best, sus = _time(fn, iters)
    bpp = (28 if kind == mpt.OPT_ADAM else 20) + (2 if clip > 0 else 0)
    return {"kernel": "update_opt", "optimizer": ["sgd", "nesterov", "adagrad", "adam"][kind], "weight_decay": wd,
            "clip_norm": clip,
            "params": n, "bytes_per_param": bpp, "best_ms": best, "sustained_ms": sus, "best_gbs": bpp * n / best / 1e6,
            "sustained_gbs": bpp * n / sus / 1e6, "flags": flags.tolist()}


def bench_dp(n, R, momentum, iters):
    """Data-parallel step of ONE replica (rank 0 of R) with every replica's buffers on this GPU: the
    kernel's own memory-system rate with local "peers".  Says nothing about NVLink."""
    g = torch.Generator(device="cuda").manual_seed(3)
    gs = [(torch.randn(n, device="cuda", generator=g) * 37).half() for _ in range(R)]
    ws = [torch.empty(n, dtype=torch.half, device="cuda") for _ in range(R)]
    fl = [torch.zeros(2, dtype=torch.int32, device="cuda") for _ in range(R)]
    lo, hi = mpt.mpt_dp_shard(n, R, 0)
    w32 = torch.randn(hi - lo, device="cuda", generator=g)
    v = torch.zeros(hi - lo, device="cuda") if momentum else None
    fn = lambda: mpt.mpt_dp_step_flat(gs, fl, ws, w32, v, n, R, 0, 512.0, 1e-4, 0.9 if momentum else 0.0, fl[0])  # noqa: E731
    best, sus = _time(fn, iters)
    per_elem = 2 * R + 8 + (8 if momentum else 0) + 2 * R       # R gradients in, state in and out, R weight copies out
    nbytes = per_elem * (hi - lo)
    return {"kernel": "dp_step", "params": n, "replicas": R, "shard": hi - lo, "momentum": bool(momentum),
            "bytes_per_shard_element": per_elem, "best_ms": best, "median_ms": _time.last_median, "sustained_ms": sus,
            "best_gbs": nbytes / best / 1e6, "median_gbs": nbytes / _time.last_median / 1e6,
            "link_bytes_each_way_if_remote": 2 * (hi - lo) * (R - 1), "peers": "local (one GPU)", "flags": fl[0].tolist()}


def bench_lstm(name, iters, steps=None):
    """LSTM layer with projection: the fused gate step against the bare gate product, the backward
    gate kernel, the bias-gradient reduction, and the whole layer forward + backward."""
    cfg = dict(inputs.LSTM_CONFIGS[name])
    if steps:
        cfg["T"] = steps
    T, B, I, H, P = cfg["T"], cfg["B"], cfg["I"], cfg["H"], cfg["P"]
    K = I + P
    layer = mpt.LstmLayer(T, B, I, H, P)
    g = torch.Generator(device="cuda").manual_seed(9)

    def fill(t, scale):
        t.copy_((torch.randn(t.shape, device="cuda", generator=g) * scale).half().view(torch.int16))

    fill(layer.Wg16, K ** -0.5); fill(layer.Wp16, H ** -0.5); fill(layer.bias16, 0.1)
    fill(layer.xr, 1.0); fill(layer.c[0], 0.5); fill(layer.dr_ext, 1024.0 / B)
    out = {"kernel": "lstm", "config": name, "T": T, "B": B, "I": I, "H": H, "P": P}
    # one step's gate product with and without the fused gate arithmetic
    fused = lambda: mpt.mpt_lstm_cell_forward(B, H, K, layer.xr[0], K, layer.Wg16, K, layer.bias16, layer.c[0], H,  # noqa: E731
                                              layer.acts[0], 4 * H, layer.c[1], H, layer.h[0], H, 0, layer.status)
    bare = lambda: mpt.mpt_gemm_f16(0, B, 4 * H, K, layer.xr[0], K, layer.Wg16, K, layer.acts[0], 4 * H, 0, None, 0,  # noqa: E731
                                    None, layer.status)
    fl = 2.0 * B * 4 * H * K
    for key, fn in (("gate_fused", fused), ("gate_bare", bare)):
        best, sus = _time(fn, iters)
        out[key + "_ms"] = sus
        out[key + "_tflops"] = fl / sus / 1e9
    # whole layer
    layer.forward()
    fwd_best, fwd = _time(layer.forward, max(3, iters // 4))
    bwd_best, bwd = _time(layer.backward, max(3, iters // 4))
    flops = 3.0 * T * (2.0 * B * 4 * H * K + 2.0 * B * P * H)
    out.update({"forward_ms": fwd, "backward_ms": bwd, "layer_tflops": flops / (fwd + bwd) / 1e9,
                "forward_tflops": flops / 3 / fwd / 1e9, "backward_tflops": flops * 2 / 3 / bwd / 1e9})
    # pieces of the backward pass
    cb = lambda: mpt.mpt_lstm_cell_backward(B, H, layer.dh, H, layer.dc[0], H, layer.acts[0], 4 * H, layer.c[0], H,  # noqa: E731
                                            layer.c[1], H, layer.dG[0], 4 * H, layer.dc[1], H)
    best, sus = _time(cb, iters)
    out["cell_bwd_ms"] = sus
    out["cell_bwd_gbs"] = 26.0 * B * H / sus / 1e6
    bg = lambda: mpt.mpt_bias_grad(layer.dG, T * B, 4 * H, 4 * H, layer.bias_parts, layer.dbias16, layer.nonfinite_flag)  # noqa: E731
    best, sus = _time(bg, iters)
    out["bias_grad_ms"] = sus
    out["bias_grad_gbs"] = 2.0 * T * B * 4 * H / sus / 1e6
    out["device_error"] = layer.device_error()
    return out


def bench_softmax(B, Cn, iters):
    g = torch.Generator(device="cuda").manual_seed(4)
    z = (torch.randn((B, Cn), device="cuda", generator=g) * 3).half()
    y = torch.randint(0, Cn, (B,), device="cuda", generator=g, dtype=torch.int32)
    dz = torch.empty_like(z)
    rl = torch.empty(B, device="cuda")
    loss = torch.empty(1, device="cuda")
    fn = lambda: mpt.mpt_softmax_ce(z, Cn, y, B, Cn, 8192.0, dz, Cn, rl, loss, None)  # noqa: E731
    best, sus = _time(fn, iters)
    by = 4.0 * B * Cn
    out = {"kernel": "softmax_ce", "rows": B, "classes": Cn, "best_ms": best, "median_ms": _time.last_median,
           "sustained_ms": sus, "best_gbs": by / best / 1e6, "sustained_gbs": by / sus / 1e6, "loss": float(loss.item())}
    if by < 256e6:
        out["note"] = "working set below 256 MB: L2-resident, not an HBM claim"
    return out


def bench_step(workload, iters):
    """Latency of one whole iteration (forward, scaled backward, master pass) of a small
    configuration: calls issued one by one, and the same calls replayed from a CUDA graph."""
    import numpy as np
    cfg = inputs.MLP_CONFIGS[workload]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        net = mpt.Context(cfg["layers"], cfg["S"], cfg["lr"], cfg["momentum"], cfg["batch"], stream=side)
        for l, w in enumerate(inputs.mlp_masters(cfg)):
            net.set_master(l, w)
        X, Y = inputs.mlp_batches(cfg, 1)
        x = torch.from_numpy(X[0].view(np.int16)).cuda()
        y = torch.from_numpy(Y[0]).cuda()

        def one():
            net.forward(x)
            net.backward_scaled(y, want_loss=False)
            net.step(want_flag=False)

        def timed(fn):
            for _ in range(5):
                fn()
            side.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(iters):
                fn()
            e1.record(side)
            side.synchronize()
            return e0.elapsed_time(e1) / iters * 1e3

        n0 = net.launch_count()
        one()
        launches = net.launch_count() - n0
        eager_us = timed(one)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            one()
        graph_us = timed(graph.replay)
    fl = sum(2.0 * cfg["batch"] * i * o * (2 if l == 0 else 3) for l, (i, o, _) in enumerate(cfg["layers"]))
    return {"kernel": "step", "workload": workload, "kernel_launches": launches, "eager_us": eager_us,
            "graph_us": graph_us, "gflop_per_step": fl / 1e9, "graph_tflops": fl / graph_us / 1e6}


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    g = sub.add_parser("gemm")
    g.add_argument("--shape", nargs="*", default=None, help="MxNxK; default: the sweep and the bigLSTM shapes")
    g.add_argument("--op", nargs="*", type=int, default=[0, 1, 2])
    g.add_argument("--iters", type=int, default=20)
    g.add_argument("--no-workspace", action="store_true", help="do not offer a split-K scratch buffer")
    g.add_argument("--trace", action="store_true",
                   help="per-cluster main-loop cycles from the instrumented build (python -m paper_1710_03740_b200.build --trace)")
    g.add_argument("--kernel", default="auto", choices=["auto", "tc", "pair", "pair512", "split2", "split4"],
                   help="auto: the library's choice; tc: single-CTA 128x256 tiles; pair: cta_group::2 256x256 tiles")
    u = sub.add_parser("update")
    u.add_argument("--params", type=int, default=150994944)
    u.add_argument("--momentum", type=int, default=1)
    u.add_argument("--optimizer", default="sgd", choices=["sgd", "nesterov", "adagrad", "adam"])
    u.add_argument("--weight-decay", type=float, default=0.0)
    u.add_argument("--clip-norm", type=float, default=0.0)
    u.add_argument("--iters", type=int, default=20)
    s = sub.add_parser("softmax")
    s.add_argument("--rows", type=int, default=4096)
    s.add_argument("--classes", type=int, default=32000)
    s.add_argument("--iters", type=int, default=20)
    ls = sub.add_parser("lstm")
    ls.add_argument("--config", default="biglstm", choices=sorted(inputs.LSTM_CONFIGS))
    ls.add_argument("--steps", type=int, default=0, help="override the number of time steps")
    ls.add_argument("--iters", type=int, default=20)
    d = sub.add_parser("dp")
    d.add_argument("--params", type=int, default=150994944)
    d.add_argument("--replicas", type=int, default=8)
    d.add_argument("--momentum", type=int, default=1)
    d.add_argument("--iters", type=int, default=20)
    t = sub.add_parser("step")
    t.add_argument("--workload", default="tiny", choices=["tiny", "scale_sweep", "scale_sweep_twin", "large_twin"])
    t.add_argument("--iters", type=int, default=50)
    args = ap.parse_args()
    if args.cmd == "step":
        print(json.dumps(bench_step(args.workload, args.iters)), flush=True)
    elif args.cmd == "gemm" and args.trace:
        import os
        mpt.LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmpt_trace.so")
        for t in args.shape or ["4096x12288x12288"]:
            M, N, K = (int(x) for x in t.split("x"))
            for op in args.op:
                print(json.dumps(trace_gemm(M, N, K, op)), flush=True)
    elif args.cmd == "gemm":
        shapes = ([tuple(int(x) for x in t.split("x")) for t in args.shape] if args.shape
                  else inputs.GEMM_SWEEP + [inputs.LSTM_GATE, inputs.LSTM_PROJ])
        for (M, N, K) in shapes:
            for op in args.op:
                flags = {"auto": 0, "tc": mpt.GEMM_FORCE_TC, "pair": mpt.GEMM_FORCE_PAIR, "pair512": mpt.GEMM_FORCE_PAIR512,
                         "split2": mpt.GEMM_FORCE_SPLIT2, "split4": mpt.GEMM_FORCE_SPLIT4}[args.kernel]
                res = bench_gemm(M, N, K, op, args.iters, flags, not args.no_workspace)
                res["kernel_choice"] = args.kernel
                print(json.dumps(res), flush=True)
    elif args.cmd == "dp":
        print(json.dumps(bench_dp(args.params, args.replicas, args.momentum, args.iters)), flush=True)
    elif args.cmd == "lstm":
        print(json.dumps(bench_lstm(args.config, args.iters, args.steps)), flush=True)
    elif args.cmd == "update":
        kind = ["sgd", "nesterov", "adagrad", "adam"].index(args.optimizer)
        if kind == 0 and args.weight_decay == 0.0 and args.clip_norm == 0.0:
            print(json.dumps(bench_update(args.params, args.momentum, args.iters)), flush=True)
        else:
            print(json.dumps(bench_update_opt(args.params, kind, args.weight_decay, args.iters, args.clip_norm)), flush=True)
    else:
        print(json.dumps(bench_softmax(args.rows, args.classes, args.iters)), flush=True)


if __name__ == "__main__":
    main()
