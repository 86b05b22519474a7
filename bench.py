#!/usr/bin/env python
"""Benchmark of the mixed-precision training step (forward GEMMs, scaled softmax-CE,
backward GEMMs, FP32 master update) on synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mine|reference] [--workload NAME]

One "step" is one pass of the whole hot path over one batch: mpt_forward,
mpt_backward_scaled, mpt_step.  The default workload "large" is the large-MLP
configuration (8 x 12288^2 ReLU layers + 12288 -> 32000 head, batch 4096, S = 8192,
SGD momentum 0.9); "large_twin" and "tiny" are small cases.  Prints ONE JSON line on
rank 0.  With N > 1 every rank runs an independent replica of the step on its own GPU (the
path has no exchange step); the time is the maximum over ranks and the value the sum of all
ranks' work over that time.  `--gpus N` run plainly (no WORLD_SIZE in the environment) starts
its own N ranks under torch.distributed.run on 127.0.0.1; launched by torch.distributed.run it
takes rank and world size from the environment, and the two must agree.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1710_03740_b200 import inputs  # noqa: E402

METRIC = "train_step_tflops"
UNIT = "TFLOP/s"
NOMINAL_FP16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def spawn_ranks(n, argv):
    """Re-runs this script as n ranks of one node under torch.distributed.run (rendezvous on
    127.0.0.1, a free port) and returns its exit code.  Rank 0's JSON line goes to stdout."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def rank_check(args, rank, world):
    """The rank plumbing of the N > 1 path without a GPU: gloo ranks, a made-up per-rank time,
    maximum over ranks, whole-job value, one line from rank 0.  Used by the CPU tests."""
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("gloo")
    ms = max_over_ranks([10.0 + rank])[0]
    if rank == 0:
        print(json.dumps({"rank_check": True, "n_gpus": world, "gpus_arg": args.gpus, "ms_per_step": ms,
                          "value": job_tflops(1e12, world, ms), "scaling": "weak"}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def bench_config(args, cfg):
    """The `config` object of the JSON line; both arms print the same one."""
    return {"workload": args.workload, "layers": len(cfg["layers"]), "batch": cfg["batch"], "params": n_params(cfg),
            "S": cfg["S"], "momentum": cfg["momentum"], "parallelism": "replicas only",
            "l2": "inputs larger than L2 (weights %.1f GB per pass)" % (n_params(cfg) * 2 / 1e9),
            "flop_per_step": step_flops(cfg)}


def dp_step_over_peers(n, iters, dev):
    """The data-parallel step (one kernel per replica: gradient reduce-scatter over peer loads,
    master pass on the owned shard, FP16 weight all-gather over peer stores) across the N GPUs of
    this job: every rank owns exchange buffers the others map.  Times the kernel with CUDA events
    between process-group barriers; returns the slowest rank's median and the bytes each GPU pulls
    and pushes over NVLink per step.  An extra: not part of the step metric."""
    import datetime
    import torch
    import torch.distributed as dist
    from paper_1710_03740_b200 import binding as mpt
    # Every collective of this extra runs on its own gloo group with a short time limit: a rank that
    # fails (no peer access, a launch error) must end this measurement on all ranks within a minute,
    # never hang the benchmark whose line is still to be printed.
    grp = dist.new_group(backend="gloo", timeout=datetime.timedelta(seconds=60))
    dp = None
    try:
        err = None
        try:
            dp = mpt.DataParallelFlat(n, 512.0, 1e-4, 0.9, group=grp)
        except Exception as ex:       # e.g. no peer access between two of the GPUs
            err = repr(ex)
        ok = torch.tensor([0 if dp is None else 1], dtype=torch.int32)
        dist.all_reduce(ok, op=dist.ReduceOp.MIN, group=grp)
        if int(ok.item()) == 0:
            return {"error": err or "set-up failed on another rank"}
        g = torch.Generator(device=dev).manual_seed(3 + dp.rank)
        dp.g16.copy_((torch.randn(n, device=dev, generator=g) * 37).half().view(torch.int16))
        times = []
        for it in range(iters + 2):
            dp._barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            mpt.mpt_dp_step_flat([p["g16"] for p in dp._peers], [p["flags"] for p in dp._peers], [p["w16"] for p in dp._peers],
                                 dp.w32, dp.v, dp.n, dp.R, dp.rank, dp.S, dp.lr, dp.mu, dp._own["flags"])
            e1.record()
            dp._barrier()
            if it >= 2:
                times.append(e0.elapsed_time(e1))
        times.sort()
        t = torch.tensor([times[len(times) // 2]], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=grp)
        med = float(t.item())
        shard = dp.hi - dp.lo
        link = 2 * shard * (dp.R - 1)
        res = {"replicas": dp.R, "params": n, "shard": shard, "ms": med, "peers": "remote (one GPU per replica)",
               "link_bytes_each_way": link, "link_gbs_each_way": link / med / 1e6, "hbm_bytes": (2 + 16 + 2) * shard}
        dp.close()
        return res
    except BaseException as ex:       # an extra: whatever goes wrong here is reported, not raised
        return {"error": repr(ex)}


def step_flops(cfg):
    """GEMM flop of one iteration: forward + wgrad for every layer, dgrad for all but the first."""
    B = cfg["batch"]
    tot = 0
    for l, (fin, fout, _) in enumerate(cfg["layers"]):
        tot += 2 * B * fin * fout * (2 if l == 0 else 3)
    return float(tot)


def n_params(cfg):
    return sum(fin * fout for fin, fout, _ in cfg["layers"])


# dram__bytes_read.sum + dram__bytes_write.sum of the representative GEMM launch of each workload
# (ncu capture summarised in profiles/k_gemm_tc2_pair_4096x12288x12288.md), bytes per launch.
NCU_GEMM_TRAFFIC = {"large": {"launch": "forward 4096x12288x12288", "bytes": 1.285e9, "algorithmic_bytes": 0.503e9}}


def max_over_ranks(vals, device=None):
    """Element-wise maximum of per-rank timings over all ranks (identity for one process)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in vals]
    t = torch.tensor([float(v) for v in vals], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_tflops(flop_per_step_per_rank, world, ms_per_step):
    """Whole-job rate: every rank does the same work per step (weak scaling), time = max over ranks."""
    return flop_per_step_per_rank * world / (ms_per_step * 1e-3) / 1e12


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while a region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        # keep samples taken under load (clock above idle)
        busy = [c for c in sm if c > 500] or sm
        return {"sm_mhz": float(np.median(busy)) if busy else None,
                "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_operands(cfg, seconds_target):
    from oracle import mpo
    B = cfg["batch"]
    fin, fout, _ = max(cfg["layers"], key=lambda l: l[0] * l[1])
    cores = mpo.num_threads()
    # ~1.3 GFLOP/s per core is typical for the plain loops; aim for `seconds_target`
    rows = int(seconds_target * 1.3e9 * cores / (2.0 * fin * fout))
    rows = max(cores, min(B, rows))
    return inputs.gemm_operands(0, rows, fout, fin, seed=2, fast=True)


def oracle_sample(cfg, seconds_target=12.0, operands=None):
    """Times the CPU oracle, as it stands, on a slab of output rows of the dominant GEMM of
    this workload (a hidden-layer forward product) and returns TFLOP/s."""
    from oracle import mpo
    B = cfg["batch"]
    A, W = operands if operands is not None else oracle_operands(cfg, seconds_target)
    rows, fin = A.shape
    fout = W.shape[0]
    cores = mpo.num_threads()
    t0 = time.perf_counter()
    mpo.gemm_f16(mpo.OP_FWD, A, W, relu=True)
    dt = time.perf_counter() - t0
    flops = 2.0 * rows * fin * fout
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "forward GEMM slab: %d of %d rows x N=%d x K=%d in %.1f s" % (rows, B, fout, fin, dt)}


def oracle_streaming_samples():
    """The oracle's master update (P = 150,994,944 parameters with momentum, 20 B each: the update
    of the LSTM-shaped config) and softmax cross-entropy (4096 x 32000 logits, 4 B each), timed as
    they stand on the host cores; GB/s on the same algorithmic bytes as the GPU figures."""
    from oracle import mpo
    n = 150994944
    rng = np.random.default_rng(7)
    g16 = inputs.normal_f16_fast(np.random.SeedSequence(7), (n // 4096, 4096), 37.0).reshape(-1)
    w32 = np.ones(n, dtype=np.float32)
    v = np.zeros(n, dtype=np.float32)
    w16 = np.zeros(n, dtype=np.uint16)
    t0 = time.perf_counter()
    mpo.update_apply(g16, w32, v, w16, np.float32(1.0 / 512), np.float32(0.01), np.float32(0.9), True)
    t_upd = time.perf_counter() - t0
    B, Cn = 4096, 32000
    z = inputs.normal_f16_fast(np.random.SeedSequence(8), (B, Cn), 3.0)
    y = rng.integers(0, Cn, B).astype(np.int32)
    t0 = time.perf_counter()
    mpo.softmax_ce(z, y, 8192.0)
    t_sm = time.perf_counter() - t0
    return {"update_gbs": 20.0 * n / t_upd / 1e9, "update_sample": "P=%d with momentum in %.2f s" % (n, t_upd),
            "softmax_gbs": 4.0 * B * Cn / t_sm / 1e9, "softmax_sample": "%dx%d in %.2f s" % (B, Cn, t_sm)}


def run_reference(args, cfg, rank):
    """Reference arm: the CPU oracle on the host cores, bounded sample per step."""
    if rank != 0:
        return
    vals = []
    ops = oracle_operands(cfg, 4.0)
    for i in range(args.warmup + args.steps):
        r = oracle_sample(cfg, operands=ops)
        if i >= args.warmup:
            vals.append(r)
    v = float(np.mean([r["value"] for r in vals]))
    sample = vals[-1]["sample"]
    # time one full step would take at this rate
    ms = step_flops(cfg) / (v * 1e12) * 1e3
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f16", "data": "synthetic",
           "config": bench_config(args, cfg),
           "note": "CPU oracle, bounded sample per step, extrapolated to a whole step",
           "cpu_baseline": {"value": v, "unit": UNIT, "cores": vals[-1]["cores"], "kind": "oracle", "sample": sample},
           "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="mine", choices=["mine", "reference"])
    ap.add_argument("--workload", default="large", choices=sorted(inputs.MLP_CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the LSTM-layer timing appended to the JSON line")
    ap.add_argument("--rank-check", action="store_true", help="run only the rank plumbing on CPU (gloo); for tests")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.impl == "reference"):
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    args.warmup = max(args.warmup, 3) if args.impl == "mine" else args.warmup
    cfg = inputs.MLP_CONFIGS[args.workload]

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "mine" and world != args.gpus:
        raise SystemExit("--gpus %d but WORLD_SIZE=%d: launch with --nproc-per-node equal to --gpus" % (args.gpus, world))

    if args.rank_check:
        rank_check(args, rank, world)
        return
    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_1710_03740_b200 import binding as mpt   # raises if the CUDA library is missing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    nccl_log = None
    if world > 1:
        # keep NCCL's communicator log (transport, NVLS or not) but out of stdout, where the one JSON line goes
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_FILE", os.path.join(tempfile.gettempdir(), "mpt_bench_nccl_%h_%p.log"))
        nccl_log = os.environ["NCCL_DEBUG_FILE"]
        dist.init_process_group("nccl", device_id=dev)

    # ---- synthetic inputs (seeded; rank r uses seed + 100 r so replicas differ)
    cfg = dict(cfg)
    cfg["seed"] = cfg["seed"] + 100 * rank
    big = n_params(cfg) > (1 << 26)
    L = len(cfg["layers"])
    net = mpt.Context(cfg["layers"], cfg["S"], cfg["lr"], cfg["momentum"], cfg["batch"], device=dev)
    seqs = np.random.SeedSequence(cfg["seed"]).spawn(L + 2 * cfg["steps"])
    for l, (fin, fout, _) in enumerate(cfg["layers"]):
        scale = fin ** -0.5 * (cfg["head_scale"] if l == L - 1 else 1.0)
        if big:
            w16 = inputs.normal_f16_fast(seqs[l], (fout, fin), scale, threads=min(32, os.cpu_count() or 8))
        else:
            w16 = inputs.normal_f16(np.random.default_rng(seqs[l]), (fout, fin), scale)
        net.set_master(l, w16.astype(np.float32))
        del w16
    X, Y = inputs.mlp_batches(cfg)
    nb = X.shape[0]
    Xd = [torch.from_numpy(X[t].view(np.int16)).to(dev) for t in range(nb)]
    Yd = [torch.from_numpy(Y[t]).to(dev) for t in range(nb)]
    Xp = [torch.from_numpy(X[t].view(np.int16)).pin_memory() for t in range(nb)]
    Yp = [torch.from_numpy(Y[t]).pin_memory() for t in range(nb)]

    def step_dev(t):
        net.forward(Xd[t % nb])
        net.backward_scaled(Yd[t % nb], want_loss=False)
        net.step(want_flag=False)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput
    for t in range(args.warmup):
        step_dev(t)
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.15)
    n0 = net.launch_count()
    net.profile(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for t in range(args.steps):
        step_dev(args.warmup + t)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    prof = net.profile_read()
    net.profile(False)
    launches = net.launch_count() - n0
    clocks = sampler.stop() if sampler else None
    # loss and flag of one more step, to show the job is live (outside the timed region)
    net.forward(Xd[0])
    loss = net.backward_scaled(Yd[0], want_loss=True)
    flag = net.step(want_flag=True)

    # ---- end to end through the host-buffer entry points: every step copies one batch from pinned
    # host memory (staged on a second stream, overlapping the previous step's compute) and reads
    # loss and overflow flag back (synchronising)
    copy_stream = torch.cuda.Stream(device=dev)
    for t in range(2):
        net.train_step_host(Xp[t % nb], Yp[t % nb])
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    net.stage_batch_host(Xp[0], Yp[0], copy_stream)
    for t in range(args.steps):
        if t + 1 < args.steps:
            net.stage_batch_host(Xp[(t + 1) % nb], Yp[(t + 1) % nb], copy_stream)
        net.train_step_staged()
    e1.record()
    barrier()
    # every call synchronises, so host wall-clock and device events bracket the same work
    ms_e2e = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dev)

    dp_peers = None
    if world > 1 and not args.no_extras:
        # every rank takes part; rank 0 reports.  Not part of the step metric.
        dp_peers = dp_step_over_peers(150994944, 10, dev)

    if rank == 0:
        peaks, peak_src = measured_peaks()
        fl = step_flops(cfg)
        ms_step = ms_total / args.steps
        value = job_tflops(fl, world, ms_step)
        e2e_val = job_tflops(fl, world, ms_e2e / args.steps)
        g_ms, g_work, g_n = prof["gemm"]
        u_ms, u_work, u_n = prof["update"]
        s_ms, s_work, s_n = prof["softmax"]
        gemm_tflops = g_work / (g_ms * 1e-3) / 1e12 if g_ms > 0 else None
        upd_gbs = u_work / (u_ms * 1e-3) / 1e9 if u_ms > 0 else None
        sm_gbs = s_work / (s_ms * 1e-3) / 1e9 if s_ms > 0 else None
        peak_t = peaks["bf16_tflops_sustained"]
        tr = NCU_GEMM_TRAFFIC.get(args.workload)
        traffic = tr["bytes"] if tr else None
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": bench_config(args, cfg),
            "frac_of_nominal_fp16_peak": value / world / NOMINAL_FP16_TFLOPS,
            "roofline": {"bound": "tensor", "kernel": "pair::k_gemm_tc2 (all GEMM launches of the step)",
                         "achieved": gemm_tflops, "peak": peak_t, "peak_source": peak_src + " (sustained bf16 GEMM; fp16 has the same nominal rate)",
                         "unit": "TFLOP/s", "frac": (gemm_tflops / peak_t) if gemm_tflops else None,
                         "frac_of_nominal": (gemm_tflops / NOMINAL_FP16_TFLOPS) if gemm_tflops else None,
                         "frac_of_clock_ceiling": (gemm_tflops * 1e12 / (148 * 8192 * clocks["sm_mhz"] * 1e6))
                         if gemm_tflops and clocks and clocks.get("sm_mhz") else None,
                         "clock_ceiling_note": "148 SMs x 8192 dense FP16 flop per clock x median sampled SM clock",
                         "launches": g_n, "avg_launch_ms": g_ms / g_n if g_n else None, "traffic": traffic,
                         "traffic_note": ("ncu dram bytes of one %s launch; algorithmic minimum %.3e"
                                          % (tr["launch"], tr["algorithmic_bytes"])) if tr else None},
            "update": {"bound": "hbm", "kernel": "k_update_quad", "achieved": upd_gbs, "peak": peaks["hbm_gbs"],
                       "peak_source": peak_src, "unit": "GB/s", "frac": (upd_gbs / peaks["hbm_gbs"]) if upd_gbs else None,
                       "frac_of_nominal": (upd_gbs / NOMINAL_HBM_GBS) if upd_gbs else None,
                       "bytes_per_param": 20 if cfg["momentum"] else 12, "avg_launch_ms": u_ms / u_n if u_n else None},
            "softmax": {"bound": "hbm", "achieved": sm_gbs, "unit": "GB/s", "avg_launch_ms": s_ms / s_n if s_n else None},
            "phase_ms_per_step": {"gemm": g_ms / args.steps, "update": u_ms / args.steps, "softmax": s_ms / args.steps},
            "e2e": {"value": e2e_val, "unit": UNIT, "ms_per_step": ms_e2e / args.steps,
                    "h2d_bytes_per_step": int(X[0].nbytes + Y[0].nbytes), "d2h_bytes_per_step": 64,
                    "api": "mpt_stage_batch_host + mpt_train_step_staged (copy of batch t+1 overlaps step t)"},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "last_loss": loss, "last_overflow": flag,
        }
        if world == 1 and not args.no_extras:
            # not part of the step metric: the LSTM layer of the paper's language model (section 4.5),
            # forward + backward through time, timed with CUDA events after the step benchmark
            try:
                from paper_1710_03740_b200.kernel_bench import bench_lstm
                r = bench_lstm("biglstm", 8)
                out["lstm_layer"] = {"config": {k: r[k] for k in ("T", "B", "I", "H", "P")}, "forward_ms": r["forward_ms"],
                                     "backward_ms": r["backward_ms"], "tflops": r["layer_tflops"],
                                     "gate_step_fused_ms": r["gate_fused_ms"], "gate_product_alone_ms": r["gate_bare_ms"],
                                     "cell_backward_gbs": r["cell_bwd_gbs"], "bias_grad_gbs": r["bias_grad_gbs"],
                                     "device_error": r["device_error"]}
            except Exception as ex:  # an extra; never fatal for the bench line
                out["lstm_layer"] = {"error": repr(ex)}
            # not part of the step metric either: the data-parallel step of one replica of 8 for a
            # 151 M parameter model, with all eight replicas' buffers on this GPU (the kernel's own
            # rate; nothing here crosses NVLink)
            try:
                from paper_1710_03740_b200.kernel_bench import bench_dp
                r = bench_dp(150994944, 8, 1, 10)
                out["dp_step"] = {"replicas": r["replicas"], "params": r["params"], "shard": r["shard"], "ms": r["median_ms"],
                                  "gbs": r["median_gbs"], "bytes_per_shard_element": r["bytes_per_shard_element"],
                                  "peers": r["peers"], "link_bytes_each_way_if_remote": r["link_bytes_each_way_if_remote"]}
            except Exception as ex:
                out["dp_step"] = {"error": repr(ex)}
        if dp_peers is not None:
            out["dp_step"] = dp_peers
        if nccl_log:
            out["nccl_log"] = nccl_log
        if not args.no_cpu_baseline:
            try:
                out["cpu_baseline"] = oracle_sample(cfg)
                out["cpu_baseline"].update(oracle_streaming_samples())
            except Exception as ex:  # the oracle is a reported baseline; never fatal for the bench line
                out["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                       "sample": "failed: %r" % (ex,)}
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
