"""Host-side logic of the N > 1 benchmark path on CPU: two gloo ranks, max-over-ranks timing,
whole-job value, and the reference arm's "rank 0 only" rule.  (The path itself has no exchange
step: ranks are independent replicas.)"""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    rank = int(os.environ["RANK"])
    dist.init_process_group("gloo")
    got = bench.max_over_ranks([10.0 + rank, 20.0 - rank])
    val = bench.job_tflops(1e12, dist.get_world_size(), got[0])
    print(json.dumps({"rank": rank, "got": got, "val": val}), flush=True)
    dist.barrier()
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_maximum_time():
    import json
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=180)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    for o in outs:
        assert o["got"] == [11.0, 20.0]
        # 2 ranks x 1e12 flop in 11 ms
        assert abs(o["val"] - 2e12 / 11e-3 / 1e12) < 1e-9


def test_single_process_is_identity_and_reference_arm_runs_on_rank0_only(capsys):
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.5]) == [3.0, 4.5]

    class A:
        pass
    a = A()
    a.steps, a.warmup, a.gpus, a.workload = 1, 0, 2, "tiny"
    assert bench.run_reference(a, None, rank=1) is None
    assert capsys.readouterr().out == ""


def test_step_flops_counts_every_gemm_of_an_iteration():
    sys.path.insert(0, ROOT)
    import bench
    from paper_1710_03740_b200 import inputs
    cfg = inputs.MLP_CONFIGS["tiny"]
    # 256->512: forward + wgrad; 512->10: forward + wgrad + dgrad; batch 64
    assert bench.step_flops(cfg) == 2 * 64 * (256 * 512 * 2 + 512 * 10 * 3)
    big = inputs.MLP_CONFIGS["large"]
    assert abs(bench.step_flops(big) - 3.8113539784704e13) < 1e6
    assert bench.n_params(big) == 8 * 12288 * 12288 + 12288 * 32000


def test_bench_gpus_2_starts_its_own_two_ranks():
    """`python bench.py --gpus 2` run plainly starts two ranks by itself (torch.distributed.run on
    127.0.0.1) and reports n_gpus = 2; here with the CPU-only rank check (gloo) in place of the
    GPU step."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check"], env=env,
                       stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, p.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["gpus_arg"] == 2
    assert out["ms_per_step"] == 11.0                       # maximum over the ranks' 10 and 11 ms
    assert abs(out["value"] - 2e12 / 11e-3 / 1e12) < 1e-9   # both ranks' work over that time


def test_bench_refuses_a_world_size_that_contradicts_gpus():
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check"], env=env,
                       stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=120)
    assert p.returncode != 0 and "WORLD_SIZE" in p.stderr
