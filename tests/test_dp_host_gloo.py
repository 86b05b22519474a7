"""Host-side logic of the data-parallel step on CPU: the shard partition, and two gloo ranks
exchanging their buffer handles in rank order (no device work; the kernel is covered on the GPU)."""
import json
import os
import socket
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 100, 4096, 4099, 151_000_000, (1 << 33) + 5])
@pytest.mark.parametrize("R", [1, 2, 3, 4, 7, 8, 16])
def test_shards_partition_the_array_on_vector_boundaries(n, R):
    from paper_1710_03740_b200 import binding as b
    shards = [b.mpt_dp_shard(n, R, q) for q in range(R)]
    pos = 0
    for lo, hi in shards:
        assert lo == pos and lo <= hi <= n            # contiguous, in replica order, no overlap
        assert lo % 8 == 0 or lo == n                 # every shard starts on a 16-byte boundary
        pos = hi
    assert pos == n                                   # nothing left out
    sizes = [hi - lo for lo, hi in shards]
    assert all(s <= sizes[0] for s in sizes)
    assert sizes[0] <= (n + R - 1) // R + 8           # balanced to within one vector


def test_shard_rejects_bad_arguments():
    from paper_1710_03740_b200 import binding as b
    for R, q in ((0, 0), (17, 0), (2, 2), (2, -1)):
        with pytest.raises(b.MptError):
            b.mpt_dp_shard(100, R, q)


CHILD = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    from paper_1710_03740_b200 import binding as b
    rank = int(os.environ["RANK"])
    dist.init_process_group("gloo")
    mine = {"g16": bytes([rank]) * b.DP_HANDLE_BYTES, "w16": bytes([16 + rank]) * b.DP_HANDLE_BYTES}
    table = b.dp_exchange_handles(mine)
    ok = all(table[q]["g16"] == bytes([q]) * b.DP_HANDLE_BYTES and table[q]["w16"] == bytes([16 + q]) * b.DP_HANDLE_BYTES
             for q in range(dist.get_world_size()))
    print(json.dumps({"rank": rank, "n": len(table), "ok": ok}), flush=True)
    dist.barrier()
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_exchange_handles_in_rank_order():
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
    for p in procs:
        o, e = p.communicate(timeout=180)
        assert p.returncode == 0, e
        got = json.loads(o.strip().splitlines()[-1])
        assert got["n"] == 2 and got["ok"]
