"""The multi-rank bookkeeping of the benchmark (replicas only: no data crosses ranks) with two
gloo ranks on the CPU, plus the pure host logic of sharding and aggregation."""
import os
import socket
import subprocess
import sys

import pytest

from paper_2603_14549_b200 import replicas as R

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import sys
sys.path.insert(0, {root!r})
from paper_2603_14549_b200 import replicas as R
rank, size, local = R.init("gloo")
assert size == 2 and rank in (0, 1)
R.barrier()
slow = R.max_over_ranks(10.0 + 5.0 * rank)            # rank 1 is the slow one
tokens = R.sum_over_ranks(9216 * (rank + 1))
mine = R.shard_sequences(7, size, rank)
count = R.sum_over_ranks(len(mine))
seeds = R.sum_over_ranks(R.replica_seed(100, rank))
R.barrier()
print("RESULT", rank, slow, tokens, mine, count, seeds, flush=True)
R.shutdown()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_gloo_ranks_agree_on_time_and_totals(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e[-2000:]
        outs.append([l for l in o.splitlines() if l.startswith("RESULT")][0])
    for rank, line in enumerate(outs):
        assert line.startswith(f"RESULT {rank} 15.0 27648.0 ")
        assert line.endswith(f" 7.0 {float(100 + 100 + 100003)}")
    assert "[0, 1, 2, 3]" in outs[0] and "[4, 5, 6]" in outs[1]


def test_single_process_needs_no_group():
    assert R.world() == (0, 1, 0) or "RANK" in os.environ
    assert R.max_over_ranks(3.5) == 3.5 and R.sum_over_ranks(2.0) == 2.0
    R.barrier()


@pytest.mark.parametrize("n,w", [(16, 1), (16, 2), (7, 4), (3, 8), (64, 8)])
def test_shards_partition_the_batch(n, w):
    parts = [R.shard_sequences(n, w, r) for r in range(w)]
    flat = [b for p in parts for b in p]
    assert flat == list(range(n))
    sizes = [len(p) for p in parts]
    assert max(sizes) - min(sizes) <= 1


def test_aggregate_throughput_uses_the_slowest_rank():
    assert R.aggregate_throughput([100, 100], [1.0, 2.0]) == 100.0
    assert R.aggregate_throughput([9216] * 8, [0.001] * 8) == pytest.approx(8 * 9216 / 0.001)


def test_bench_spawns_its_own_ranks_without_a_launcher():
    """`bench.py --gpus 2` started with no launcher environment starts the two ranks itself; here they
    run the host-only rendezvous check over gloo (join, barrier, the two reductions of the benchmark)."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "rendezvous-check"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout                       # rank 0 alone prints
    got = json.loads(lines[0])
    assert got == {"impl": "rendezvous-check", "n_gpus": 2, "slowest": 2.0, "total": 200.0}
