"""The N > 1 path of the layer library on CPU: world_size-2 gloo ranks agree on the request partition and on the
max-over-ranks timing that bench.py reports (the data path itself has no collective: requests are independent)."""
import os
import socket

import numpy as np
import pytest

from paper_2504_12397_b200 import sharding as sh


def test_partition_requests_is_a_disjoint_cover():
    for n in (0, 1, 7, 8, 64, 65):
        for world in (1, 2, 3, 8):
            parts = sh.partition_requests(n, world)
            assert len(parts) == world and parts[0][0] == 0 and parts[-1][1] == n
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sh.partition_requests(4, 0)


def test_partition_by_tokens_balances_and_is_deterministic():
    rng = np.random.default_rng(3)
    tokens = rng.integers(16, 513, 32)
    a = sh.partition_by_tokens(tokens, 4)
    assert a == sh.partition_by_tokens(tokens, 4)
    assert sorted(i for part in a for i in part) == list(range(32))
    loads = [int(tokens[p].sum()) for p in a]
    assert max(loads) - min(loads) <= int(tokens.max())


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = sh.partition_requests(9, world)[rank]
        step_ms = 1.0 + rank            # the slower rank decides the reported time
        t = sh.max_over_ranks(step_ms)
        dist.barrier()
        q.put((rank, lo, hi, t, sh.rank_seed(2, rank), sh.aggregate_throughput(2048, t / 1e3, world)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_partition_and_timing():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, lo0, hi0, t0, s0, v0), (r1, lo1, hi1, t1, s1, v1) = got
    assert (lo0, hi0, lo1, hi1) == (0, 5, 5, 9)
    assert t0 == t1 == 2.0                      # max over ranks, identical on both
    assert s0 != s1                             # every rank draws its own batch
    assert v0 == v1 == 2 * 2048 / 2e-3


def test_bench_starts_its_own_ranks_and_agrees_on_the_timing():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself; with --dry-run on the gloo
    backend the ranks do everything but the GPU work: process group, request partition, barrier, max over ranks.
    The line rank 0 prints counts the ranks that really took part and carries the slower rank's time."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--backend", "gloo", "--dry-run"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2 and rec["dry_run"] is True and rec["backend"] == "gloo"
    assert rec["ms_per_step"] == 2.0                       # rank 1 reports 2.0 ms, rank 0 1.0 ms: the max
    assert rec["config"]["requests_per_gpu"] == 8 and len(set(rec["config"]["rank_seeds"])) == 2
