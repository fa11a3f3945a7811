"""N > 1 path of bench.py on CPU: two gloo ranks, max / sum over ranks, per-rank seeds.

The attention path shards over (batch, head) units with no data-path collective; the
only cross-rank traffic is the timing reduction, which is what this test covers.
"""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    from paper_2410_09397_b200 import inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mx = bench.max_over_ranks([1.0 + rank, 5.0 - rank], world)
    sm = bench.sum_over_ranks([10.0 * (rank + 1), 1.0], world)
    # every rank draws its own batch: same recipe, seed shifted by the rank
    w = inputs.WORKLOADS["C1"]
    wr = inputs.Workload(**{**w.__dict__, "seed": w.seed + 1000 * rank})
    q = wr.tensors()["Q"]
    out.put((rank, mx, sm, float(q.sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_times_and_draw_distinct_batches():
    torch = pytest.importorskip("torch")
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, sm, _ in res:
        assert mx == [2.0, 5.0]
        assert sm == [30.0, 2.0]
    assert res[0][3] != res[1][3]


def test_single_rank_reductions_are_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    assert bench.sum_over_ranks([1.5], 1) == [1.5]


def test_flop_conventions():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2410_09397_b200 import inputs
    w = inputs.WORKLOADS["C3"]
    ff, fb = bench.flops(w, None)
    assert fb == pytest.approx(1.374e12, rel=1e-3) and ff == pytest.approx(5.50e11, rel=1e-3)
    w5 = inputs.WORKLOADS["C5"]
    bm = w5.block_mask()
    kept = bench.kept_entries(w5, bm)
    assert kept == bm[0].sum() * 128 * 128
    assert abs(bm[0].sum() - 6784) < 400   # expected number of kept blocks: 256 + 0.1 * 65280
