"""The whole-job aggregation bench.py uses for N replicas (maximum of the ranks' times, sum of their
tokens), run as two gloo ranks on the CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, tok = bench.max_over_ranks_sum_tokens(10.0 + 5.0 * rank, 100 + rank, dist, None)
    out.put((rank, ms, tok))
    dist.destroy_process_group()


def test_two_ranks_max_time_sum_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, 2, 29533, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, 15.0, 201.0), (1, 15.0, 201.0)]


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks_sum_tokens(3.5, 7) == (3.5, 7.0)
