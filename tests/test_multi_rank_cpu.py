"""The N>1 path of the benchmark on CPU: two gloo ranks.  Ranks are replicas (request streams are
independent, no data-path collective); the only communication is the MAX reduction of the step time."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    step_s = [0.50, 0.80][rank]          # rank 1 is slower
    e2e_s = [0.90, 0.70][rank]
    agg = bench.aggregate_over_ranks(step_s, e2e_s, chunks_per_rank=512, world=world)
    ids = bench.rank_stream_ids(32, rank)
    dist.barrier()
    out.put((rank, agg, ids))
    dist.destroy_process_group()


def test_two_rank_aggregation_and_stream_sharding():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    res.sort()
    for rank, agg, ids in res:
        assert agg["chunks"] == 1024                          # both ranks' chunks count
        assert abs(agg["step_s"] - 0.80) < 1e-12              # the slowest rank sets the time
        assert abs(agg["value"] - 1024 / 0.80) < 1e-9
        assert abs(agg["e2e_value"] - 1024 / 0.90) < 1e-9
    assert res[0][2] == list(range(32)) and res[1][2] == list(range(32, 64))      # disjoint request streams


def test_single_rank_aggregation_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    agg = bench.aggregate_over_ranks(0.25, None, 16, 1)
    assert agg["value"] == 64.0 and agg["e2e_value"] is None
