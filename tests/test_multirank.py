"""The N > 1 path of bench.py on CPU: two gloo ranks.  The hot path does not shard (replicas only), so
what several ranks share is the timing rule (maximum over ranks, whole-job value) and the rule that
every rank works on sequences of its own."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2601_12212_b200 import synth
    own = [100.0 + 10.0 * rank, 5.0 - rank, 7.0]
    got = bench.max_over_ranks(own, world, "cpu")
    # every rank draws sequences of its own (rank * batch ...) from the same seeded workload
    w = synth.WORKLOADS[1]
    root = int(synth.root_token(w, 0, rank * w.batch))
    dist.barrier()
    out.put((rank, got, root))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_rank_and_the_whole_job_value():
    import bench
    world, port = 2, 29000 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, _ in res:
        assert got == [110.0, 5.0, 7.0]  # the maximum of each time over both ranks, on every rank
    roots = [r[2] for r in res]
    if roots[0] is not None:
        assert roots[0] != roots[1]  # different sequences on different ranks
    assert bench.whole_job_value(110.0, 2) == 55.0
    assert bench.whole_job_value(110.0, 1) == 110.0
    assert bench.max_over_ranks([3.0, 4.0], 1, "cpu") == [3.0, 4.0]


def _gather_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2601_12212_b200 import binding
    cols = binding.shard_columns(128256, world)
    # what a rank would hand to the merge calls after scanning its columns: small per-row arrays
    val = torch.full((2, 5, 3), float(rank))
    ids = torch.full((2, 5, 3), rank, dtype=torch.int32)
    all_val, all_id = binding.all_gather_parts([val, ids])
    out.put((rank, cols, tuple(all_val.shape), all_val[:, 0, 0, 0].tolist(), all_id[:, 1, 2, 1].tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_gather_their_vocabulary_shards():
    """The exchange step of the vocabulary-sharded path: every rank ends up with every rank's partial rows,
    stacked in rank order, and the ranks agree on the column ranges."""
    world, port = 2, 31000 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_gather_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, cols, shape, vals, ids in res:
        assert cols == [(0, 64128), (64128, 64128)]
        assert shape == (2, 2, 5, 3) and vals == [0.0, 1.0] and ids == [0, 1]
