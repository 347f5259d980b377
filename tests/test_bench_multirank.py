"""The N > 1 path of bench.py is plain replication: every rank samples its own batch with the same model,
and only the timing is reduced (max over ranks).  Checked here with two gloo ranks on CPU."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        cfg, seed, steps, batch, guidance, interval, latent, labels, vc = bench.rank_inputs("ddim50", rank, world)
        ms = bench.reduce_max_ms(100.0 + 50.0 * rank, dist)          # rank 1 is the slow one
        value = bench.images_per_second(world, batch, 3, ms)
        out.put((rank, seed, float(latent.sum()), int(labels.sum()), float(vc.sum()), ms, value, batch))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_replicate_with_own_batches_and_max_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, lat0, lab0, vc0, ms0, v0, b0), (r1, seed1, lat1, lab1, vc1, ms1, v1, b1) = res
    assert seed0 == seed1 and vc0 == vc1            # same model and sampler tables on every rank
    assert lat0 != lat1                              # each rank has its own noise
    assert ms0 == ms1 == 150.0                       # the slowest rank's time, on every rank
    assert v0 == v1 == 2 * b0 * 3 / 0.150            # whole-job images/s: all ranks' images over that time


def test_single_rank_inputs_are_the_workload_itself():
    sys.path.insert(0, ROOT)
    import bench
    a = bench.rank_inputs("ddim50", 0, 1)
    b = bench.workload_inputs("ddim50")
    np.testing.assert_array_equal(a[6], b[6])
    np.testing.assert_array_equal(a[7], b[7])
    assert bench.reduce_max_ms(12.5, None) == 12.5
