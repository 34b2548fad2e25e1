"""The N > 1 path of the benchmark on CPU (gloo, world_size 2): ranks replay their own seeded batches (weak
scaling, no data-path collective) and the only reduction is MAX of the elapsed time / SUM of the units."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from gdn_workloads import config_concurrent_hits
    inp = config_concurrent_hits(num_seqs=3, lo=5, hi=40, seed_offset=rank)    # tiny: only lengths matter here
    units = inp.total_tokens * inp.num_v_heads
    ms, total = bench.reduce_over_ranks(10.0 + 5.0 * rank, units, "cpu")
    out[rank] = (ms, total, units, tuple(int(x) for x in inp.tail_lens()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_time_by_max_and_units_by_sum():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    (ms0, tot0, u0, l0), (ms1, tot1, u1, l1) = out[0], out[1]
    assert ms0 == ms1 == 15.0                               # max over ranks
    assert tot0 == tot1 == float(u0 + u1)                   # whole-job units
    assert l0 != l1                                         # ranks replay different batches (seed offset)


def test_single_process_is_identity():
    import bench
    assert bench.reduce_over_ranks(3.5, 100, "cpu") == (3.5, 100.0)
