"""The multi-GPU leg of bench.py is "replicas only": every rank runs the whole workload on its own
GPU and the only exchange is the max of the step times.  That host logic is checked here with two
gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    out[rank] = (ms, bench.whole_job_value(32768, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_step_and_add_the_tokens():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, 29500 + os.getpid() % 500, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 15.0                                   # the slower rank's time
    assert abs(value - 2 * 32768 / 15e-3) < 1e-6        # whole-job tokens per second


def test_single_rank_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1, torch.device("cpu")) == 7.5
    assert bench.whole_job_value(1000, 1, 2.0) == 500000.0
