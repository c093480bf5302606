"""The multi-GPU form of the benchmark is N independent replicas (the path has no exchange step): what ranks share
is only the timing rule — the step time of the job is the slowest rank's, the value is all ranks' work over it.
Run here as two gloo ranks on the CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), ".."))


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 0.100 + 0.025 * rank                    # rank 1 is the slower replica
    ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.whole_job_value(404_750_336, world, ms))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_work():
    import bench
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank, args=(world, 29611, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]                            # every rank sees the same job-wide numbers
    ms, value = res[0]
    assert ms == pytest.approx(0.125)
    assert value == pytest.approx(2 * 404_750_336 / 0.125e-3 / 1e9)
    # one rank alone: no collective, its own time
    assert bench.max_over_ranks(0.1, None, None) == 0.1
    assert bench.whole_job_value(1000, 1, 1.0) == pytest.approx(1000 / 1e-3 / 1e9)


def test_launch_groups_follow_the_layers_data_dependencies():
    import bench
    import workloads as wl
    assert bench.launch_groups(wl.LAYER_LLAMA7B, "deps") == [[0, 1, 2], [3], [4, 5], [6]]
    assert bench.launch_groups(wl.LAYER_LLAMA7B, "all") == [list(range(7))]
    assert bench.launch_groups(wl.LAYER_LLAMA7B, "none") == [[i] for i in range(7)]
    assert bench.launch_groups(wl.FFN_70B, "deps") == [[0], [1]]
