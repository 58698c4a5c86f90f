"""The N > 1 path of bench.py on CPU: two gloo ranks.  The method does not shard across GPUs
(replicas only), so the multi-rank logic is the timing reduction (MAX over ranks) and the
whole-job aggregation; both are exercised here without a GPU."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r measured (10 + r) ms for the device-resident steps and (20 + 2r) ms end to end
    total_ms, e2e_ms = bench.reduce_max_over_ranks([10.0 + rank, 20.0 + 2 * rank])
    dist.barrier()
    value = bench.whole_job_value(units_per_step=8192, steps=5, total_ms=total_ms, world=world)
    out[rank] = (total_ms, e2e_ms, value)
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_to_the_slowest():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
    assert len(out) == world
    for rank in range(world):
        total_ms, e2e_ms, value = out[rank]
        assert total_ms == 11.0 and e2e_ms == 22.0          # the slower rank's times, on every rank
        assert abs(value - world * 8192 * 5 / 11.0e-3) < 1e-6 * value


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_value(100, 2, 1000.0, 1) == 200.0
