"""The N > 1 path of the benchmark is 'replicas only': ranks share a barrier, the max of their
times and the aggregate throughput. Checked with two gloo ranks on CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2602_06183_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    replicas.barrier()
    ms = replicas.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
    val = replicas.aggregate_tflops(1e12, steps=4, ms_max=ms)
    out.put((rank, replicas.world(), ms, val))
    replicas.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_max_time_and_aggregate_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, ms, val in res:
        assert world == 2
        assert ms == 15.0                                      # the slowest rank's time
        assert abs(val - 2 * 1e12 * 4 / 15e-3 / 1e12) < 1e-9   # two replicas' work over that time


def test_single_process_defaults():
    sys.path.insert(0, ROOT)
    from paper_2602_06183_b200 import replicas
    assert replicas.world() == 1
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.aggregate_tflops(2e12, 5, 10.0) == 2e12 * 5 / 10e-3 / 1e12
