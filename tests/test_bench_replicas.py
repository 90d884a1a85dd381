"""The N > 1 path of bench.py on CPU: ranks are independent replicas; rank times combine by max,
accepted tokens by sum.  Two gloo processes on the loopback interface."""
import os
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.distributed.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, e2e, acc = bench.aggregate_over_ranks(10.0 + 5 * rank, 20.0 - 3 * rank, 7 + rank, world, torch.device("cpu"))
    out.put((rank, ms, e2e, acc))
    torch.distributed.barrier()
    torch.distributed.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_summed_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, acc in got:
        assert (ms, e2e, acc) == (15.0, 20.0, 15.0)      # max(10, 15), max(20, 17), 7 + 8


def test_single_rank_passes_through():
    import bench
    assert bench.aggregate_over_ranks(3.0, 4.0, 5, 1, torch.device("cpu")) == (3.0, 4.0, 5)
