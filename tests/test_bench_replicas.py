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


def test_stage_times_from_a_synthetic_trace():
    """bench.stage_times: marks are (time in ns, kind) at the end of every kernel's dependency wait; the gap to the
    next mark belongs to the earlier kernel; whole passes are delimited by the commit mark (kind 11)."""
    import bench
    layers = 2
    # one pass: prologue-ish (0) 1 us, then per layer qkv (1) 10, rotary (8) 2, attention (6) 5, o (2) 4, norm (7) 1,
    # gate/up (3) 20, swiglu (9) 2, down (4) 8, norm (7) 1; LM head (5) 30, pick (10) 3, commit (11) 7 (until the next pass)
    per_layer = [(1, 10), (8, 2), (6, 5), (2, 4), (7, 1), (3, 20), (9, 2), (4, 8), (7, 1)]
    one_pass = [(0, 1)] + per_layer * layers + [(5, 30), (10, 3), (11, 7)]
    ts, kinds, t = [], [], 1000
    for kind, us in [(11, 7)] + one_pass * 3:          # starts in the middle of a pass: only whole passes count
        ts.append(t)
        kinds.append(kind)
        t += us * 1000
    got = bench.stage_times((ts, kinds), layers)
    assert got["steps_traced"] == 3
    assert got["us_per_layer"] == {"gemm_qkv": 10.0, "attention": 5.0, "gemm_o": 4.0, "rmsnorm": 2.0, "gemm_gate_up": 20.0,
                                   "gemm_down": 8.0, "rotary_kv": 2.0, "swiglu": 2.0}
    assert got["us_per_step"] == {"gemm_lm_head": 30.0, "pick_accept": 3.0, "other": 1.0, "between_passes": 7.0}
    assert got["us_per_layer_projections"] == 42.0 and got["us_per_layer_total"] == 53.0
    assert bench.stage_times(([1, 2], [0, 11]), layers) is None       # no whole pass in the trace
