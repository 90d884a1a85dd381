"""Benchmark of the verification step: accepted tokens/s and verify-step latency on one B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c4] [--impl ours|reference]

A step is one decode step of the loop: the 64-node draft tree retrieved from the tri-gram table
with the last two tokens of the text, its verification (all layers, LM head, greedy choice,
approval, cache compaction), the tri-gram count update from the emitted tokens and the next
context -- one library call, every stage on the device.  Two passes over the same deterministic decode:
  * end to end: `aded_decode_step_host` -- the step's filler tokens come from pinned host memory,
    the emitted tokens and the accept length are read back to the host before the next step starts;
  * device resident: the cache and the table are rolled back and the same steps run through
    `aded_decode_step` from device memory only.  The emitted tokens must equal the first pass's.
With --gpus N every rank runs an independent replica (nothing in the step is exchanged).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2407_12021_b200 import inputs as gen  # noqa: E402

SEED = 2407
METRIC = "accepted_tokens_per_s"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c4"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (debugging only)")
    ap.add_argument("--context", type=int, default=0, help="override the prompt length (debugging only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.rows = []
        self.proc = None
        self.idx = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 9 for n, v in zip(names, r[5:9]) if v.lower() == "active"})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def run_ours(args, rank, world):
    from paper_2407_12021_b200 import build as libbuild
    if rank == 0:
        libbuild.build()
    if world > 1:
        torch.distributed.barrier()
    from paper_2407_12021_b200 import binding as B

    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(dev)
    wl = gen.WORKLOADS[args.workload]
    shape = wl.shape if not args.layers else wl.shape.with_layers(args.layers)
    context = args.context or wl.context
    steps, warm = args.steps, max(args.warmup, 3)
    total = steps + warm

    t0 = time.time()
    w = gen.model_weights(shape, SEED + rank, device=dev)
    model = B.aded_model_create(shape, w, max_rows=128, max_batch=1)
    cap = context + (total + 2) * wl.tree_nodes + 256
    kv = B.aded_kv_create(model, [cap])
    prompt = gen.zipf_tokens(context, shape.vocab, SEED + rank, 50)
    if args.workload == "c2":   # pre-filled N(0,1) cache instead of a prefill
        for l in range(shape.n_layers):
            k, v = gen.kv_normal(shape, context - 1, SEED + rank, l, device=dev)
            B.aded_kv_load(kv, 0, l, k, v)
    else:
        pd = prompt[:-1].to(dev)
        for s in range(0, context - 1, 128):
            B.aded_append(model, kv, pd[s:s + 128].contiguous())
    torch.cuda.synchronize()
    base_len = B.aded_kv_len(kv, 0)
    assert base_len == context - 1 and B.aded_model_poll_status(model) == 0
    setup_s = time.time() - t0

    def fresh_table():
        t = B.aded_trigram_create(shape.vocab, log2_buckets=20, overflow_buckets=1 << 16)
        B.aded_trigram_update(t, prompt.to(dev))
        return t

    n = wl.tree_nodes
    nf = 4 * n
    fill_h = torch.stack([gen.zipf_tokens(nf, shape.vocab, SEED + rank, 9000 + s).to(torch.int32) for s in range(total)]).pin_memory()
    fill_d = fill_h.to(dev)
    out_h = torch.empty(n, dtype=torch.int32).pin_memory()
    len_h = torch.empty(1, dtype=torch.int32).pin_memory()
    ctx0 = prompt[-2:].to(torch.int32).to(dev)

    # ---------------- pass 1: end to end, one host-buffer call per step; records the decode ----------
    tg = fresh_table()
    ctx = ctx0.clone()
    torch.cuda.synchronize()
    rec = []
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    sampler = ClockSampler(dev.index or 0)
    accepted_e2e = 0
    for step in range(total):
        if step == warm:
            if world > 1:
                torch.distributed.barrier()
            torch.cuda.synchronize()
            ev[0].record()
        B.aded_decode_step_host(model, kv, tg, ctx, n, wl.tree_depth, wl.topk, fill_h[step], out_h, len_h)
        a = int(len_h[0])
        assert a >= 1, (B.aded_model_poll_status(model), B.aded_trigram_poll_status(tg))
        rec.append(out_h[:a].tolist())
        if step >= warm:
            accepted_e2e += a
    ev[1].record()
    torch.cuda.synchronize()
    e2e_ms = ev[0].elapsed_time(ev[1])
    h2d, d2h = 4 * nf, 4 * (n + 1)
    assert B.aded_trigram_poll_status(tg) == 0 and B.aded_model_poll_status(model) == 0

    # ---------------- pass 2: the same decode from device-resident inputs ---------------------------------
    d_out = torch.zeros((total, n), dtype=torch.int32, device=dev)
    d_len = torch.zeros((total, 1), dtype=torch.int32, device=dev)
    d_real = torch.zeros((total, 1), dtype=torch.int32, device=dev)

    def replay(profile):
        """Rolls cache, table and context back to the end of the prompt and runs all steps from device
        memory.  profile=False is the timed run; profile=True repeats it with per-kernel event timing."""
        B.aded_kv_set_len(kv, 0, base_len)
        table = fresh_table()
        ctx.copy_(ctx0)
        d_out.zero_()
        d_len.zero_()
        torch.cuda.synchronize()
        step_ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        launches0 = 0
        for step in range(total):
            if step == warm:
                if world > 1:
                    torch.distributed.barrier()
                torch.cuda.synchronize()
                launches0 = B.aded_launch_count()
                if profile:
                    B.aded_profile_begin(model)
                step_ev[0].record()
            B.aded_decode_step(model, kv, table, ctx, n, wl.tree_depth, wl.topk, fill_d[step], d_out[step], d_len[step],
                               d_real[step])
            if step >= warm:
                step_ev[step - warm + 1].record()
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        prof = B.aded_profile_end(model) if profile else None
        launches = B.aded_launch_count() - launches0
        lens = d_len[:, 0].tolist()
        for step in range(total):   # the replay must reproduce the recorded decode
            assert d_out[step, :lens[step]].tolist() == rec[step], f"replay diverged at step {step}"
        per_step = [step_ev[i].elapsed_time(step_ev[i + 1]) for i in range(steps)]
        return step_ev[0].elapsed_time(step_ev[-1]), per_step, launches, sum(lens[warm:]), prof

    sampler.start()
    dev_ms, per_step, launches, accepted, _ = replay(profile=False)
    clocks = sampler.stop()
    assert accepted == accepted_e2e
    final_len = B.aded_kv_len(kv, 0)
    _, _, _, _, (prof_ms, prof_n) = replay(profile=True)

    # ---------------- roofline of the dominant kernel (the weight-streaming GEMMs) ------------------------
    pk = peaks()
    gemm_bytes_step = shape.weight_bytes_per_step
    gemm_launches_step = 4 * shape.n_layers + 1
    gemm_ms_launch = prof_ms["gemm"] / max(prof_n["gemm"], 1)
    achieved = (gemm_bytes_step / gemm_launches_step) / (gemm_ms_launch * 1e-3) / 1e9
    kv_bytes_step = shape.kv_bytes_per_position() * (base_len + final_len) / 2
    step_bytes = gemm_bytes_step + kv_bytes_step
    whole = step_bytes / (dev_ms / steps * 1e-3) / 1e9
    result = {
        "ms": dev_ms, "e2e_ms": e2e_ms, "accepted": accepted, "per_step": per_step, "clocks": clocks,
        "launches": launches, "h2d": h2d, "d2h": d2h, "setup_s": setup_s,
        "roofline": {"bound": "hbm", "kernel": "projection/FFN/LM-head GEMM", "achieved": round(achieved, 1),
                     "peak": pk["hbm_gbs"], "peak_source": pk["source"], "unit": "GB/s",
                     "frac": round(achieved / pk["hbm_gbs"], 4), "traffic": gemm_traffic_per_launch(shape),
                     "algorithmic_bytes_per_launch": gemm_bytes_step // gemm_launches_step,
                     "avg_launch_us": round(gemm_ms_launch * 1e3, 2),
                     "time_share": {k: round(v / max(sum(prof_ms.values()), 1e-9), 4) for k, v in prof_ms.items()},
                     "whole_step": {"bytes": int(step_bytes), "achieved_gbs": round(whole, 1),
                                    "frac_of_measured_peak": round(whole / pk["hbm_gbs"], 4),
                                    "frac_of_8tbs": round(whole / 8000.0, 4)}},
        "shape": shape, "wl": wl, "context": context, "from_topk": float(d_real[warm:].float().mean()),
        "weights": w, "prompt": prompt,
    }
    return result


def cpu_oracle_sample(shape, wl, weights, context, layers_timed=6, threads=None):
    """Times the CPU checker on a bounded sample of one verify step: `layers_timed` decoder layers over
    the workload's tree and context, plus the LM head; scaled to the full depth."""
    import numpy as np
    from oracle import verify as ov
    if threads:
        torch.set_num_threads(threads)
    sub = shape.with_layers(min(layers_timed, shape.n_layers))
    arch = ov.arch_from_shape(sub)
    raw = {k: v for k, v in weights.items() if k != "layers"}
    raw["layers"] = weights["layers"][:sub.n_layers]
    ow = ov.Weights(raw)
    cache = ov.Cache(arch)
    for l in range(sub.n_layers):
        k, v = gen.kv_normal(shape, context - 1, SEED, l)
        cache.load(l, k, v)
    tokens, parents = gen.make_tree(wl.tree_nodes, wl.tree_depth, wl.branch_max, shape.vocab, SEED)
    t0 = time.perf_counter()
    logits, _, _ = ov.forward_tree(arch, ow, cache, tokens, parents, want_logits=False)
    t_layers = time.perf_counter() - t0
    t0 = time.perf_counter()
    h = np.zeros((len(tokens), shape.d_model))
    x = ov.round_bf16(ov.rmsnorm(h + 1.0, ow.top("final_norm"), shape.rms_eps))
    ov.greedy(x @ ow.top("lm_head").T)
    t_head = time.perf_counter() - t0
    step_s = t_layers * shape.n_layers / sub.n_layers + t_head
    return step_s, f"1 verify step ({wl.tree_nodes}-node tree, context {context}): {sub.n_layers} of {shape.n_layers} layers + LM head timed ({t_layers + t_head:.1f} s), scaled to {shape.n_layers} layers"


def aggregate_over_ranks(ms, e2e_ms, accepted, world, device):
    """Replicas are independent: the job's time is the slowest rank's, its tokens the sum over ranks."""
    if world <= 1:
        return ms, e2e_ms, accepted
    t = torch.tensor([ms, e2e_ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    a = torch.tensor([accepted], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(a, op=torch.distributed.ReduceOp.SUM)
    return float(t[0]), float(t[1]), float(a[0])


def gemm_traffic_per_launch(shape):
    """DRAM bytes per GEMM launch from the committed ncu capture (profiles/k_gemm_ws_traffic.json), averaged
    over the launches of one step; None when the capture does not belong to the current kernel source."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "k_gemm_ws_traffic.json")
    src = os.path.join(ROOT, "paper_2407_12021_b200", "csrc", "gemm_ws.cu")
    if not (os.path.exists(path) and os.path.exists(src)):
        return None
    with open(path) as f:
        rec = json.load(f)
    with open(src, "rb") as f:
        if hashlib.sha256(f.read()).hexdigest() != rec.get("gemm_ws_sha256"):
            return None
    per = rec.get("dram_bytes_per_launch", {})
    d, f_, v = shape.d_model, shape.d_ffn, shape.vocab
    keys = [f"{3 * d}x{d}", f"{d}x{d}", f"{2 * f_}x{d}", f"{d}x{f_}", f"{v}x{d}"]
    if any(k not in per for k in keys):
        return None
    total = shape.n_layers * sum(per[k] for k in keys[:4]) + per[keys[4]]
    return int(total / (4 * shape.n_layers + 1))


def main():
    args = parse_args()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    wl = gen.WORKLOADS[args.workload]

    if args.impl == "reference":
        # the CPU checker as it stands, rank 0 only
        if rank != 0:
            return
        shape = wl.shape if not args.layers else wl.shape.with_layers(args.layers)
        context = args.context or wl.context
        sub = shape.with_layers(min(2, shape.n_layers))
        w = gen.model_weights(sub, SEED)
        w_full = dict(w)
        times = []
        for _ in range(max(args.warmup, 0) + args.steps):
            s, sample = cpu_oracle_sample(shape, wl, w_full, context, layers_timed=sub.n_layers)
            times.append(s)
        times = times[max(args.warmup, 0):]
        step_s = statistics.mean(times)
        val = 1.0 / step_s     # one token per step: random-init drafts are accepted at the floor rate
        line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": shape.dtype, "data": "synthetic",
                "config": {"workload": f"{args.workload}: {shape.name}, context {context}, {wl.tree_nodes}-node trees",
                           "note": "accept length taken as 1 token per step"},
                "cpu_baseline": {"value": val, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                                 "sample": sample},
                "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0))))
    res = run_ours(args, rank, world)
    acc = res["accepted"]
    ms, e2e_ms, acc_total = aggregate_over_ranks(res["ms"], res["e2e_ms"], acc, world,
                                                 torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0))))
    if rank != 0:
        torch.distributed.destroy_process_group()
        return
    shape, wl, steps = res["shape"], res["wl"], args.steps
    line = {
        "metric": METRIC, "value": acc_total / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": shape.dtype, "data": "synthetic",
        "config": {"workload": f"{args.workload}: {shape.name} ({shape.n_layers} layers, d={shape.d_model}, vocab {shape.vocab}), "
                               f"Zipf(1.1) prompt {res['context']}, {wl.tree_nodes}-node depth-{wl.tree_depth} trees retrieved on the device from tri-gram top-{wl.topk}, "
                               "greedy, batch 1, table updated every step",
                   "l2": "inputs larger than L2 (every step streams all weights)", "replicas": world,
                   "accept_len_mean": acc / steps, "tree_nodes_from_topk_mean": res["from_topk"],
                   "verify_us_median": statistics.median(res["per_step"]) * 1e3},
        "e2e": {"value": acc_total / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms / steps,
                "h2d_bytes_per_step": res["h2d"], "d2h_bytes_per_step": res["d2h"]},
        "gpu_launches": res["launches"], "clocks": res["clocks"], "roofline": res["roofline"],
    }
    if not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        step_s, sample = cpu_oracle_sample(shape, wl, res["weights"], res["context"], threads=cores)
        line["cpu_baseline"] = {"value": (acc / steps) / step_s, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": sample + f"; tokens/s uses the run's mean accept length {acc / steps:.2f}"}
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
