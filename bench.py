"""Benchmark of the verification step: accepted tokens/s and verify-step latency on one B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c4|c5|tg] [--impl ours|reference]

A step is one decode step of the loop: the 64-node draft tree retrieved from the tri-gram table
with the last two tokens of the text, its verification (all layers, LM head, greedy choice,
approval, cache compaction), the tri-gram count update from the emitted tokens and the next
context -- one library call, every stage on the device.  Two passes over the same deterministic decode:
  * end to end: `aded_decode_step_host` -- the step's filler tokens come from pinned host memory,
    the emitted tokens and the accept length are read back to the host before the next step starts;
  * device resident: the cache and the table are rolled back and the same steps run through
    `aded_decode_step` from device memory only.  The emitted tokens must equal the first pass's.
With --gpus N every rank runs an independent replica (nothing in the step is exchanged).
Two more workloads, not part of the default run: `--workload tg` times the tri-gram store alone (bulk update
and top-4 queries on 10^6- and 5 x 10^7-token Zipf corpora, the CPU checker's store beside it), `--workload c5`
the ragged batches of 1, 4 and 16 sequences at the 7B model's full depth.
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
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c4", "c5", "tg"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (debugging only)")
    ap.add_argument("--context", type=int, default=0, help="override the prompt length (debugging only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tg-tokens", default="1000000,50000000", help="corpus sizes of --workload tg")
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
    B.aded_trace_begin(model)      # one timestamp per kernel, taken by one thread: the timed pass is the traced pass
    dev_ms, per_step, launches, accepted, _ = replay(profile=False)
    marks = B.aded_trace_end(model)
    clocks = sampler.stop()
    in_step = stage_times(marks, shape.n_layers)
    assert accepted == accepted_e2e
    final_len = B.aded_kv_len(kv, 0)
    _, _, _, _, (prof_ms, prof_n) = replay(profile=True)

    # ---------------- planted arm: the same decode with a table that knows part of the model's own text ----
    planted = planted_arm(B, model, kv, fresh_table, ctx, ctx0, base_len, fill_d, wl, shape, steps, warm, dev, world, rank)

    # ---------------- roofline of the dominant kernel (the weight-streaming GEMMs) ------------------------
    pk = peaks()
    gemm_bytes_step = shape.weight_bytes_per_step
    gemm_launches_step = 4 * shape.n_layers + 1
    gemm_ms_launch = prof_ms["gemm"] / max(prof_n["gemm"], 1)
    achieved = (gemm_bytes_step / gemm_launches_step) / (gemm_ms_launch * 1e-3) / 1e9
    kv_bytes_step = shape.kv_bytes_per_position() * (base_len + final_len) / 2
    step_bytes = gemm_bytes_step + kv_bytes_step
    whole = step_bytes / (dev_ms / steps * 1e-3) / 1e9
    if in_step:     # the same kernel inside the timed, overlapped pass: weight bytes over the GEMM stages' own time
        gemm_us_step = in_step["us_per_layer_projections"] * shape.n_layers + in_step["us_per_step"].get("gemm_lm_head", 0.0)
        if gemm_us_step > 0:
            in_step["gemm_gbs"] = round(gemm_bytes_step / (gemm_us_step * 1e-6) / 1e9, 1)
            in_step["gemm_frac_of_peak"] = round(in_step["gemm_gbs"] / pk["hbm_gbs"], 4)
    result = {
        "ms": dev_ms, "e2e_ms": e2e_ms, "accepted": accepted, "per_step": per_step, "clocks": clocks,
        "launches": launches, "h2d": h2d, "d2h": d2h, "setup_s": setup_s,
        "roofline": {"bound": "hbm", "kernel": "projection/FFN/LM-head GEMM", "achieved": round(achieved, 1),
                     "peak": pk["hbm_gbs"], "peak_source": pk["source"], "unit": "GB/s",
                     "frac": round(achieved / pk["hbm_gbs"], 4), "traffic": gemm_traffic_per_launch(shape),
                     "algorithmic_bytes_per_launch": gemm_bytes_step // gemm_launches_step,
                     "avg_launch_us": round(gemm_ms_launch * 1e3, 2),
                     "serialised_time_share": {k: round(v / max(sum(prof_ms.values()), 1e-9), 4) for k, v in prof_ms.items()},
                     "in_step": in_step,
                     "whole_step": {"bytes": int(step_bytes), "achieved_gbs": round(whole, 1),
                                    "frac_of_measured_peak": round(whole / pk["hbm_gbs"], 4),
                                    "frac_of_8tbs": round(whole / 8000.0, 4)}},
        "shape": shape, "wl": wl, "context": context, "from_topk": float(d_real[warm:].float().mean()),
        "weights": w, "prompt": prompt, "planted": planted,
    }
    return result


PLANT_KEEP = 0.6        # chance that the table already knows the next tri-gram of the model's text


def planted_arm(B, model, kv, fresh_table, ctx, ctx0, base_len, fill_d, wl, shape, steps, warm, dev, world, rank):
    """A second timed decode in which drafts are approved.  With random-init weights the model's greedy text is
    unrelated to the Zipf prompt, so a table built from the prompt never predicts it (accept length 1 in the main
    arm).  Here the table is taught, step by step, part of what the model is about to say -- the state the paper's
    adaptive table reaches on text it has seen before.  Every step has a seeded target accept length a (geometric:
    one more token with probability PLANT_KEEP, at most depth + 1; mean about 2.4, the range of the paper's
    Table 1).  Before the timed call, a - 1 untimed rehearsal calls of the same step run on the same cache state:
    each emits one token more than the one before and the step's own table update learns its tri-grams; cache
    length and context are rolled back after each.  The timed call then finds the model's path in the top-k
    trees, approves about a tokens and compacts their K/V rows.  (A recorded text cannot be planted instead:
    in a random-init bf16 network a token's logits move by a few percent with its slot in the tree, so a
    replay drifts off any recording within some tens of tokens; rehearsing on the spot keeps the numerics of
    the timed call identical to the last rehearsal's.)  Steps are timed one by one with CUDA events, the
    device idle before each; same model, prompt, cache and filler as the main arm."""
    n, total = wl.tree_nodes, steps + warm
    u = gen.uniform01(total * 8, SEED + rank, 7777).tolist()
    targets = []
    for s in range(total):
        a = 1
        while a < wl.tree_depth + 1 and u[s * 8 + a] < PLANT_KEEP:
            a += 1
        targets.append(a)
    B.aded_kv_set_len(kv, 0, base_len)
    table = fresh_table()
    ctx.copy_(ctx0)
    s_out = torch.zeros(n, dtype=torch.int32, device=dev)
    s_len = torch.zeros(1, dtype=torch.int32, device=dev)
    p_out = torch.zeros((total, n), dtype=torch.int32, device=dev)
    p_len = torch.zeros((total, 1), dtype=torch.int32, device=dev)
    p_real = torch.zeros((total, 1), dtype=torch.int32, device=dev)
    length, times = base_len, []
    if world > 1:
        torch.distributed.barrier()
    for step in range(total):
        saved = ctx.clone()
        for _ in range(targets[step] - 1):                        # rehearsals (untimed)
            B.aded_decode_step(model, kv, table, ctx, n, wl.tree_depth, wl.topk, fill_d[step], s_out, s_len, None)
            B.aded_kv_set_len(kv, 0, length)                      # (synchronises)
            ctx.copy_(saved)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.aded_decode_step(model, kv, table, ctx, n, wl.tree_depth, wl.topk, fill_d[step], p_out[step], p_len[step], p_real[step])
        e1.record()
        torch.cuda.synchronize()
        a = int(p_len[step])
        assert a >= 1, (B.aded_model_poll_status(model), B.aded_trigram_poll_status(table))
        length += a
        times.append(e0.elapsed_time(e1))
    assert B.aded_model_poll_status(model) == 0 and B.aded_trigram_poll_status(table) == 0
    assert B.aded_kv_len(kv, 0) == length
    plens = p_len[:, 0].tolist()
    accepted = sum(plens[warm:])
    ms = sum(times[warm:])
    hist = {}
    for a in plens[warm:]:
        hist[a] = hist.get(a, 0) + 1
    return {"ms": ms, "accepted": accepted, "ms_per_step": ms / steps, "accept_len_mean": accepted / steps,
            "accept_len_target_mean": sum(targets[warm:]) / steps,
            "steps_reaching_their_target": sum(1 for s in range(warm, total) if plens[s] >= targets[s]),
            "accept_len_histogram": {str(k): hist[k] for k in sorted(hist)},
            "tree_nodes_from_table_mean": float(p_real[warm:].float().mean()),
            "timing": "sum of per-step CUDA-event times, device idle before each step (untimed rehearsal calls in between)",
            "table": f"prompt tri-grams, then taught on the spot: target accept length per step geometric with p = {PLANT_KEEP}"}


def stage_times(marks, n_layers):
    """Per-stage times of the timed pass from the device-side trace: every kernel of a pass records when its
    wait for the previous kernel ended; the gap to the next mark is what that kernel added to the pass,
    overlap under programmatic dependent launch included.  Returns microseconds per layer for the per-layer
    stages and per step for the rest, averaged over the whole steps the trace holds."""
    from paper_2407_12021_b200.binding import TRACE_KINDS
    ts, kinds = marks
    ends = [i for i, k in enumerate(kinds) if k == 11]          # a commit ends a pass
    if len(ends) < 2:
        return None
    first, last = ends[0], ends[-1]
    n_steps = len(ends) - 1
    tot = {}
    for i in range(first, last):
        name = "between_passes" if kinds[i] == 11 else TRACE_KINDS.get(kinds[i], str(kinds[i]))
        tot[name] = tot.get(name, 0.0) + (ts[i + 1] - ts[i]) * 1e-3
    per_layer = {k: round(tot.get(k, 0.0) / n_steps / n_layers, 2) for k in
                 ("gemm_qkv", "attention", "gemm_o", "rmsnorm", "gemm_gate_up", "gemm_down", "rotary_kv", "swiglu") if k in tot}
    per_step = {k: round(tot.get(k, 0.0) / n_steps, 1) for k in ("gemm_lm_head", "pick_accept", "other", "between_passes") if k in tot}
    proj = sum(per_layer.get(k, 0.0) for k in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down"))
    return {"steps_traced": n_steps, "us_per_layer": per_layer, "us_per_step": per_step,
            "us_per_layer_projections": round(proj, 2), "us_per_layer_total": round(sum(per_layer.values()), 2),
            "note": "device timestamps at the end of each kernel's dependency wait, in the timed pass; 'between_passes' is the "
                    "commit, the table update, the next context and the next draft tree"}


def zipf_tokens_on(dev, n, vocab, seed, stream):
    """gen.zipf_tokens computed on the device (the same inverse-CDF arithmetic on the same uniform numbers)."""
    out = torch.empty(n, dtype=torch.int32, device=dev)
    cdf = gen.zipf_cdf(vocab).to(dev)
    for s0 in range(0, n, 1 << 24):
        m = min(1 << 24, n - s0)
        u = gen.uniform01(m, seed, stream, device=dev, offset=s0)
        out[s0:s0 + m] = torch.searchsorted(cdf, u).clamp_(max=vocab - 1).to(torch.int32)
    return out


def run_tg(args, rank, world):
    """The tri-gram store alone: Algorithm 2 over a whole corpus in one call, then top-4 lookups (Eq. 1 ranking)
    for contexts drawn from the corpus.  One JSON line per corpus size is printed; the last one is the line of
    the larger corpus (the table then is in the hundreds-of-MB regime the paper reports for its corpora)."""
    from paper_2407_12021_b200 import build as libbuild
    libbuild.build()
    from paper_2407_12021_b200 import binding as B
    from oracle.trigram import TrigramStore
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(dev)
    vocab, k, n_q = 32000, 4, 1 << 20
    pk = peaks()
    reps = max(args.steps if args.steps != 256 else 5, 3)
    lines = []
    for n_tok in [int(v) for v in args.tg_tokens.split(",")]:
        log2b = max(16, min(26, (2 * n_tok - 1).bit_length()))         # about one home bucket per token, a power of two
        overflow = max(1 << 19, n_tok // 6)
        toks = zipf_tokens_on(dev, n_tok, vocab, SEED + rank, 60)
        qi = (gen.uniform01(n_q, SEED + rank, 61, device=dev) * (n_tok - 2)).long()
        ctxs = torch.stack([toks[qi], toks[qi + 1]], dim=1).contiguous()
        out_t = torch.empty((n_q, k), dtype=torch.int32, device=dev)
        out_c = torch.empty((n_q, k), dtype=torch.int32, device=dev)
        upd_ms, top_ms = [], []
        for r in range(reps + 1):                      # first repetition is the warm-up
            t = B.aded_trigram_create(vocab, log2_buckets=log2b, overflow_buckets=overflow)
            torch.cuda.synchronize()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            e[0].record()
            B.aded_trigram_update(t, toks)
            e[1].record()
            B.aded_trigram_topk(t, ctxs, k, out_t, out_c)      # first pass over the queries: table lines come from HBM
            e[2].record()
            torch.cuda.synchronize()
            assert B.aded_trigram_poll_status(t) == 0
            if r:
                upd_ms.append(e[0].elapsed_time(e[1]))
                top_ms.append(e[1].elapsed_time(e[2]))
            entries, buckets = B.aded_trigram_stats(t)
            if r < reps:
                del t
        upd, top = statistics.median(upd_ms), statistics.median(top_ms)
        windows = n_tok - 2
        # algorithmic traffic: one 64-byte bucket read + one 4-byte count written back per window; one bucket per query
        upd_gbs = windows * 68 / (upd * 1e-3) / 1e9
        top_gbs = n_q * 64 / (top * 1e-3) / 1e9
        # the checker's dictionary store on a bounded sample of the same corpus and queries
        sample_tok, sample_q = min(n_tok, 300_000), 20_000
        st = TrigramStore()
        host = toks[:sample_tok].cpu().tolist()
        t0 = time.perf_counter(); st.update(host); cpu_upd = time.perf_counter() - t0
        hq = ctxs[:sample_q].cpu().tolist()
        t0 = time.perf_counter()
        for a, b in hq:
            st.topk(a, b, k)
        cpu_top = time.perf_counter() - t0
        if n_tok == sample_tok:                        # the small corpus is checked in full: lists equal the checker's
            got_t, got_c = out_t[:sample_q].cpu().tolist(), out_c[:sample_q].cpu().tolist()
            for i, (a, b) in enumerate(hq[:2000]):
                assert (got_t[i], got_c[i]) == st.topk(a, b, k), (a, b)
        lines.append({
            "metric": "trigram_update_windows_per_s", "value": windows / (upd * 1e-3), "unit": "windows/s", "n_gpus": 1,
            "steps": reps, "warmup": 1, "ms_per_step": upd, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u32", "data": "synthetic",
            "config": {"workload": f"tg: Zipf(1.1) corpus of {n_tok} tokens over {vocab} ids, one bulk update, then {n_q} top-{k} queries for contexts drawn from the corpus",
                       "l2": "table larger than L2" if buckets * 64 > 126e6 else "table fits L2 (the update of the small corpus is L2 traffic)",
                       "table_mb": round(buckets * 64 / 1e6, 1), "entries": entries, "buckets_in_use": buckets},
            "topk": {"queries_per_s": n_q / (top * 1e-3), "ms": top, "bytes_per_query": 64, "achieved_gbs": round(top_gbs, 1),
                     "frac_of_hbm_peak": round(top_gbs / pk["hbm_gbs"], 4),
                     "note": "64 bytes = the context's home bucket; contexts are drawn by corpus frequency, so most queries hit the few "
                             "hot contexts of a Zipf corpus, whose continuations fill chains of hundreds of buckets that one warp walks"},
            "roofline": {"bound": "hbm", "kernel": "k_tg_update", "achieved": round(upd_gbs, 1), "peak": pk["hbm_gbs"],
                         "peak_source": pk["source"], "unit": "GB/s", "frac": round(upd_gbs / pk["hbm_gbs"], 4), "traffic": None,
                         "algorithmic_bytes_per_window": 68,
                         "note": "random 64-byte buckets: a DRAM sector access is 32-64 bytes of a 64-byte burst, and every window is an atomic read-modify-write"},
            "gpu_launches": 2,
            "cpu_baseline": {"value": (sample_tok - 2) / cpu_upd, "unit": "windows/s", "cores": 1, "kind": "oracle",
                             "sample": f"dictionary store: first {sample_tok} tokens of the corpus ({cpu_upd:.2f} s), {sample_q} of the queries ({cpu_top:.2f} s)",
                             "topk_queries_per_s": sample_q / cpu_top},
            "e2e": None,
        })
        del t, toks
    for line in lines:
        print(json.dumps(line))


def run_c5(args, rank, world):
    """Ragged batches of 1, 4 and 16 sequences at the 7B model's full depth: contexts from U[512, 8192], trees of
    32..128 nodes, caches pre-filled with N(0,1) keys/values; one aded_verify_batch call per step."""
    from paper_2407_12021_b200 import build as libbuild
    libbuild.build()
    from paper_2407_12021_b200 import binding as B
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(dev)
    shape = gen.LLAMA7B if not args.layers else gen.LLAMA7B.with_layers(args.layers)
    w = gen.model_weights(shape, SEED + rank, device=dev)
    pk = peaks()
    bf16_peak = 1388.9
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            bf16_peak = float(json.load(f).get("bf16_tflops_sustained", bf16_peak))
    steps, warm = (args.steps if args.steps != 256 else 10), max(args.warmup, 3)
    batches = {}
    for batch in (1, 4, 16):
        ctx_len = [512 + v for v in gen.randint(batch, 8192 - 512 + 1, SEED + batch, 1)]
        n_nodes = [32 + v for v in gen.randint(batch, 128 - 32 + 1, SEED + batch, 2)]
        depth = [3 + v for v in gen.randint(batch, 6, SEED + batch, 3)]
        rows = sum(n_nodes)
        model = B.aded_model_create(shape, w, max_rows=rows, max_batch=batch)
        kv = B.aded_kv_create(model, [c + 128 for c in ctx_len])
        for b in range(batch):
            for l in range(shape.n_layers):
                kk, vv = gen.kv_normal(shape, ctx_len[b], SEED + 100 + b, l, device=dev)
                B.aded_kv_load(kv, b, l, kk, vv)
        trees = [gen.make_tree(n_nodes[b], depth[b], 6, shape.vocab, SEED + 200 + b) for b in range(batch)]
        offsets = [0]
        for b in range(batch):
            offsets.append(offsets[-1] + n_nodes[b])
        tok = torch.tensor([t for tr in trees for t in tr[0]], dtype=torch.int32, device=dev)
        par = torch.tensor([p for tr in trees for p in tr[1]], dtype=torch.int32, device=dev)
        out = torch.zeros((batch, 128), dtype=torch.int32, device=dev)
        out_len = torch.zeros((batch,), dtype=torch.int32, device=dev)
        times = []
        for step in range(warm + steps):
            for b in range(batch):
                B.aded_kv_set_len(kv, b, ctx_len[b])           # every step verifies from the same committed lengths
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.aded_verify_batch(model, kv, offsets, tok, par, out, out_len)
            e1.record()
            torch.cuda.synchronize()
            if step >= warm:
                times.append(e0.elapsed_time(e1))
        assert B.aded_model_poll_status(model) == 0
        B.aded_trace_begin(model)
        for _ in range(2):                                         # (two passes so that the trace holds a whole one)
            for b in range(batch):
                B.aded_kv_set_len(kv, b, ctx_len[b])
            B.aded_verify_batch(model, kv, offsets, tok, par, out, out_len)
        ts, kinds = B.aded_trace_end(model)
        torch.cuda.synchronize()
        assert B.aded_model_poll_status(model) == 0
        ends = [i for i, kd in enumerate(kinds) if kd == 11]
        gemm_us = attn_us = 0.0
        if len(ends) >= 2:
            for i in range(ends[-2], ends[-1]):
                dt = (ts[i + 1] - ts[i]) * 1e-3
                if kinds[i] in (1, 2, 3, 4, 5):
                    gemm_us += dt
                elif kinds[i] == 6:
                    attn_us += dt
        gemm_us, attn_us = max(gemm_us, 1e-3), max(attn_us, 1e-3)
        ms = statistics.median(times)
        kv_bytes = shape.kv_bytes_per_position() * sum(ctx_len)
        flops = 2.0 * (shape.weight_bytes_per_step / 2) * rows
        passes = (rows + 255) // 256 if rows > 128 else 1      # the tensor-core GEMM takes 256 rows per pass in calls with more than 128
        batches[str(batch)] = {
            "rows": rows, "contexts": ctx_len, "tree_nodes": n_nodes, "ms_per_call": round(ms, 3),
            "accepted_tokens_per_s": float(out_len.sum()) / (ms * 1e-3),
            "algorithmic_bytes": int(shape.weight_bytes_per_step + kv_bytes),
            "hbm_frac_whole_call": round((shape.weight_bytes_per_step + kv_bytes) / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], 4),
            "attention_us": round(attn_us, 1), "attention_hbm_frac": round(kv_bytes / max(attn_us, 1e-9) / 1e3 / pk["hbm_gbs"], 4),
            "gemm_us": round(gemm_us, 1), "gemm_tensor_frac": round(flops / max(gemm_us, 1e-9) / 1e6 / bf16_peak, 4),
            "gemm_weight_passes": passes,
            "gemm_hbm_frac_of_streamed_weights": round(passes * shape.weight_bytes_per_step / max(gemm_us, 1e-9) / 1e3 / pk["hbm_gbs"], 4),
        }
        del kv, model
        torch.cuda.empty_cache()
    b16 = batches["16"]
    line = {"metric": "verify_batch_ms", "value": b16["ms_per_call"], "unit": "ms", "n_gpus": 1, "steps": steps, "warmup": warm,
            "ms_per_step": b16["ms_per_call"], "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": shape.dtype,
            "data": "synthetic",
            "config": {"workload": f"c5: {shape.name} ({shape.n_layers} layers), ragged batches 1 / 4 / 16, contexts U[512, 8192], trees of 32..128 nodes, "
                                   "pre-filled N(0,1) caches, one aded_verify_batch call per step; value = batch 16",
                       "l2": "inputs larger than L2"},
            "batches": batches, "gpu_launches": None, "e2e": None,
            "roofline": {"bound": "tensor" if b16["gemm_tensor_frac"] > b16["hbm_frac_whole_call"] else "hbm",
                         "achieved": round(b16["gemm_tensor_frac"] * bf16_peak, 1), "peak": bf16_peak, "unit": "TFLOP/s",
                         "frac": b16["gemm_tensor_frac"], "traffic": None,
                         "note": "batch 16, projections only; peak = measured sustained bf16 matmul; the tensor-core GEMM makes one pass over the "
                                 "weights per 256 rows (gemm_weight_passes), so its HBM traffic is that many times the weight bytes"}}
    print(json.dumps(line))


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
    wl = gen.WORKLOADS.get(args.workload, gen.WORKLOADS["c3"])

    if args.impl == "reference":
        # The CPU checker as it stands, on the host cores, rank 0 only.  A full 32-layer step takes it about a minute
        # and a half, so a "step" of this arm is a bounded sample of one verification step of the same workload:
        # LAYERS_TIMED decoder layers over the workload's tree and context plus the LM head.  `ms_per_step` is what
        # a step of this arm really took; `value` scales the layer part to the model's depth (stated in the line).
        if rank != 0:
            return
        shape = wl.shape if not args.layers else wl.shape.with_layers(args.layers)
        context = args.context or wl.context
        layers_timed = min(2, shape.n_layers)
        w = gen.model_weights(shape.with_layers(layers_timed), SEED)
        scaled, measured = [], []
        for _ in range(max(args.warmup, 0) + args.steps):
            t0 = time.perf_counter()
            step_s, sample = cpu_oracle_sample(shape, wl, dict(w), context, layers_timed=layers_timed)
            measured.append(time.perf_counter() - t0)
            scaled.append(step_s)
        scaled, measured = scaled[max(args.warmup, 0):], measured[max(args.warmup, 0):]
        step_s = statistics.mean(scaled)
        val = 1.0 / step_s     # one token per step: random-init drafts are accepted at the floor rate
        line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": statistics.mean(measured) * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "layers_timed": layers_timed, "layers_total": shape.n_layers,
                "ms_per_full_step_scaled": step_s * 1e3,
                "config": {"workload": f"{args.workload}: {shape.name}, context {context}, {wl.tree_nodes}-node trees",
                           "note": f"each step of this arm runs {layers_timed} of {shape.n_layers} layers + the LM head of one verification step "
                                   "(ms_per_step); value = 1 token / (layer time x layers_total / layers_timed + head time): "
                                   "accept length taken as 1 token per step"},
                "cpu_baseline": {"value": val, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                                 "sample": sample},
                "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    if args.workload in ("tg", "c5"):
        # secondary workloads: single GPU, rank 0 (replicas would only repeat them)
        if rank == 0:
            (run_tg if args.workload == "tg" else run_c5)(args, rank, world)
        return
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0))))
    res = run_ours(args, rank, world)
    acc = res["accepted"]
    here = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    ms, e2e_ms, acc_total = aggregate_over_ranks(res["ms"], res["e2e_ms"], acc, world, here)
    pl = res["planted"]
    pl_ms, _, pl_acc = aggregate_over_ranks(pl["ms"], pl["ms"], pl["accepted"], world, here)
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
    line["planted"] = {"metric": METRIC, "value": pl_acc / (pl_ms * 1e-3), "unit": UNIT, "ms_per_step": pl_ms / steps,
                       **{k: v for k, v in pl.items() if k not in ("ms", "accepted", "ms_per_step")}}
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
