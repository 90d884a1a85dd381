"""Shared code of the GPU parity tests: run one verification step through the C ABI and through
the CPU checker on the same seeded inputs, and compare."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from oracle import verify as ov
from paper_2407_12021_b200 import inputs as gen

LOGIT_TOL = {"bf16": 2e-2, "f32": 1e-4}      # max |gpu - cpu| / max |cpu| per row
MARGIN_EXEMPT = 1e-2                         # argmax positions with a smaller top-2 gap may differ


def weights_to(weights: Dict[str, object], device) -> Dict[str, object]:
    out = {k: (v.to(device) if hasattr(v, "to") else v) for k, v in weights.items() if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in p.items()} for p in weights["layers"]]
    return out


def i32(x, device="cuda") -> torch.Tensor:
    return torch.tensor(list(x), dtype=torch.int32, device=device)


class GpuSession:
    """Model + single-sequence cache on the GPU, driven through the binding."""

    def __init__(self, shape, weights_cuda, capacity: int, max_rows: int = 128):
        from paper_2407_12021_b200 import binding as B
        self.B = B
        self.shape = shape
        self.model = B.aded_model_create(shape, weights_cuda, max_rows=max_rows, max_batch=1)
        self.kv = B.aded_kv_create(self.model, [capacity])

    def append(self, tokens: Sequence[int], chunk: int = 128) -> None:
        for s in range(0, len(tokens), chunk):
            self.B.aded_append(self.model, self.kv, i32(tokens[s:s + chunk]))

    def verify(self, tokens: Sequence[int], parents: Sequence[int], capture: bool = True):
        n = len(tokens)
        out_tok = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        out_len = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        logits = best = None
        if capture:
            logits = torch.empty((n, self.shape.vocab), dtype=torch.float32, device="cuda")
            best = torch.empty((n,), dtype=torch.int32, device="cuda")
            self.B.aded_debug_capture(self.model, logits, best)
        self.B.aded_verify(self.model, self.kv, i32(tokens), i32(parents), out_tok, out_len)
        torch.cuda.synchronize()
        status = self.B.aded_model_poll_status(self.model)
        a = int(out_len[0])
        return {"status": status, "accept_len": a, "out_tokens": out_tok[:max(a, 0)].tolist(),
                "out_raw": out_tok.tolist(),
                "logits": None if logits is None else logits.cpu().double().numpy(),
                "best": None if best is None else best.cpu().numpy().astype(np.int64)}

    def length(self) -> int:
        return self.B.aded_kv_len(self.kv, 0)

    def read_kv(self, layer: int, pos0: int, n: int):
        k, v = self.B.aded_kv_read(self.kv, 0, layer, pos0, n)
        torch.cuda.synchronize()
        return k.cpu().double().numpy(), v.cpu().double().numpy()


def compare_step(shape, gpu: Dict, cpu: Dict, tokens, parents, where: str = "", beyond_allowance: int = 0,
                 logit_tol: Optional[float] = None) -> Dict[str, float]:
    """Element-wise comparison of one verification step.  Returns the worst errors seen.

    Logits: per row max |gpu - cpu| / max |cpu| within `logit_tol` (default: the dtype's tolerance).
    Greedy tokens: equal, except at near-ties.  The asserted bar is the fixed one: a differing token is
    exempt only where the checker's top-2 margin is below MARGIN_EXEMPT (1e-2).  `beyond_allowance` is the
    number of differing tokens with a larger margin a test tolerates; it is 0 unless the test states, beside
    the call, why more are expected (an end-to-end run through several layers of a random-init bf16 network,
    whose logits legitimately differ by up to the logit tolerance).  Even an allowed one must be explained by
    the measured deviation of its own row (margin < 2 x that row's max |gpu - cpu|: two logits can each move
    by that much), and every one is printed."""
    tol = LOGIT_TOL[shape.dtype] if logit_tol is None else logit_tol
    lg, lc = gpu["logits"], cpu["logits"]
    assert lg.shape == lc.shape
    rel = np.max(np.abs(lg - lc), axis=1) / np.max(np.abs(lc), axis=1)
    assert np.all(rel <= tol), f"{where}: logits off by {rel.max():.3e} (row {int(rel.argmax())}), tolerance {tol}"
    margin = ov.top2_margin(lc)
    delta = np.max(np.abs(lg - lc), axis=1)            # measured logit deviation of every row
    diff = np.nonzero(gpu["best"] != cpu["best"])[0]
    beyond = []
    for i in diff:
        if margin[i] < MARGIN_EXEMPT:
            continue
        beyond.append(int(i))
        print(f"{where}: greedy token of node {i} differs ({gpu['best'][i]} vs {cpu['best'][i]}) beyond the 1e-2 margin: "
              f"top-2 margin {margin[i]:.3e}, logit deviation of the row {delta[i]:.3e}")
        assert margin[i] < 2 * delta[i], f"{where}: node {i}: margin {margin[i]:.3e} is not explained by the row's deviation {delta[i]:.3e}"
    assert len(beyond) <= beyond_allowance, (
        f"{where}: {len(beyond)} greedy tokens differ where the checker's top-2 margin is >= {MARGIN_EXEMPT} "
        f"(nodes {beyond}); allowed here: {beyond_allowance}")
    # the accepted sequence must equal the checker's walk over the GPU's own per-node choices;
    # when no node differed that is the checker's answer itself
    path, out = ov.accept_walk(tokens, parents, gpu["best"])
    assert gpu["out_tokens"] == out, f"{where}: emitted {gpu['out_tokens']} but the walk gives {out}"
    assert gpu["accept_len"] == len(out)
    if len(diff) == 0:
        assert gpu["out_tokens"] == cpu["out_tokens"] and gpu["accept_len"] == cpu["accept_len"]
    return {"logit_rel": float(rel.max()), "flipped": int(len(diff)), "flipped_beyond_1e-2": len(beyond),
            "min_margin": float(margin.min())}


def layerwise_check(arch, ow, tokens, parents, L: int, hidden: np.ndarray, cache_before: Dict[int, tuple],
                    gpu: Dict, where: str, shape, max_tol: float = 2e-2, rms_tol: float = 1e-2) -> Dict[str, float]:
    """Teacher-forced, layer-by-layer comparison of a verification step at the model's full depth.

    `hidden` [n_layers + 1][T][d] is the device's residual stream before layer 0 and after every layer,
    `cache_before[l]` = (K, V) [H, L, hd] the committed cache of layer l the step started from, for the
    layers to check.  Each such layer is re-run by the checker from the device's own input and cache and
    must give the device's output within max_tol (max) / rms_tol (rms) of the output's scale; the LM
    head and the greedy choice are re-run from the device's final hidden states and held to the fixed
    token rule (no differing token where the checker's top-2 margin is >= 1e-2).  Returns the worst
    figures and, per checked layer, the keys/values the checker computed for the tree nodes."""
    paths, depth = ov.paths_and_depths(parents)
    pos = L + np.asarray(depth)
    assert np.array_equal(hidden[0], ow.embed_rows(tokens)), f"{where}: embedding rows are copies"
    worst_max, worst_rms, kv_new = 0.0, 0.0, {}
    for l in sorted(cache_before):
        kc, vc = cache_before[l]
        h_out, k, v = ov.decoder_layer(arch, ow.layer(l), kc, vc, hidden[l], paths, pos)
        err = np.abs(h_out - hidden[l + 1])
        rel_max = err.max() / np.abs(h_out).max()
        rel_rms = float(np.sqrt((err ** 2).mean() / (h_out ** 2).mean()))
        print(f"{where} layer {l}: max {rel_max:.3e} rms {rel_rms:.3e} differing {np.mean(err > 0):.3f}")
        assert rel_max <= max_tol and rel_rms <= rms_tol, (where, l, rel_max, rel_rms)
        worst_max, worst_rms = max(worst_max, float(rel_max)), max(worst_rms, rel_rms)
        kv_new[l] = (k, v)
    lc = ov.lm_head(arch, ow, hidden[arch.n_layers])
    step_cpu = {"logits": lc, "best": ov.greedy(lc)}
    step_cpu["out_tokens"] = ov.accept_walk(tokens, parents, step_cpu["best"])[1]
    step_cpu["accept_len"] = len(step_cpu["out_tokens"])
    head = compare_step(shape, gpu, step_cpu, tokens, parents, f"{where} LM head", beyond_allowance=0, logit_tol=2e-3)
    print(f"{where} LM head from the device's hidden states:", head)
    return {"layer_max": worst_max, "layer_rms": worst_rms, "head": head, "kv_new": kv_new, "cpu": step_cpu}


def compare_cache(shape, sess: GpuSession, cache: ov.Cache, pos0: int, n: int, layers: Sequence[int], where=""):
    """Cache rows [pos0, pos0+n) against the checker's, for the given layers."""
    tol = 2e-2 if shape.dtype == "bf16" else 1e-4
    for l in layers:
        k, v = sess.read_kv(l, pos0, n)
        for name, got, want in (("K", k, cache.k[l][:, pos0:pos0 + n]), ("V", v, cache.v[l][:, pos0:pos0 + n])):
            err = np.max(np.abs(got - want)) / max(np.max(np.abs(want)), 1e-30)
            assert err <= tol, f"{where}: layer {l} {name} rows off by {err:.3e}"
