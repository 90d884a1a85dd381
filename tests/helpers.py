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


def compare_step(shape, gpu: Dict, cpu: Dict, tokens, parents, where: str = "") -> Dict[str, float]:
    """Element-wise comparison of one verification step.  Returns the worst errors seen."""
    tol = LOGIT_TOL[shape.dtype]
    lg, lc = gpu["logits"], cpu["logits"]
    assert lg.shape == lc.shape
    rel = np.max(np.abs(lg - lc), axis=1) / np.max(np.abs(lc), axis=1)
    assert np.all(rel <= tol), f"{where}: logits off by {rel.max():.3e} (row {int(rel.argmax())}), tolerance {tol}"
    margin = ov.top2_margin(lc)
    delta = np.max(np.abs(lg - lc), axis=1)            # measured logit deviation of every row
    diff = np.nonzero(gpu["best"] != cpu["best"])[0]
    for i in diff:
        # A different greedy token is acceptable only at a near-tie: the checker's margin is below the
        # fixed threshold, or below what this row's measured logit deviation (itself inside the logit
        # tolerance, checked above) can explain -- two logits can each move by delta.
        assert margin[i] < max(MARGIN_EXEMPT, 2 * delta[i]), (
            f"{where}: greedy token of node {i} differs ({gpu['best'][i]} vs {cpu['best'][i]}) with top-2 margin "
            f"{margin[i]:.3e}, logit deviation {delta[i]:.3e}")
    # the accepted sequence must equal the checker's walk over the GPU's own per-node choices;
    # when no node differed that is the checker's answer itself
    path, out = ov.accept_walk(tokens, parents, gpu["best"])
    assert gpu["out_tokens"] == out, f"{where}: emitted {gpu['out_tokens']} but the walk gives {out}"
    assert gpu["accept_len"] == len(out)
    if len(diff) == 0:
        assert gpu["out_tokens"] == cpu["out_tokens"] and gpu["accept_len"] == cpu["accept_len"]
    beyond = int(sum(margin[i] >= MARGIN_EXEMPT for i in diff))
    return {"logit_rel": float(rel.max()), "flipped": int(len(diff)), "flipped_beyond_1e-2": beyond,
            "min_margin": float(margin.min())}


def compare_cache(shape, sess: GpuSession, cache: ov.Cache, pos0: int, n: int, layers: Sequence[int], where=""):
    """Cache rows [pos0, pos0+n) against the checker's, for the given layers."""
    tol = 2e-2 if shape.dtype == "bf16" else 1e-4
    for l in layers:
        k, v = sess.read_kv(l, pos0, n)
        for name, got, want in (("K", k, cache.k[l][:, pos0:pos0 + n]), ("V", v, cache.v[l][:, pos0:pos0 + n])):
            err = np.max(np.abs(got - want)) / max(np.max(np.abs(want)), 1e-30)
            assert err <= tol, f"{where}: layer {l} {name} rows off by {err:.3e}"
