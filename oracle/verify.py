"""Plain CPU statement of the verification step (test infrastructure, see package header).

What is verified ("Draft Construction and Verification"): the draft candidates are merged
into one pseudo-sequence in which every common prefix appears once -- a token tree -- and
the target model scores all of it in one pass, each tree token attending to the context
and to its own ancestors only ("tree attention").  At every position the model's own
(greedy, the paper's default setting) token is compared with the draft token; a draft is
kept up to its first mismatch, so the output equals plain autoregressive decoding.

The model is a Llama-style decoder (pre-norm RMSNorm, rotary embedding on pairs
(i, i + hd/2), multi-head attention, SwiGLU FFN, untied LM head), which is the family the
paper evaluates.  All arithmetic is float64.  For bf16 models activations are rounded to
bf16 at the points where a bf16 inference pipeline stores them (norm outputs, q/k/v after
rotation, the softmax numerators that multiply V, attention output, the SwiGLU product, the
residual stream); logits are never rounded.  For fp32 models nothing is rounded.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np


@dataclasses.dataclass(frozen=True)
class Arch:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    bf16: bool
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0


def arch_from_shape(shape) -> Arch:
    """Build an Arch from any object with the usual width attributes."""
    return Arch(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn,
                shape.vocab, shape.dtype == "bf16", shape.rms_eps, shape.rope_theta)


# --------------------------------------------------------------------------
# scalar building blocks
# --------------------------------------------------------------------------
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (ties to even), returned as float64.

    bfloat16 keeps 1 sign, 8 exponent and 7 mantissa bits.  A float64 has 52 mantissa bits,
    so the low 45 are rounded away on the integer image of the number; values below the
    bfloat16 normal range are rounded on its subnormal grid (multiples of 2^-133).
    """
    x = np.ascontiguousarray(x, dtype=np.float64)
    bits = x.view(np.uint64)
    lsb = (bits >> np.uint64(45)) & np.uint64(1)
    rounded = (bits + np.uint64((1 << 44) - 1) + lsb) & ~np.uint64((1 << 45) - 1)
    out = rounded.view(np.float64).copy()
    tiny = np.abs(x) < 2.0 ** -126
    if np.any(tiny):
        out[tiny] = np.round(x[tiny] * 2.0 ** 133) * 2.0 ** -133
    big = np.abs(out) > 3.3895313892515355e38  # largest finite bfloat16
    if np.any(big):
        out[big] = np.sign(out[big]) * np.inf
    return out


def rmsnorm(h: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """y = h / sqrt(mean(h^2) + eps) * gain, row by row."""
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding.  x [T, H, hd]; pos [T].  Element i < hd/2 pairs with i + hd/2 and the
    pair is rotated by the angle pos * theta^(-2 i / hd)."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / hd)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]            # [T, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def softmax(s: np.ndarray) -> np.ndarray:
    e = np.exp(s - np.max(s, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def attention_weights(s: np.ndarray, bf16: bool) -> np.ndarray:
    """Softmax weights of scaled scores s [..., n].  Exact for fp32 models.  For bf16 models the
    weights that multiply V are bf16 numbers, as in a bf16 tensor-core pipeline: with t = s * log2(e)
    and the power-of-two reference M = ceil(max t), each numerator 2^(t - M) is rounded to bf16 while
    the denominator sums the unrounded numerators.  (A power-of-two reference makes the rounding
    independent of the order in which keys are visited: rescaling by 2^k commutes with rounding.)"""
    if not bf16:
        return softmax(s)
    t = s * np.log2(np.e)
    m = np.ceil(np.max(t, axis=-1, keepdims=True))
    e = np.exp2(t - m)
    return round_bf16(e) / np.sum(e, axis=-1, keepdims=True)


# --------------------------------------------------------------------------
# tree bookkeeping
# --------------------------------------------------------------------------
def check_tree(parents: Sequence[int]) -> None:
    """Node 0 is the only root and every other node points at an earlier node."""
    if len(parents) < 1 or parents[0] != -1:
        raise ValueError("node 0 must be the root (parent -1)")
    for i in range(1, len(parents)):
        if not (0 <= parents[i] < i):
            raise ValueError(f"parents[{i}] = {parents[i]} is not an earlier node")


def paths_and_depths(parents: Sequence[int]) -> Tuple[List[List[int]], List[int]]:
    """path[i] = nodes from the root down to i (inclusive); depth[i] = edges from the root."""
    check_tree(parents)
    paths: List[List[int]] = []
    for i, p in enumerate(parents):
        paths.append([0] if p < 0 else paths[p] + [i])
    return paths, [len(p) - 1 for p in paths]


# --------------------------------------------------------------------------
# weights and cache
# --------------------------------------------------------------------------
def _f64(t) -> np.ndarray:
    """torch tensor (any float dtype, any device) or array -> float64 numpy array."""
    if hasattr(t, "detach"):
        import torch
        return t.detach().to("cpu").to(torch.float64).numpy()
    return np.asarray(t, dtype=np.float64)


class Weights:
    """Read-only float64 view of a weight dictionary (see inputs.model_weights for the layout).
    Layers are widened on demand so that a 7B model does not have to sit in float64."""

    def __init__(self, raw: Dict[str, object], keep: bool = False):
        self.raw = raw
        self.keep = keep
        self._cache: Dict[object, Dict[str, np.ndarray]] = {}

    def top(self, name: str) -> np.ndarray:
        return _f64(self.raw[name])

    def embed_rows(self, tokens: Sequence[int]) -> np.ndarray:
        e = self.raw["embed"]
        if hasattr(e, "detach"):
            import torch
            idx = torch.as_tensor(list(tokens), dtype=torch.long, device=e.device)
            return _f64(e[idx])
        return np.asarray(e, dtype=np.float64)[list(tokens)]

    def layer(self, l: int) -> Dict[str, np.ndarray]:
        if l in self._cache:
            return self._cache[l]
        out = {k: _f64(v) for k, v in self.raw["layers"][l].items()}
        if self.keep:
            self._cache[l] = out
        return out


class Cache:
    """Per layer K and V of the committed positions: lists of arrays [H, L, hd] (float64)."""

    def __init__(self, arch: Arch):
        z = np.zeros((arch.n_heads, 0, arch.head_dim))
        self.k = [z.copy() for _ in range(arch.n_layers)]
        self.v = [z.copy() for _ in range(arch.n_layers)]

    @property
    def length(self) -> int:
        return self.k[0].shape[1]

    def load(self, layer: int, k, v) -> None:
        self.k[layer] = _f64(k).copy()
        self.v[layer] = _f64(v).copy()

    def clone(self) -> "Cache":
        c = Cache.__new__(Cache)
        c.k = [a.copy() for a in self.k]
        c.v = [a.copy() for a in self.v]
        return c


# --------------------------------------------------------------------------
# the forward pass over a token tree
# --------------------------------------------------------------------------
def decoder_layer(arch: Arch, p: Dict[str, np.ndarray], cache_k: np.ndarray, cache_v: np.ndarray,
                  h: np.ndarray, paths: Sequence[Sequence[int]], pos: np.ndarray, trace: Optional[dict] = None):
    """One decoder layer over the tree's hidden states h [T, d].  cache_k / cache_v [H, L, hd] are the
    layer's committed keys/values.  Returns (h_out [T, d], k [T, H, hd], v [T, H, hd])."""
    r = round_bf16 if arch.bf16 else (lambda a: a)
    T = h.shape[0]
    H, hd, d, F = arch.n_heads, arch.head_dim, arch.d_model, arch.d_ffn
    scale = 1.0 / np.sqrt(hd)
    wq, wk, wv = p["wqkv"][:d], p["wqkv"][d:2 * d], p["wqkv"][2 * d:]
    x1 = x = r(rmsnorm(h, p["norm1"], arch.rms_eps))
    q = r(rope((x @ wq.T).reshape(T, H, hd), pos, arch.rope_theta))
    k = r(rope((x @ wk.T).reshape(T, H, hd), pos, arch.rope_theta))
    v = r((x @ wv.T).reshape(T, H, hd))
    o = np.zeros((T, H, hd))
    for i in range(T):
        # keys node i may see: every cached position, then its ancestors and itself
        keys = np.concatenate([cache_k, k[paths[i]].transpose(1, 0, 2)], axis=1)   # [H, n, hd]
        vals = np.concatenate([cache_v, v[paths[i]].transpose(1, 0, 2)], axis=1)
        s = np.einsum("hd,hnd->hn", q[i], keys) * scale
        o[i] = np.einsum("hn,hnd->hd", attention_weights(s, arch.bf16), vals)
    o = r(o).reshape(T, d)
    h_mid = h = r(h + o @ p["wo"].T)
    x = r(rmsnorm(h, p["norm2"], arch.rms_eps))
    gate, up = x @ p["wgu"][:F].T, x @ p["wgu"][F:].T
    a = r(silu(gate) * up)
    h = r(h + a @ p["wd"].T)
    if trace is not None:      # intermediates, for stage-by-stage comparisons
        trace.update(x1=x1, q=q.reshape(T, d), attn=o, h_mid=h_mid, x2=x, act=a, h=h)
    return h, k, v


def lm_head(arch: Arch, w: Weights, h: np.ndarray) -> np.ndarray:
    """Logits of hidden states h [T, d]: final RMSNorm, then the (untied) output projection."""
    r = round_bf16 if arch.bf16 else (lambda a: a)
    x = r(rmsnorm(h, w.top("final_norm"), arch.rms_eps))
    return x @ w.top("lm_head").T


def forward_tree(arch: Arch, w: Weights, cache: Cache, tokens: Sequence[int],
                 parents: Sequence[int], want_logits: bool = True, trace: Optional[dict] = None):
    """Score every tree node in one pass.

    Returns (logits [T, V] or None, k_new, v_new) where k_new[l], v_new[l] are the tree
    nodes' keys/values of layer l, shape [H, T, hd].  The cache is not modified.  `trace`, when
    given, receives the last layer's intermediates.
    """
    paths, depth = paths_and_depths(parents)
    pos = cache.length + np.asarray(depth)            # a node sits `depth` tokens after the context
    h = w.embed_rows(tokens)                          # residual stream [T, d]
    k_new, v_new = [], []
    for l in range(arch.n_layers):
        h, k, v = decoder_layer(arch, w.layer(l), cache.k[l], cache.v[l], h, paths, pos, trace)
        k_new.append(k.transpose(1, 0, 2).copy())
        v_new.append(v.transpose(1, 0, 2).copy())
    logits = lm_head(arch, w, h) if want_logits else None
    return logits, k_new, v_new


def greedy(logits: np.ndarray) -> np.ndarray:
    """Greedy choice per row: the largest logit, the lowest token id among exact ties."""
    return np.argmax(logits, axis=-1).astype(np.int64)


def top2_margin(logits: np.ndarray) -> np.ndarray:
    """Gap between the largest and second largest logit of every row."""
    part = np.partition(logits, -2, axis=-1)
    return part[:, -1] - part[:, -2]


def accept_walk(tokens: Sequence[int], parents: Sequence[int], best: Sequence[int]):
    """Walk down from the root: emit the model's token at the current node, move to the
    (lowest-numbered) child whose draft token equals it, stop when there is none.
    Returns (path nodes, emitted tokens); len(emitted) = accepted drafts + 1."""
    cur, path, out = 0, [0], []
    while True:
        out.append(int(best[cur]))
        nxt = [c for c in range(cur + 1, len(tokens)) if parents[c] == cur and tokens[c] == best[cur]]
        if not nxt:
            return path, out
        cur = nxt[0]
        path.append(cur)


def verify(arch: Arch, w: Weights, cache: Cache, tokens: Sequence[int], parents: Sequence[int], choose=None):
    """One verification step.  Appends the accepted path's K/V to the cache (root first) and
    returns a dict with out_tokens, accept_len, path, best (per-node chosen token), logits.
    `choose` maps the logits [n, V] to one token per node; the default is the greedy choice."""
    logits, k_new, v_new = forward_tree(arch, w, cache, tokens, parents)
    best = greedy(logits) if choose is None else np.asarray(choose(logits), dtype=np.int64)
    path, out = accept_walk(tokens, parents, best)
    for l in range(arch.n_layers):
        cache.k[l] = np.concatenate([cache.k[l], k_new[l][:, path]], axis=1)
        cache.v[l] = np.concatenate([cache.v[l], v_new[l][:, path]], axis=1)
    return {"out_tokens": out, "accept_len": len(out), "path": path, "best": best, "logits": logits}


def append(arch: Arch, w: Weights, cache: Cache, tokens: Sequence[int], chunk: int = 128) -> None:
    """Put a run of committed tokens into the cache (prefill): a chain 'tree' whose every node
    is accepted by construction.  No logits are needed."""
    for s in range(0, len(tokens), chunk):
        part = list(tokens[s:s + chunk])
        parents = [-1] + list(range(len(part) - 1))
        _, k_new, v_new = forward_tree(arch, w, cache, part, parents, want_logits=False)
        for l in range(arch.n_layers):
            cache.k[l] = np.concatenate([cache.k[l], k_new[l]], axis=1)
            cache.v[l] = np.concatenate([cache.v[l], v_new[l]], axis=1)
