"""Seeded synthetic inputs shared by the CUDA path and the CPU checker.

Everything here produces *inputs*: model shapes, random weights, Zipf token
streams, draft-tree parent arrays, pre-filled KV values and the breadth-first
draft-tree builder that turns top-k continuation lists into a tree.  None of the
verification arithmetic (attention, projections, acceptance, counting) lives in
this module; both implementations consume the same bytes from it.

Random numbers come from one counter-based generator: element ``i`` of stream
``(seed, stream_id)`` is ``mix64(seed * K1 + stream_id * K2 + i)`` with the
SplitMix64 finaliser, so a tensor does not depend on the order in which tensors
are generated.  The generator is written with integer torch ops and runs on
either device; a run generates each tensor once and hands the same bytes to
both implementations.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import torch

_MASK64 = (1 << 64) - 1


# --------------------------------------------------------------------------
# model shapes (the five workloads)
# --------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Llama-style decoder widths."""
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: str  # "f32" or "bf16"
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    def with_layers(self, n_layers: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n_layers,
                                   name=f"{self.name}-{n_layers}L")

    @property
    def params_per_layer(self) -> int:
        d, f = self.d_model, self.d_ffn
        return 4 * d * d + 3 * d * f

    @property
    def weight_bytes_per_step(self) -> int:
        """Bytes of projection, FFN and LM-head weights one verify pass reads."""
        el = 4 if self.dtype == "f32" else 2
        return (self.n_layers * self.params_per_layer + self.vocab * self.d_model) * el

    def kv_bytes_per_position(self) -> int:
        el = 4 if self.dtype == "f32" else 2
        return self.n_layers * 2 * self.d_model * el


TINY = ModelShape("tiny", 2, 256, 4, 64, 688, 4096, "f32")
LLAMA7B_1L = ModelShape("llama7b-1L", 1, 4096, 32, 128, 11008, 32000, "bf16")
LLAMA7B = ModelShape("llama7b", 32, 4096, 32, 128, 11008, 32000, "bf16")
LLAMA13B = ModelShape("llama13b", 40, 5120, 40, 128, 13824, 32000, "bf16")


@dataclasses.dataclass(frozen=True)
class Workload:
    """One of the benchmark/parity workloads: a model shape plus tree/context sizes."""
    key: str
    shape: ModelShape
    context: int            # tokens already in the cache when verification starts
    tree_nodes: int
    tree_depth: int
    branch_max: int
    decode_steps: int = 1
    topk: int = 4
    batch: int = 1


WORKLOADS: Dict[str, Workload] = {
    "c1": Workload("c1", TINY, 64, 16, 4, 4),
    "c2": Workload("c2", LLAMA7B_1L, 1024, 64, 6, 4),
    "c3": Workload("c3", LLAMA7B, 2048, 64, 6, 4, decode_steps=256),
    "c4": Workload("c4", LLAMA13B, 4096, 128, 8, 6, decode_steps=128),
    "c5": Workload("c5", LLAMA7B, 8192, 128, 8, 6, batch=16),
}


# --------------------------------------------------------------------------
# counter-based generator
# --------------------------------------------------------------------------
def _wrap(x: int) -> int:
    """Python int -> the int64 with the same low 64 bits."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def mix64(x: torch.Tensor) -> torch.Tensor:
    """SplitMix64 finaliser on an int64 tensor (two's-complement wrap-around)."""
    x = (x ^ _lsr(x, 30)) * _wrap(0xBF58476D1CE4E5B9)
    x = (x ^ _lsr(x, 27)) * _wrap(0x94D049BB133111EB)
    return x ^ _lsr(x, 31)


def random_bits(n: int, seed: int, stream: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n 64-bit words of stream (seed, stream), as int64."""
    base = _wrap(seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03)
    idx = torch.arange(offset, offset + n, dtype=torch.int64, device=device)
    return mix64(mix64(idx + base) + _wrap(0x9E3779B97F4A7C15))


def uniform01(n: int, seed: int, stream: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n doubles in (0, 1): top 53 bits of each word, plus half an ulp."""
    bits = _lsr(random_bits(n, seed, stream, device, offset), 11)
    return (bits.to(torch.float64) + 0.5) * (1.0 / (1 << 53))


def normal(shape: Sequence[int], std: float, seed: int, stream: int, device="cpu",
           dtype=torch.float32, chunk: int = 1 << 26) -> torch.Tensor:
    """i.i.d. N(0, std^2) by Box-Muller on the counter stream, cast to dtype (RNE)."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    for start in range(0, n, chunk):
        m = min(chunk, n - start)
        u1 = uniform01(m, seed, 2 * stream, device, start)
        u2 = uniform01(m, seed, 2 * stream + 1, device, start)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[start:start + m] = (z * std).to(dtype)
    return out.reshape(*shape)


def randint(n: int, high: int, seed: int, stream: int) -> List[int]:
    """n integers in [0, high) (python list, host)."""
    u = uniform01(n, seed, stream)
    return [min(int(v * high), high - 1) for v in u.tolist()]


# --------------------------------------------------------------------------
# tokens
# --------------------------------------------------------------------------
_ZIPF_CDF: Dict[Tuple[int, float], torch.Tensor] = {}


def zipf_cdf(vocab: int, s: float = 1.1) -> torch.Tensor:
    key = (vocab, s)
    if key not in _ZIPF_CDF:
        r = torch.arange(1, vocab + 1, dtype=torch.float64)
        w = r.pow(-s)
        _ZIPF_CDF[key] = torch.cumsum(w, 0) / w.sum()
    return _ZIPF_CDF[key]


def zipf_tokens(n: int, vocab: int, seed: int, stream: int, s: float = 1.1) -> torch.Tensor:
    """n token ids with P(id = r - 1) proportional to r^-s (inverse CDF), int32 on the host."""
    u = uniform01(n, seed, stream)
    ids = torch.searchsorted(zipf_cdf(vocab, s), u)
    return ids.clamp_(max=vocab - 1).to(torch.int32)


# --------------------------------------------------------------------------
# weights and cache contents
# --------------------------------------------------------------------------
_TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}


def torch_dtype(shape: ModelShape) -> torch.dtype:
    return _TORCH_DTYPE[shape.dtype]


def model_weights(shape: ModelShape, seed: int, device="cpu") -> Dict[str, object]:
    """Random-init weights: every matrix i.i.d. N(0, 0.02^2) in the model dtype, norm gains 1.

    Layout (row-major, output feature major):
      embed [V, d]; per layer wqkv [3d, d] (q rows, then k rows, then v rows; head h owns
      rows h*hd..(h+1)*hd-1 of each block), wo [d, d], wgu [2F, d] (gate rows then up rows),
      wd [d, F], norm1 [d], norm2 [d]; final_norm [d]; lm_head [V, d].
    """
    dt = torch_dtype(shape)
    d, f, v = shape.d_model, shape.d_ffn, shape.vocab
    w: Dict[str, object] = {}
    w["embed"] = normal((v, d), 0.02, seed, 1, device, dt)
    w["lm_head"] = normal((v, d), 0.02, seed, 2, device, dt)
    w["final_norm"] = torch.ones(d, dtype=dt, device=device)
    layers = []
    for l in range(shape.n_layers):
        s0 = 16 + 8 * l
        layers.append({
            "wqkv": normal((3 * d, d), 0.02, seed, s0 + 0, device, dt),
            "wo": normal((d, d), 0.02, seed, s0 + 1, device, dt),
            "wgu": normal((2 * f, d), 0.02, seed, s0 + 2, device, dt),
            "wd": normal((d, f), 0.02, seed, s0 + 3, device, dt),
            "norm1": torch.ones(d, dtype=dt, device=device),
            "norm2": torch.ones(d, dtype=dt, device=device),
        })
    w["layers"] = layers
    return w


def kv_normal(shape: ModelShape, n_pos: int, seed: int, layer: int, device="cpu"):
    """Pre-filled cache contents: K and V [H, n_pos, hd], i.i.d. N(0, 1) in the model dtype."""
    dt = torch_dtype(shape)
    dims = (shape.n_heads, n_pos, shape.head_dim)
    k = normal(dims, 1.0, seed, 4096 + 2 * layer, device, dt)
    v = normal(dims, 1.0, seed, 4096 + 2 * layer + 1, device, dt)
    return k, v


# --------------------------------------------------------------------------
# draft trees
# --------------------------------------------------------------------------
def _unique_sibling_token(existing: set, vocab: int, seed: int, stream: int, start: int) -> Tuple[int, int]:
    """Next Zipf token from the stream that no sibling already uses."""
    pos = start
    while True:
        tok = int(zipf_tokens(1, vocab, seed, stream + pos)[0])
        pos += 1
        if tok not in existing:
            return tok, pos


def make_tree(n_nodes: int, depth: int, branch_max: int, vocab: int, seed: int,
              root_token: Optional[int] = None) -> Tuple[List[int], List[int]]:
    """Seeded draft tree: (tokens, parents), node 0 the root, parents[i] < i.

    Nodes 1..depth form one chain of full depth; every later node picks a parent
    uniformly among nodes with depth < `depth` and fewer than `branch_max` children.
    Sibling tokens are distinct Zipf(1.1) draws.
    """
    assert n_nodes >= 1 and depth >= 0
    parents = [-1]
    dep = [0]
    nchild = [0]
    r = randint(4 * n_nodes + 8, 1 << 30, seed, 7001)
    ri = 0
    for i in range(1, n_nodes):
        if i <= depth:
            p = i - 1
        else:
            cand = [j for j in range(i) if dep[j] < depth and nchild[j] < branch_max]
            if not cand:
                raise ValueError("tree cannot hold that many nodes under the depth/branch limits")
            p = cand[r[ri] % len(cand)]
            ri += 1
        parents.append(p)
        dep.append(dep[p] + 1)
        nchild.append(0)
        nchild[p] += 1
    toks = zipf_tokens(4 * n_nodes + 64, vocab, seed, 7002).tolist()
    ti = 0
    tokens = [toks[0] if root_token is None else int(root_token)]
    ti = 1
    child_tokens: List[set] = [set() for _ in range(n_nodes)]
    for i in range(1, n_nodes):
        p = parents[i]
        while True:
            if ti >= len(toks):
                toks += zipf_tokens(4 * n_nodes, vocab, seed, 7003 + ti).tolist()
            t = toks[ti]
            ti += 1
            if t not in child_tokens[p]:
                break
        child_tokens[p].add(t)
        tokens.append(t)
    return tokens, parents


def tree_depths(parents: Sequence[int]) -> List[int]:
    dep = []
    for i, p in enumerate(parents):
        dep.append(0 if p < 0 else dep[p] + 1)
    return dep


def plant_path(tokens: List[int], parents: Sequence[int], continuation: Sequence[int]) -> List[int]:
    """Overwrite the tokens of the chain 1, 2, ... (node i child of node i-1) with
    `continuation`, keeping sibling tokens distinct.  Used to force chosen accept lengths:
    the caller supplies the tokens it wants accepted."""
    out = list(tokens)
    for j, t in enumerate(continuation):
        i = j + 1
        if i >= len(out) or parents[i] != i - 1:
            break
        for s in range(len(out)):
            if s != i and parents[s] == parents[i] and out[s] == t:
                out[s] = out[i]  # swap the clashing sibling's token away
        out[i] = int(t)
    return out


def expand_tree_from_topk(prev_token: int, root_token: int,
                          topk: Callable[[int, int], Sequence[int]],
                          n_nodes: int, max_depth: int, vocab: int, seed: int,
                          fill: bool = True) -> Tuple[List[int], List[int], int]:
    """Breadth-first draft tree from top-k continuation lists.

    The root holds `root_token`; its context is (prev_token, root_token).  A node with
    context (u, w) gets one child per token of topk(u, w) (negative entries are padding),
    in list order, until `n_nodes` nodes or `max_depth` edges.  When `fill` is set and the
    lists run dry, the remaining nodes are seeded Zipf tokens hung under the shallowest
    nodes that still have room (distinct among siblings), so the verified shape is always
    `n_nodes`.  Returns (tokens, parents, nodes_that_came_from_topk).
    """
    tokens = [int(root_token)]
    parents = [-1]
    dep = [0]
    ctx_prev = [int(prev_token)]
    head = 0
    while head < len(tokens) and len(tokens) < n_nodes:
        if dep[head] < max_depth:
            for t in topk(ctx_prev[head], tokens[head]):
                if t < 0:
                    continue
                if len(tokens) >= n_nodes:
                    break
                tokens.append(int(t))
                parents.append(head)
                dep.append(dep[head] + 1)
                ctx_prev.append(tokens[head])
        head += 1
    from_topk = len(tokens)
    if fill and len(tokens) < n_nodes:
        kids: List[set] = [set() for _ in range(n_nodes)]
        for i in range(1, len(tokens)):
            kids[parents[i]].add(tokens[i])
        pos = 0
        p = 0
        misses = 0
        while len(tokens) < n_nodes:
            # hang one filler under node p if it has room, then move on round-robin
            if dep[p] < max_depth and len(kids[p]) < 4:
                t, pos = _unique_sibling_token(kids[p], vocab, seed, 9000, pos)
                kids[p].add(t)
                tokens.append(t)
                parents.append(p)
                dep.append(dep[p] + 1)
                misses = 0
            else:
                misses += 1
                if misses > len(tokens):
                    raise ValueError("no room left in the tree for filler nodes")
            p = (p + 1) % len(tokens)
    return tokens, parents, from_topk
