"""ctypes binding of libaded.so: one Python function per C entry point, same names.

Argument marshalling only: tensors are passed as raw pointers, every computation happens in the
library's CUDA kernels.  There is no CPU fallback: importing this module without the built
library raises, and a non-OK status raises AdedError.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_float, c_int32, c_uint32, c_uint64, c_void_p
from typing import Dict, List, Optional, Sequence

import torch

# ADED_LIBRARY names another build of the same library (the index-checking debug build, libaded_debug.so)
_LIB_PATH = os.environ.get("ADED_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libaded.so")

ADED_OK = 0
ADED_F32, ADED_BF16 = 0, 1
ADED_MAX_NODES = 128
STATUS_NAMES = {0: "ADED_OK", 1: "ADED_ERR_INVALID_ARG", 2: "ADED_ERR_BAD_TREE", 3: "ADED_ERR_KV_CAPACITY",
                4: "ADED_ERR_TABLE_FULL", 5: "ADED_ERR_OOM", 6: "ADED_ERR_CUDA", 7: "ADED_ERR_UNSUPPORTED",
                8: "ADED_ERR_TIMEOUT", 9: "ADED_ERR_INTERNAL"}

EXPORTS = [
    "aded_model_create", "aded_model_destroy", "aded_kv_create", "aded_kv_destroy", "aded_kv_len",
    "aded_kv_load", "aded_kv_set_len", "aded_kv_read", "aded_append", "aded_verify", "aded_verify_batch", "aded_verify_host",
    "aded_debug_capture", "aded_debug_capture_hidden", "aded_debug_gemm", "aded_debug_read_buffer", "aded_greedy_noalloc", "aded_profile_begin", "aded_profile_end", "aded_trace_begin", "aded_trace_end", "aded_debug_attention_kernel", "aded_debug_weight_layout", "aded_debug_wait_timeout", "aded_launch_count", "aded_model_poll_status", "aded_trigram_create", "aded_trigram_destroy",
    "aded_trigram_update", "aded_trigram_update_host", "aded_trigram_topk", "aded_trigram_topk_host",
    "aded_trigram_get", "aded_trigram_stats", "aded_trigram_poll_status", "aded_draft_tree", "aded_decode_step",
    "aded_decode_step_host", "aded_verify_sampled", "aded_sample_tokens", "aded_trigram_export",
    "aded_trigram_import", "aded_mcts_draft", "aded_decode_step_mcts", "aded_trigram_clear", "aded_trigram_prune", "aded_trigram_save", "aded_trigram_load", "aded_status_string",
]


class AdedError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class ModelConfig(Structure):
    _fields_ = [("n_layers", c_int32), ("d_model", c_int32), ("n_heads", c_int32), ("head_dim", c_int32),
                ("d_ffn", c_int32), ("vocab", c_int32), ("dtype", c_int32), ("rms_eps", c_float),
                ("rope_theta", c_float), ("max_rows", c_int32), ("max_batch", c_int32)]


class LayerWeights(Structure):
    _fields_ = [(n, c_void_p) for n in ("wqkv", "wo", "wgu", "wd", "norm1", "norm2")]


class Weights(Structure):
    _fields_ = [("embed", c_void_p), ("final_norm", c_void_p), ("lm_head", c_void_p),
                ("layers", POINTER(LayerWeights))]


class TrigramConfig(Structure):
    _fields_ = [("vocab", c_int32), ("log2_buckets", c_int32), ("overflow_buckets", c_int32),
                ("cap", c_uint32), ("min_count", c_uint32)]


def load_library(path: str = _LIB_PATH) -> ctypes.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2407_12021_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    for name in EXPORTS:
        fn = getattr(lib, name)          # AttributeError if the symbol is not exported
        fn.restype = {"aded_status_string": c_char_p, "aded_launch_count": c_uint64}.get(name, c_int32)
    return lib


_lib = load_library()


def _check(status: int, where: str) -> None:
    if status != ADED_OK:
        raise AdedError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> c_void_p:
    return c_void_p(0 if t is None else t.data_ptr())


def _stream() -> c_void_p:
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev_i32(t: torch.Tensor, what: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
        raise TypeError(f"{what} must be a contiguous int32 CUDA tensor")
    return t


def _host_i32(t: torch.Tensor, what: str) -> torch.Tensor:
    if t.is_cuda or t.dtype != torch.int32 or not t.is_contiguous():
        raise TypeError(f"{what} must be a contiguous int32 host tensor")
    return t


class Model:
    """Owns an aded_model* and keeps the weight tensors alive."""

    def __init__(self, handle: c_void_p, keep, cfg: ModelConfig):
        self.handle, self._keep, self.cfg = handle, keep, cfg

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.aded_model_destroy(self.handle)
            self.handle = None


class KV:
    def __init__(self, handle: c_void_p, model: Model, batch: int):
        self.handle, self.model, self.batch = handle, model, batch

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.aded_kv_destroy(self.handle)
            self.handle = None


class Trigram:
    def __init__(self, handle: c_void_p, cfg: TrigramConfig):
        self.handle, self.cfg = handle, cfg

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.aded_trigram_destroy(self.handle)
            self.handle = None


# ---- model / cache -----------------------------------------------------------------------
def aded_model_create(shape, weights: Dict[str, object], max_rows: int = 128, max_batch: int = 1) -> Model:
    """shape: any object with n_layers, d_model, n_heads, head_dim, d_ffn, vocab, dtype ("f32"/"bf16"),
    rms_eps, rope_theta.  weights: dict laid out as inputs.model_weights, CUDA tensors."""
    dt = {"f32": (ADED_F32, torch.float32), "bf16": (ADED_BF16, torch.bfloat16)}[shape.dtype]
    cfg = ModelConfig(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                      dt[0], shape.rms_eps, shape.rope_theta, max_rows, max_batch)
    keep = []

    def dev(t: torch.Tensor, dims) -> int:
        if not (t.is_cuda and t.dtype == dt[1] and t.is_contiguous() and tuple(t.shape) == tuple(dims)):
            raise TypeError(f"weight tensor must be contiguous CUDA {dt[1]} of shape {tuple(dims)}, got "
                            f"{t.dtype} {tuple(t.shape)} on {t.device}")
        keep.append(t)
        return t.data_ptr()

    d, f, v = shape.d_model, shape.d_ffn, shape.vocab
    layers = (LayerWeights * shape.n_layers)()
    for l, p in enumerate(weights["layers"]):
        layers[l] = LayerWeights(dev(p["wqkv"], (3 * d, d)), dev(p["wo"], (d, d)), dev(p["wgu"], (2 * f, d)),
                                 dev(p["wd"], (d, f)), dev(p["norm1"], (d,)), dev(p["norm2"], (d,)))
    w = Weights(dev(weights["embed"], (v, d)), dev(weights["final_norm"], (d,)), dev(weights["lm_head"], (v, d)),
                layers)
    out = c_void_p()
    _check(_lib.aded_model_create(ctypes.byref(cfg), ctypes.byref(w), ctypes.byref(out)), "aded_model_create")
    return Model(out, keep, cfg)


def aded_kv_create(model: Model, capacities: Sequence[int]) -> KV:
    caps = (c_int32 * len(capacities))(*capacities)
    out = c_void_p()
    _check(_lib.aded_kv_create(model.handle, c_int32(len(capacities)), caps, ctypes.byref(out)), "aded_kv_create")
    return KV(out, model, len(capacities))


def aded_kv_len(kv: KV, seq: int = 0) -> int:
    out = c_int32()
    _check(_lib.aded_kv_len(kv.handle, c_int32(seq), ctypes.byref(out), _stream()), "aded_kv_len")
    return out.value


def aded_kv_load(kv: KV, seq: int, layer: int, k: torch.Tensor, v: torch.Tensor) -> None:
    assert k.is_cuda and v.is_cuda and k.is_contiguous() and v.is_contiguous() and k.shape == v.shape
    _check(_lib.aded_kv_load(kv.handle, c_int32(seq), c_int32(layer), _ptr(k), _ptr(v), c_int32(k.shape[1]),
                             _stream()), "aded_kv_load")


def aded_kv_set_len(kv: KV, seq: int, new_len: int) -> None:
    _check(_lib.aded_kv_set_len(kv.handle, c_int32(seq), c_int32(new_len), _stream()), "aded_kv_set_len")


def aded_kv_read(kv: KV, seq: int, layer: int, pos0: int, n_pos: int):
    cfg = kv.model.cfg
    dt = torch.bfloat16 if cfg.dtype == ADED_BF16 else torch.float32
    k = torch.empty((cfg.n_heads, n_pos, cfg.head_dim), dtype=dt, device="cuda")
    v = torch.empty_like(k)
    _check(_lib.aded_kv_read(kv.handle, c_int32(seq), c_int32(layer), c_int32(pos0), c_int32(n_pos), _ptr(k),
                             _ptr(v), _stream()), "aded_kv_read")
    return k, v


def aded_append(model: Model, kv: KV, tokens_dev: torch.Tensor, seq: int = 0) -> None:
    _dev_i32(tokens_dev, "tokens")
    _check(_lib.aded_append(model.handle, kv.handle, c_int32(seq), _ptr(tokens_dev), c_int32(tokens_dev.numel()),
                            _stream()), "aded_append")


# ---- verification -----------------------------------------------------------------------
def aded_verify(model: Model, kv: KV, tree_tokens: torch.Tensor, tree_parents: torch.Tensor,
                out_tokens: torch.Tensor, out_accept_len: torch.Tensor) -> None:
    """All four are int32 CUDA tensors; out_tokens has at least as many entries as the tree."""
    n = _dev_i32(tree_tokens, "tree_tokens").numel()
    _dev_i32(tree_parents, "tree_parents"), _dev_i32(out_tokens, "out_tokens"), _dev_i32(out_accept_len, "out_accept_len")
    if tree_parents.numel() != n or out_tokens.numel() < n or out_accept_len.numel() < 1:
        raise ValueError("tree_parents / out_tokens / out_accept_len are too short for the tree")
    _check(_lib.aded_verify(model.handle, kv.handle, _ptr(tree_tokens), _ptr(tree_parents), c_int32(n),
                            _ptr(out_tokens), _ptr(out_accept_len), _stream()), "aded_verify")


def aded_verify_batch(model: Model, kv: KV, tree_offsets: Sequence[int], tree_tokens: torch.Tensor,
                      tree_parents: torch.Tensor, out_tokens: torch.Tensor, out_accept_len: torch.Tensor) -> None:
    """tree_offsets: host list of batch+1 ints; out_tokens [batch, stride] int32 CUDA."""
    _dev_i32(tree_tokens, "tree_tokens"), _dev_i32(tree_parents, "tree_parents")
    _dev_i32(out_tokens, "out_tokens"), _dev_i32(out_accept_len, "out_accept_len")
    if len(tree_offsets) != kv.batch + 1 or out_tokens.dim() != 2 or out_tokens.shape[0] != kv.batch:
        raise ValueError("tree_offsets needs batch+1 entries and out_tokens one row per sequence")
    if tree_tokens.numel() < tree_offsets[-1] or tree_parents.numel() < tree_offsets[-1] or out_accept_len.numel() < kv.batch:
        raise ValueError("token / parent / accept-length arrays are too short")
    offs = (c_int32 * len(tree_offsets))(*tree_offsets)
    _check(_lib.aded_verify_batch(model.handle, kv.handle, offs, _ptr(tree_tokens), _ptr(tree_parents),
                                  _ptr(out_tokens), c_int32(out_tokens.shape[1]), _ptr(out_accept_len), _stream()),
           "aded_verify_batch")


def aded_verify_host(model: Model, kv: KV, tree_tokens: torch.Tensor, tree_parents: torch.Tensor,
                     out_tokens: torch.Tensor, out_accept_len: torch.Tensor) -> None:
    """Same with int32 HOST tensors (pinned memory makes the copies asynchronous); blocks until done."""
    n = _host_i32(tree_tokens, "tree_tokens").numel()
    _host_i32(tree_parents, "tree_parents"), _host_i32(out_tokens, "out_tokens"), _host_i32(out_accept_len, "out_accept_len")
    if tree_parents.numel() != n or out_tokens.numel() < n or out_accept_len.numel() < 1:
        raise ValueError("tree_parents / out_tokens / out_accept_len are too short for the tree")
    _check(_lib.aded_verify_host(model.handle, kv.handle, _ptr(tree_tokens), _ptr(tree_parents), c_int32(n),
                                 _ptr(out_tokens), _ptr(out_accept_len), _stream()), "aded_verify_host")


def aded_debug_capture(model: Model, logits: Optional[torch.Tensor], best: Optional[torch.Tensor]) -> None:
    if logits is not None:
        assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    if best is not None:
        _dev_i32(best, "best")
    _check(_lib.aded_debug_capture(model.handle, _ptr(logits), _ptr(best)), "aded_debug_capture")


def aded_debug_gemm(model: Model, layer: int, which: int, x: torch.Tensor) -> torch.Tensor:
    """y = x @ W^T in fp32 through the library's GEMM kernel; which: 0 wqkv, 1 wo, 2 wgu, 3 wd, 4 LM head."""
    cfg = model.cfg
    d, f = cfg.d_model, cfg.d_ffn
    n = {0: 3 * d, 1: d, 2: 2 * f, 3: d, 4: cfg.vocab}[which]
    k = f if which == 3 else d
    dt = torch.bfloat16 if cfg.dtype == ADED_BF16 else torch.float32
    if not (x.is_cuda and x.dtype == dt and x.is_contiguous() and x.dim() == 2 and x.shape[1] == k):
        raise TypeError(f"x must be a contiguous CUDA {dt} tensor [rows, {k}]")
    y = torch.empty((x.shape[0], n), dtype=torch.float32, device=x.device)
    _check(_lib.aded_debug_gemm(model.handle, c_int32(layer), c_int32(which), _ptr(x), c_int32(x.shape[0]), _ptr(y),
                                _stream()), "aded_debug_gemm")
    return y


def aded_debug_capture_hidden(model: Model, hidden: torch.Tensor) -> None:
    """hidden: CUDA tensor [n_layers + 1, rows, d] in the model dtype; filled by the next verify call."""
    assert hidden.is_cuda and hidden.is_contiguous()
    _check(_lib.aded_debug_capture_hidden(model.handle, _ptr(hidden)), "aded_debug_capture_hidden")


def aded_debug_read_buffer(model: Model, which: int, rows: int) -> torch.Tensor:
    """Activation buffer after the last call's last layer: 0 h, 1 x, 2 q, 3 attention output, 4 SwiGLU product."""
    cfg = model.cfg
    width = cfg.d_ffn if which == 4 else cfg.d_model
    dt = torch.bfloat16 if cfg.dtype == ADED_BF16 else torch.float32
    out = torch.empty((rows, width), dtype=dt, device="cuda")
    _check(_lib.aded_debug_read_buffer(model.handle, c_int32(which), c_int32(rows), _ptr(out), _stream()),
           "aded_debug_read_buffer")
    return out


ADED_NOALLOC_MAX_ROWS = 128


def aded_greedy_noalloc(logits: torch.Tensor, out_best: torch.Tensor) -> None:
    """Greedy token per row of a [rows, vocab] fp32 CUDA logits tensor into out_best ([rows] int32 CUDA),
    without a handle and without any allocation (for callers whose device memory is owned by another
    allocator, or whose decode loop may not call cudaMalloc).  rows <= ADED_NOALLOC_MAX_ROWS.  Calls
    share one fixed scratch array inside the library: keep them on one stream."""
    if not (logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous() and logits.dim() == 2):
        raise TypeError("logits must be a contiguous fp32 CUDA tensor [rows, vocab]")
    _dev_i32(out_best, "out_best")
    if out_best.numel() < logits.shape[0]:
        raise ValueError("out_best is shorter than the number of rows")
    _check(_lib.aded_greedy_noalloc(_ptr(logits), c_int32(logits.shape[0]), c_int32(logits.shape[1]), _ptr(out_best),
                                    _stream()), "aded_greedy_noalloc")


def aded_profile_begin(model: Model) -> None:
    _check(_lib.aded_profile_begin(model.handle), "aded_profile_begin")


def aded_profile_end(model: Model):
    """-> ({"gemm": ms, "attention": ms, "other": ms}, {"gemm": launches, ...})"""
    ms = (c_float * 3)()
    n = (c_int32 * 3)()
    _check(_lib.aded_profile_end(model.handle, ms, n, _stream()), "aded_profile_end")
    names = ("gemm", "attention", "other")
    return dict(zip(names, [float(v) for v in ms])), dict(zip(names, [int(v) for v in n]))


TRACE_KINDS = {0: "other", 1: "gemm_qkv", 2: "gemm_o", 3: "gemm_gate_up", 4: "gemm_down", 5: "gemm_lm_head", 6: "attention",
               7: "rmsnorm", 8: "rotary_kv", 9: "swiglu", 10: "pick_accept", 11: "commit"}


def aded_trace_begin(model: Model) -> None:
    _check(_lib.aded_trace_begin(model.handle, _stream()), "aded_trace_begin")


def aded_trace_end(model: Model, max_marks: int = 16384):
    """Returns (times in ns, kinds) of the last marks, oldest first, as two python lists."""
    ts = (c_uint64 * max_marks)()
    kinds = (c_int32 * max_marks)()
    n = c_int32(0)
    _check(_lib.aded_trace_end(model.handle, ts, kinds, c_int32(max_marks), ctypes.byref(n), _stream()), "aded_trace_end")
    return list(ts[:n.value]), list(kinds[:n.value])


def aded_debug_wait_timeout(model: Model, which: int, limit_cycles: int) -> None:
    _check(_lib.aded_debug_wait_timeout(model.handle, c_int32(which), c_uint64(limit_cycles), _stream()), "aded_debug_wait_timeout")


def aded_debug_attention_kernel(model: Model, which: int) -> None:
    _check(_lib.aded_debug_attention_kernel(model.handle, c_int32(which)), "aded_debug_attention_kernel")


def aded_debug_weight_layout(model: Model, which: int) -> None:
    _check(_lib.aded_debug_weight_layout(model.handle, c_int32(which)), "aded_debug_weight_layout")


def aded_launch_count() -> int:
    return int(_lib.aded_launch_count())


def aded_model_poll_status(model: Model) -> int:
    out = c_int32()
    _check(_lib.aded_model_poll_status(model.handle, ctypes.byref(out), _stream()), "aded_model_poll_status")
    return out.value


# ---- tri-gram store ------------------------------------------------------------------------
def aded_trigram_create(vocab: int, log2_buckets: int = 20, overflow_buckets: int = 1 << 18, cap: int = 0,
                        min_count: int = 0) -> Trigram:
    cfg = TrigramConfig(vocab, log2_buckets, overflow_buckets, cap, min_count)
    out = c_void_p()
    _check(_lib.aded_trigram_create(ctypes.byref(cfg), ctypes.byref(out)), "aded_trigram_create")
    return Trigram(out, cfg)


def aded_trigram_update(t: Trigram, tokens_dev: torch.Tensor) -> None:
    _dev_i32(tokens_dev, "tokens")
    _check(_lib.aded_trigram_update(t.handle, _ptr(tokens_dev), c_int32(tokens_dev.numel()), _stream()),
           "aded_trigram_update")


def aded_trigram_update_host(t: Trigram, tokens_host: torch.Tensor) -> None:
    _host_i32(tokens_host, "tokens")
    _check(_lib.aded_trigram_update_host(t.handle, _ptr(tokens_host), c_int32(tokens_host.numel()), _stream()),
           "aded_trigram_update_host")


def aded_trigram_topk(t: Trigram, ctx_dev: torch.Tensor, k: int, out_tokens: torch.Tensor, out_counts: torch.Tensor,
                      out_total: Optional[torch.Tensor] = None) -> None:
    """ctx_dev [q, 2] int32 CUDA; out_tokens [q, k] int32, out_counts [q, k] int32 (bit pattern of uint32),
    out_total [q] int32 or None."""
    _dev_i32(ctx_dev, "ctx"), _dev_i32(out_tokens, "out_tokens"), _dev_i32(out_counts, "out_counts")
    q = ctx_dev.numel() // 2
    if out_tokens.numel() < q * k or out_counts.numel() < q * k or (out_total is not None and out_total.numel() < q):
        raise ValueError("output arrays are too short")
    _check(_lib.aded_trigram_topk(t.handle, _ptr(ctx_dev), c_int32(q), c_int32(k), _ptr(out_tokens), _ptr(out_counts),
                                  _ptr(out_total), _stream()), "aded_trigram_topk")


def aded_trigram_topk_host(t: Trigram, ctx_host: torch.Tensor, k: int, out_tokens: torch.Tensor,
                           out_counts: torch.Tensor, out_total: Optional[torch.Tensor] = None) -> None:
    _host_i32(ctx_host, "ctx"), _host_i32(out_tokens, "out_tokens"), _host_i32(out_counts, "out_counts")
    q = ctx_host.numel() // 2
    if out_tokens.numel() < q * k or out_counts.numel() < q * k or (out_total is not None and out_total.numel() < q):
        raise ValueError("output arrays are too short")
    _check(_lib.aded_trigram_topk_host(t.handle, _ptr(ctx_host), c_int32(q), c_int32(k), _ptr(out_tokens),
                                       _ptr(out_counts), _ptr(out_total), _stream()), "aded_trigram_topk_host")


def aded_trigram_get(t: Trigram, a: int, b: int, c: int) -> int:
    out = c_uint32()
    _check(_lib.aded_trigram_get(t.handle, c_int32(a), c_int32(b), c_int32(c), ctypes.byref(out), _stream()),
           "aded_trigram_get")
    return out.value


def aded_trigram_stats(t: Trigram):
    e, b = c_uint64(), c_uint64()
    _check(_lib.aded_trigram_stats(t.handle, ctypes.byref(e), ctypes.byref(b), _stream()), "aded_trigram_stats")
    return e.value, b.value


def aded_trigram_poll_status(t: Trigram) -> int:
    out = c_int32()
    _check(_lib.aded_trigram_poll_status(t.handle, ctypes.byref(out), _stream()), "aded_trigram_poll_status")
    return out.value


def aded_draft_tree(t: Trigram, context_dev: torch.Tensor, n_nodes: int, max_depth: int, k: int,
                    filler_dev: Optional[torch.Tensor], tree_tokens: torch.Tensor, tree_parents: torch.Tensor,
                    n_from_table: Optional[torch.Tensor] = None) -> None:
    """context_dev [2] int32 CUDA (second-last, last token); filler_dev int32 CUDA or None;
    tree_tokens / tree_parents [n_nodes] int32 CUDA; n_from_table [1] int32 CUDA or None."""
    _dev_i32(context_dev, "context"), _dev_i32(tree_tokens, "tree_tokens"), _dev_i32(tree_parents, "tree_parents")
    if context_dev.numel() < 2 or tree_tokens.numel() < n_nodes or tree_parents.numel() < n_nodes:
        raise ValueError("arrays are too short")
    nf = 0
    if filler_dev is not None:
        _dev_i32(filler_dev, "filler")
        nf = filler_dev.numel()
    if n_from_table is not None:
        _dev_i32(n_from_table, "n_from_table")
    _check(_lib.aded_draft_tree(t.handle, _ptr(context_dev), c_int32(n_nodes), c_int32(max_depth), c_int32(k),
                                _ptr(filler_dev), c_int32(nf), _ptr(tree_tokens), _ptr(tree_parents),
                                _ptr(n_from_table), _stream()), "aded_draft_tree")


def aded_decode_step(model: Model, kv: KV, t: Trigram, context_dev: torch.Tensor, n_nodes: int, max_depth: int, k: int,
                     filler_dev: Optional[torch.Tensor], out_tokens: torch.Tensor, out_accept_len: torch.Tensor,
                     n_from_table: Optional[torch.Tensor] = None) -> None:
    """One decoding step on the device; context_dev [2] int32 CUDA is read and advanced."""
    _dev_i32(context_dev, "context"), _dev_i32(out_tokens, "out_tokens"), _dev_i32(out_accept_len, "out_accept_len")
    if context_dev.numel() < 2 or out_tokens.numel() < n_nodes or out_accept_len.numel() < 1:
        raise ValueError("arrays are too short")
    nf = 0
    if filler_dev is not None:
        _dev_i32(filler_dev, "filler")
        nf = filler_dev.numel()
    if n_from_table is not None:
        _dev_i32(n_from_table, "n_from_table")
    _check(_lib.aded_decode_step(model.handle, kv.handle, t.handle, _ptr(context_dev), c_int32(n_nodes),
                                 c_int32(max_depth), c_int32(k), _ptr(filler_dev), c_int32(nf), _ptr(out_tokens),
                                 _ptr(out_accept_len), _ptr(n_from_table), _stream()), "aded_decode_step")


def aded_decode_step_host(model: Model, kv: KV, t: Trigram, context_dev: torch.Tensor, n_nodes: int, max_depth: int,
                          k: int, filler_host: Optional[torch.Tensor], out_tokens_host: torch.Tensor,
                          out_accept_len_host: torch.Tensor) -> None:
    """Same with filler, emitted tokens and accept length in (pinned) host memory; returns when done."""
    _dev_i32(context_dev, "context"), _host_i32(out_tokens_host, "out_tokens"), _host_i32(out_accept_len_host, "out_accept_len")
    if context_dev.numel() < 2 or out_tokens_host.numel() < n_nodes or out_accept_len_host.numel() < 1:
        raise ValueError("arrays are too short")
    nf = 0
    if filler_host is not None:
        _host_i32(filler_host, "filler")
        nf = filler_host.numel()
    _check(_lib.aded_decode_step_host(model.handle, kv.handle, t.handle, _ptr(context_dev), c_int32(n_nodes),
                                      c_int32(max_depth), c_int32(k), _ptr(filler_host), c_int32(nf),
                                      _ptr(out_tokens_host), _ptr(out_accept_len_host), _stream()),
           "aded_decode_step_host")


def _dev_f32(t: torch.Tensor, what: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError(f"{what} must be a contiguous CUDA float32 tensor")
    return t


def aded_verify_sampled(model: Model, kv: KV, tree_tokens: torch.Tensor, tree_parents: torch.Tensor, temperature: float,
                        top_p: float, u: torch.Tensor, out_tokens: torch.Tensor, out_accept_len: torch.Tensor) -> None:
    """aded_verify with node i's token drawn with u[i] (CUDA float32 [n_nodes]) instead of the greedy choice."""
    _dev_i32(tree_tokens, "tree_tokens"), _dev_i32(tree_parents, "tree_parents")
    _dev_i32(out_tokens, "out_tokens"), _dev_i32(out_accept_len, "out_accept_len"), _dev_f32(u, "u")
    n = tree_tokens.numel()
    if tree_parents.numel() != n or out_tokens.numel() < n or out_accept_len.numel() < 1 or u.numel() < n:
        raise ValueError("array lengths do not match the tree")
    _check(_lib.aded_verify_sampled(model.handle, kv.handle, _ptr(tree_tokens), _ptr(tree_parents), c_int32(n),
                                    c_float(temperature), c_float(top_p), _ptr(u), _ptr(out_tokens), _ptr(out_accept_len),
                                    _stream()), "aded_verify_sampled")


def aded_sample_tokens(logits: torch.Tensor, temperature: float, top_p: float, u: torch.Tensor, out_tokens: torch.Tensor) -> None:
    """logits CUDA float32 [rows, vocab]; u CUDA float32 [rows]; out_tokens CUDA int32 [rows]."""
    _dev_f32(logits, "logits"), _dev_f32(u, "u"), _dev_i32(out_tokens, "out_tokens")
    if logits.dim() != 2 or u.numel() < logits.shape[0] or out_tokens.numel() < logits.shape[0]:
        raise ValueError("logits must be [rows, vocab] with one u and one output per row")
    _check(_lib.aded_sample_tokens(_ptr(logits), c_int32(logits.shape[0]), c_int32(logits.shape[1]), c_float(temperature),
                                   c_float(top_p), _ptr(u), _ptr(out_tokens), _stream()), "aded_sample_tokens")


def aded_trigram_export(t: Trigram, min_count: int = 0):
    """(keys [n, 3] int32, counts [n] int32 holding uint32 bit patterns) of the entries with count >= min_count, on the device."""
    n = c_uint64()
    _check(_lib.aded_trigram_export(t.handle, c_uint32(min_count), None, None, c_uint64(0), ctypes.byref(n), _stream()),
           "aded_trigram_export")
    keys = torch.empty((n.value, 3), dtype=torch.int32, device="cuda")
    counts = torch.empty((n.value,), dtype=torch.int32, device="cuda")
    if n.value:
        m = c_uint64()
        _check(_lib.aded_trigram_export(t.handle, c_uint32(min_count), _ptr(keys), _ptr(counts), c_uint64(n.value),
                                        ctypes.byref(m), _stream()), "aded_trigram_export")
        if m.value != n.value:
            raise RuntimeError("the table changed during the export")
    return keys, counts


def aded_trigram_import(t: Trigram, keys: torch.Tensor, counts: torch.Tensor) -> None:
    _dev_i32(keys, "keys"), _dev_i32(counts, "counts")
    n = counts.numel()
    if keys.numel() != 3 * n:
        raise ValueError("keys must hold three tokens per count")
    _check(_lib.aded_trigram_import(t.handle, _ptr(keys), _ptr(counts), c_uint64(n), _stream()), "aded_trigram_import")


def aded_trigram_clear(t: Trigram) -> None:
    _check(_lib.aded_trigram_clear(t.handle, _stream()), "aded_trigram_clear")


def aded_trigram_prune(t: Trigram, min_count: int) -> None:
    _check(_lib.aded_trigram_prune(t.handle, c_uint32(min_count), _stream()), "aded_trigram_prune")


def aded_trigram_save(t: Trigram, path: str) -> None:
    _check(_lib.aded_trigram_save(t.handle, path.encode(), _stream()), "aded_trigram_save")


def aded_trigram_load(t: Trigram, path: str) -> None:
    _check(_lib.aded_trigram_load(t.handle, path.encode(), _stream()), "aded_trigram_load")


def aded_mcts_draft(t: Trigram, context_dev: torch.Tensor, iterations: int, length: int, n_candidates: int, k: int,
                    u: torch.Tensor, c1: float = 32.0, c2: float = 8.0, n_nodes_target: int = 0,
                    filler_dev: Optional[torch.Tensor] = None):
    """Runs the tree search; returns (tokens, parents, sentences) as Python lists after synchronising:
    the merged prefix tree (completed to n_nodes_target nodes from filler_dev when given) and the ranked
    sentences [(tokens after the root, mean score)]."""
    nf = 0
    if filler_dev is not None:
        _dev_i32(filler_dev, "filler")
        nf = filler_dev.numel()
    _dev_i32(context_dev, "context"), _dev_f32(u, "u")
    if u.numel() < iterations * length:
        raise ValueError("u must hold iterations * length numbers")
    tok = torch.full((ADED_MAX_NODES,), -9, dtype=torch.int32, device="cuda")
    par = torch.full((ADED_MAX_NODES,), -9, dtype=torch.int32, device="cuda")
    n = torch.zeros(2, dtype=torch.int32, device="cuda")
    st = torch.full((n_candidates, length), -9, dtype=torch.int32, device="cuda")
    sc = torch.zeros(n_candidates, dtype=torch.float64, device="cuda")
    _check(_lib.aded_mcts_draft(t.handle, _ptr(context_dev), c_int32(iterations), c_int32(length), c_int32(n_candidates),
                                c_int32(k), c_float(c1), c_float(c2), _ptr(u), _ptr(tok), _ptr(par), c_void_p(n.data_ptr()),
                                _ptr(st), _ptr(sc), c_void_p(n.data_ptr() + 4), c_int32(n_nodes_target), _ptr(filler_dev), c_int32(nf),
                                _stream()), "aded_mcts_draft")
    torch.cuda.synchronize()
    nn, ns = int(n[0]), int(n[1])
    sentences = [([x for x in st[r].tolist() if x >= 0], float(sc[r])) for r in range(ns)]
    return tok[:nn].tolist(), par[:nn].tolist(), sentences


def aded_decode_step_mcts(model: Model, kv: KV, t: Trigram, context_dev: torch.Tensor, n_nodes: int, iterations: int, length: int,
                          n_candidates: int, k: int, u: torch.Tensor, filler_dev: torch.Tensor, out_tokens: torch.Tensor,
                          out_accept_len: torch.Tensor, c1: float = 32.0, c2: float = 8.0) -> None:
    """One decoding step whose draft tree comes from the tree search; context_dev [2] is read and advanced."""
    _dev_i32(context_dev, "context"), _dev_f32(u, "u"), _dev_i32(filler_dev, "filler")
    _dev_i32(out_tokens, "out_tokens"), _dev_i32(out_accept_len, "out_accept_len")
    if u.numel() < iterations * length or out_tokens.numel() < n_nodes or out_accept_len.numel() < 1:
        raise ValueError("arrays are too short")
    _check(_lib.aded_decode_step_mcts(model.handle, kv.handle, t.handle, _ptr(context_dev), c_int32(n_nodes), c_int32(iterations),
                                      c_int32(length), c_int32(n_candidates), c_int32(k), c_float(c1), c_float(c2), _ptr(u),
                                      _ptr(filler_dev), c_int32(filler_dev.numel()), _ptr(out_tokens), _ptr(out_accept_len),
                                      _stream()), "aded_decode_step_mcts")


def aded_status_string(status: int) -> str:
    return _lib.aded_status_string(c_int32(status)).decode()
