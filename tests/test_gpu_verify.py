"""GPU parity of the verification step against the CPU checker, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import verify as ov
from paper_2407_12021_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _c1_setup(cuda_device, seed=11):
    shape = gen.TINY
    w = gen.model_weights(shape, seed)
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=256)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    prompt = gen.zipf_tokens(64, shape.vocab, seed, 50).tolist()
    cache = ov.Cache(arch)
    ov.append(arch, ow, cache, prompt[:-1])
    sess.append(prompt[:-1])
    assert sess.length() == 63
    return shape, arch, ow, cache, sess, prompt


def test_c1_tiny_fp32_tree(cuda_device):
    """Workload 1: 2-layer fp32 decoder, 64-token Zipf prompt, 16-node depth-4 tree."""
    shape, arch, ow, cache, sess, prompt = _c1_setup(cuda_device)
    H.compare_cache(shape, sess, cache, 0, 63, range(shape.n_layers), "prefill")
    tokens, parents = gen.make_tree(16, 4, 4, shape.vocab, 3, root_token=prompt[-1])
    cpu = ov.verify(arch, ow, cache, tokens, parents)
    gpu = sess.verify(tokens, parents)
    assert gpu["status"] == 0
    worst = H.compare_step(shape, gpu, cpu, tokens, parents, "c1")
    assert worst["flipped"] == 0
    assert sess.length() == cache.length
    H.compare_cache(shape, sess, cache, 63, cpu["accept_len"], range(shape.n_layers), "after verify")


def test_c1_planted_paths_and_multi_step(cuda_device):
    """Accept lengths 1..5: plant the checker's own greedy continuation on the deep chain, then keep
    decoding from the resulting cache so that compaction errors would surface in the next step."""
    shape, arch, ow, cache, sess, prompt = _c1_setup(cuda_device, seed=12)
    # the checker's autoregressive continuation
    probe = cache.clone()
    cur, ar = prompt[-1], []
    for _ in range(24):
        cur = ov.verify(arch, ow, probe, [cur], [-1])["out_tokens"][0]
        ar.append(cur)
    done = 0
    root = prompt[-1]
    seen = set()
    for step, p in enumerate([2, 0, 4, 1, 3, 4]):
        tokens, parents = gen.make_tree(16, 4, 4, shape.vocab, 100 + step, root_token=root)
        tokens = gen.plant_path(tokens, parents, ar[done:done + p])
        cpu = ov.verify(arch, ow, cache, tokens, parents)
        gpu = sess.verify(tokens, parents)
        assert gpu["status"] == 0
        worst = H.compare_step(shape, gpu, cpu, tokens, parents, f"step {step}")
        assert worst["flipped"] == 0
        assert cpu["accept_len"] >= p + 1
        seen.add(cpu["accept_len"])
        assert gpu["out_tokens"] == ar[done:done + cpu["accept_len"]]
        done += cpu["accept_len"]
        root = gpu["out_tokens"][-1]
        assert sess.length() == cache.length == 63 + done
        H.compare_cache(shape, sess, cache, 63, done, range(shape.n_layers), f"cache after step {step}")
    assert {1, 2, 3, 5} <= seen


def test_scattered_accept_path_is_compacted(cuda_device):
    shape, arch, ow, cache, sess, prompt = _c1_setup(cuda_device, seed=13)
    probe = cache.clone()
    cur, ar = prompt[-1], []
    for _ in range(4):
        cur = ov.verify(arch, ow, probe, [cur], [-1])["out_tokens"][0]
        ar.append(cur)
    wrong = lambda t: (t + 17) % shape.vocab
    parents = [-1, 0, 0, 1, 1, 2, 2, 5, 5, 8]
    tokens = [prompt[-1], wrong(ar[0]), ar[0], wrong(ar[1]), wrong(ar[0]), ar[1], wrong(ar[1]), wrong(ar[2]),
              ar[2], wrong(ar[3])]
    cpu = ov.verify(arch, ow, cache, tokens, parents)
    assert cpu["path"] == [0, 2, 5, 8]
    gpu = sess.verify(tokens, parents)
    H.compare_step(shape, gpu, cpu, tokens, parents, "scattered")
    assert gpu["out_tokens"] == ar[:4]
    H.compare_cache(shape, sess, cache, 63, 4, range(shape.n_layers), "scattered path")
    # the next step reads the compacted rows
    tokens2, parents2 = gen.make_tree(9, 3, 3, shape.vocab, 5, root_token=ar[3])
    cpu2 = ov.verify(arch, ow, cache, tokens2, parents2)
    gpu2 = sess.verify(tokens2, parents2)
    H.compare_step(shape, gpu2, cpu2, tokens2, parents2, "after compaction")


def test_single_node_tree_is_autoregressive_decoding(cuda_device):
    shape, arch, ow, cache, sess, prompt = _c1_setup(cuda_device, seed=14)
    cur = prompt[-1]
    for step in range(5):
        cpu = ov.verify(arch, ow, cache, [cur], [-1])
        gpu = sess.verify([cur], [-1])
        H.compare_step(shape, gpu, cpu, [cur], [-1], f"ar {step}")
        assert gpu["accept_len"] == 1
        cur = gpu["out_tokens"][0]


def test_chain_tree_equals_append(cuda_device):
    """A chain verified as a tree leaves the same K/V rows as appending the same tokens."""
    shape, arch, ow, cache, sess, prompt = _c1_setup(cuda_device, seed=15)
    more = gen.zipf_tokens(7, shape.vocab, 15, 77).tolist()
    sess.append(more)
    k_app, v_app = sess.read_kv(1, 63, 7)
    # a second session verifies the chain; whatever is accepted, slots 63.. hold the chain rows before compaction
    w = gen.model_weights(shape, 15)
    sess2 = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=256)
    sess2.append(prompt[:-1])
    gpu = sess2.verify(more, [-1] + list(range(6)))
    n = gpu["accept_len"]
    k2, v2 = sess2.read_kv(1, 63, n)
    assert np.array_equal(k2, k_app[:, :n]) and np.array_equal(v2, v_app[:, :n])


def test_device_detected_errors_leave_cache_unchanged(cuda_device):
    shape, arch, ow, cache, sess, prompt = _c1_setup(cuda_device, seed=16)
    before = sess.read_kv(0, 0, 63)
    for tokens, parents, code in (([1, 2, 3], [-1, 2, 0], 2), ([1, 2, 3], [0, 0, 1], 2), ([1, 2, 3], [-1, -1, 0], 2),
                                  ([1, shape.vocab, 3], [-1, 0, 0], 1)):
        gpu = sess.verify(tokens, parents, capture=False)
        assert gpu["status"] == code and gpu["accept_len"] == 0
        assert gpu["out_raw"] == [-7] * len(tokens)
        assert sess.length() == 63
    after = sess.read_kv(0, 0, 63)
    assert np.array_equal(before[0], after[0]) and np.array_equal(before[1], after[1])
    # capacity: 63 cached + 200 > 256 is caught on the device ...
    small = H.GpuSession(shape, H.weights_to(gen.model_weights(shape, 16), cuda_device), capacity=70)
    small.append(prompt[:-1])
    tokens, parents = gen.make_tree(16, 4, 4, shape.vocab, 3)
    gpu = small.verify(tokens, parents, capture=False)
    assert gpu["status"] == 3 and gpu["accept_len"] == 0 and small.length() == 63
    # ... and the handle works again after the status was read
    gpu = small.verify(tokens[:5], [-1, 0, 1, 2, 3], capture=False)
    assert gpu["status"] == 0 and gpu["accept_len"] >= 1
    # host-detected: too many nodes
    from paper_2407_12021_b200.binding import AdedError
    with pytest.raises(AdedError):
        sess.verify(list(range(129)), [-1] + list(range(128)), capture=False)


def test_verify_host_entry_point(cuda_device):
    shape, arch, ow, cache, sess, prompt = _c1_setup(cuda_device, seed=17)
    tokens, parents = gen.make_tree(16, 4, 4, shape.vocab, 9, root_token=prompt[-1])
    cpu = ov.verify(arch, ow, cache, tokens, parents)
    B = sess.B
    t = torch.tensor(tokens, dtype=torch.int32).pin_memory()
    p = torch.tensor(parents, dtype=torch.int32).pin_memory()
    out = torch.zeros(16, dtype=torch.int32).pin_memory()
    n = torch.zeros(1, dtype=torch.int32).pin_memory()
    B.aded_verify_host(sess.model, sess.kv, t, p, out, n)
    assert int(n[0]) == cpu["accept_len"] and out[:int(n[0])].tolist() == cpu["out_tokens"]


def test_c2_one_7b_layer_bf16(cuda_device):
    """Workload 2: one Llama-2-7B-shaped layer + LM head in bf16, cache pre-filled with 1024 N(0,1)
    positions, 64-node depth-6 tree with branching <= 4."""
    shape = gen.LLAMA7B_1L
    w = gen.model_weights(shape, 21, device=cuda_device)
    sess = H.GpuSession(shape, w, capacity=1024 + 128)
    k, v = gen.kv_normal(shape, 1024, 21, 0, device=cuda_device)
    sess.B.aded_kv_load(sess.kv, 0, 0, k, v)
    assert sess.length() == 1024
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    cache = ov.Cache(arch)
    cache.load(0, k, v)
    tokens, parents = gen.make_tree(64, 6, 4, shape.vocab, 22)
    cpu = ov.verify(arch, ow, cache, tokens, parents)
    gpu = sess.verify(tokens, parents)
    assert gpu["status"] == 0
    worst = H.compare_step(shape, gpu, cpu, tokens, parents, "c2")
    print("c2 worst", worst)
    if worst["flipped"] == 0:
        H.compare_cache(shape, sess, cache, 1024, cpu["accept_len"], [0], "c2 cache")
    # planted: the checker's greedy tokens along the deep chain are accepted
    cache2 = ov.Cache(arch)
    cache2.load(0, k, v)
    sess.B.aded_kv_load(sess.kv, 0, 0, k, v)
    planted = list(tokens)
    paths, _ = ov.paths_and_depths(parents)
    planted[1] = int(cpu["best"][0])
    cpu2 = ov.verify(arch, ow, cache2, planted, parents)
    gpu2 = sess.verify(planted, parents)
    H.compare_step(shape, gpu2, cpu2, planted, parents, "c2 planted")
    assert cpu2["accept_len"] >= 2


def test_one_7b_layer_stage_by_stage(cuda_device):
    """Where a layer's deviation arises: one 7B-shaped layer from identical inputs (the embedding rows are copies),
    the device's buffers after the rotary step, the attention, the SwiGLU product and the second residual add
    against the checker's intermediates.  Every stage is held to the layer tolerance (2e-2 of the stage's range,
    1e-2 rms); the share of elements that differ at all is printed: the first stage differs only where an fp32
    sum lands within rounding distance of a bf16 tie, and every later stage inherits and spreads those."""
    shape = gen.LLAMA7B_1L
    w = gen.model_weights(shape, 21, device=cuda_device)
    sess = H.GpuSession(shape, w, capacity=1024 + 128)
    k, v = gen.kv_normal(shape, 1024, 21, 0, device=cuda_device)
    sess.B.aded_kv_load(sess.kv, 0, 0, k, v)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    cache = ov.Cache(arch)
    cache.load(0, k, v)
    tokens, parents = gen.make_tree(64, 6, 4, shape.vocab, 22)
    trace = {}
    ov.forward_tree(arch, ow, cache, tokens, parents, want_logits=False, trace=trace)
    gpu = sess.verify(tokens, parents, capture=False)
    assert gpu["status"] == 0
    T = len(tokens)
    for which, name in ((2, "q"), (3, "attn"), (4, "act"), (0, "h")):
        dev = sess.B.aded_debug_read_buffer(sess.model, which, T).double().cpu().numpy()
        ref = np.asarray(trace[name], dtype=np.float64).reshape(dev.shape)
        err = np.abs(dev - ref)
        scale = np.abs(ref).max()
        rms = float(np.sqrt((err ** 2).mean() / (ref ** 2).mean()))
        print(f"stage {name}: {100.0 * np.count_nonzero(err) / err.size:.3f} % of elements differ, "
              f"max {err.max() / scale:.2e} of the range, rms {rms:.2e}")
        assert err.max() <= 2e-2 * scale and rms <= 1e-2, name


@pytest.mark.parametrize("nodes,ctx,depth", [(100, 300, 6), (64, 2047, 6), (5, 1, 2), (128, 1000, 8), (65, 31, 7), (97, 4100, 5)])
def test_attention_kernels_agree(cuda_device, nodes, ctx, depth):
    """head_dim 128 has two attention kernels: tcgen05 (the default) and mma.sync (selected with
    aded_debug_attention_kernel).  Same rounding points (integer reference in the log2 domain, numerators
    rounded to bf16, unrounded row sums); the fp32 sums run in another order, so outputs agree to a few bf16 ulps."""
    from paper_2407_12021_b200 import binding as B
    shape = gen.ModelShape("bf16-4x128", 2, 512, 4, 128, 1024, 1024, "bf16")
    w = H.weights_to(gen.model_weights(shape, 31), cuda_device)
    tokens, parents = gen.make_tree(nodes, depth, 4, shape.vocab, 32)
    results = []
    for mma in (False, True):
        m = B.aded_model_create(shape, w, max_rows=128, max_batch=1)
        B.aded_debug_attention_kernel(m, 1 if mma else 0)
        kv = B.aded_kv_create(m, [ctx + 256])
        for l in range(shape.n_layers):
            k, v = gen.kv_normal(shape, ctx, 33, l, device=cuda_device)
            B.aded_kv_load(kv, 0, l, k, v)
        out = torch.full((nodes,), -7, dtype=torch.int32, device="cuda")
        alen = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        B.aded_verify(m, kv, H.i32(tokens), H.i32(parents), out, alen)
        torch.cuda.synchronize()
        assert B.aded_model_poll_status(m) == 0
        results.append((B.aded_debug_read_buffer(m, 3, nodes).float().clone(), B.aded_debug_read_buffer(m, 0, nodes).float().clone()))
    (att0, h0), (att1, h1) = results
    assert (att0 - att1).abs().max() <= 2e-2 * att0.abs().max()
    assert (h0 - h1).abs().max() <= 2e-2 * h0.abs().max()
    assert att0.abs().max() > 0


def test_weight_layouts_agree_bit_for_bit(cuda_device):
    """The tensor-core GEMM reads the model's re-tiled private copies of the weight matrices by default and the
    caller's row-major matrices on request (aded_debug_weight_layout): the same sums in the same order, so logits,
    tokens and cache rows are identical; both against the checker once."""
    from paper_2407_12021_b200 import binding as B
    shape = gen.ModelShape("bf16-4x128", 2, 512, 4, 128, 1408, 1024, "bf16")
    w = gen.model_weights(shape, 91)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    tokens, parents = gen.make_tree(100, 7, 4, shape.vocab, 92)
    prompt = gen.zipf_tokens(150, shape.vocab, 93, 50).tolist()
    results = []
    for which in (0, 1):
        sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=512)
        B.aded_debug_weight_layout(sess.model, which)
        sess.append(prompt)
        gpu = sess.verify(tokens, parents)
        assert gpu["status"] == 0
        k, v = sess.read_kv(1, 0, sess.length())
        results.append((gpu, k, v))
    (g0, k0, v0), (g1, k1, v1) = results
    assert np.array_equal(g0["logits"], g1["logits"]) and g0["out_tokens"] == g1["out_tokens"]
    assert np.array_equal(k0, k1) and np.array_equal(v0, v1)
    cache = ov.Cache(arch)
    ov.append(arch, ow, cache, prompt)
    cpu = ov.verify(arch, ow, cache, tokens, parents)
    H.compare_step(shape, g0, cpu, tokens, parents, "re-tiled weights")


@pytest.mark.parametrize("nodes", [40, 100])
def test_attention_reference_moves_within_a_split(cuda_device, nodes):
    """Keys whose magnitude grows with the position: every 64-key block's largest score exceeds the previous
    block's by far more than the slack the tensor-core kernel allows its integer reference, so the rare path that
    rescales the running output in tensor memory runs in every block.  Same answer as the checker (whose reference
    is the row's overall maximum: scaling by a power of two commutes with the bf16 rounding of the numerators)."""
    shape = gen.ModelShape("bf16-4x128", 1, 512, 4, 128, 3 * 128, 1024, "bf16")      # one layer: q is the same on both sides
    w = gen.model_weights(shape, 77)
    for p in w["layers"]:
        for k in ("wqkv", "wo", "wgu", "wd"):
            p[k] = (p[k].float() * 3).to(torch.bfloat16)
    ctx = 2000
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=ctx + 256)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    cache = ov.Cache(arch)
    ramp = (1.0 + torch.arange(ctx, dtype=torch.float32) / 20.0).view(1, ctx, 1)
    for l in range(shape.n_layers):
        k, v = gen.kv_normal(shape, ctx, 78, l)
        k = (k.float() * ramp).to(torch.bfloat16)
        sess.B.aded_kv_load(sess.kv, 0, l, k.to(cuda_device), v.to(cuda_device))
        cache.load(l, k, v)
    tokens, parents = gen.make_tree(nodes, 6, 4, shape.vocab, 79)
    # the scores do climb: per head, the best key of the last quarter beats the best of the first by more than 2^8
    trace = {}
    ov.forward_tree(arch, ow, cache, tokens, parents, want_logits=False, trace=trace)
    q = np.asarray(trace["q"]).reshape(nodes, shape.n_heads, shape.head_dim)
    kl = np.asarray(cache.k[shape.n_layers - 1], dtype=np.float64)          # [H, L, hd]
    sc = np.einsum("thd,hld->thl", q, kl[:, :ctx]) * (1.4426950408889634 / np.sqrt(shape.head_dim))
    assert np.all(sc[:, :, 3 * ctx // 4:].max(axis=2) - sc[:, :, :ctx // 4].max(axis=2) > 8.0)
    cpu = ov.verify(arch, ow, cache, tokens, parents)
    gpu = sess.verify(tokens, parents)
    assert gpu["status"] == 0
    H.compare_step(shape, gpu, cpu, tokens, parents, f"climbing keys, {nodes} nodes")
    att = sess.B.aded_debug_read_buffer(sess.model, 3, nodes).double().cpu().numpy()
    ref = np.asarray(trace["attn"], dtype=np.float64).reshape(att.shape)
    assert np.abs(att - ref).max() <= 2e-2 * np.abs(ref).max()


@pytest.mark.parametrize("heads,hd,nodes,depth,ctx", [(4, 64, 128, 8, 100), (2, 128, 37, 5, 191), (2, 128, 128, 8, 70),
                                                     (4, 64, 16, 3, 64), (2, 128, 1, 0, 129)])
def test_bf16_small_models_tree_shapes(cuda_device, heads, hd, nodes, depth, ctx):
    """bf16 path (tensor-core GEMM + split-KV attention) on small models: both head sizes, trees of
    1..128 nodes, contexts that are not multiples of the key block, prefill through append."""
    d = heads * hd
    shape = gen.ModelShape(f"bf16-{heads}x{hd}", 2, d, heads, hd, 3 * 128, 1024, "bf16")
    w = gen.model_weights(shape, 60 + nodes)
    for p in w["layers"]:                       # livelier activations than N(0, 0.02) gives at this width
        for k in ("wqkv", "wo", "wgu", "wd"):
            p[k] = (p[k].float() * 3).to(torch.bfloat16)
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=ctx + 300)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    prompt = gen.zipf_tokens(ctx + 1, shape.vocab, 61, 50).tolist()
    cache = ov.Cache(arch)
    ov.append(arch, ow, cache, prompt[:-1])
    sess.append(prompt[:-1])
    assert sess.length() == ctx
    H.compare_cache(shape, sess, cache, 0, ctx, range(shape.n_layers), "prefill")
    root = prompt[-1]
    for step in range(2):
        tokens, parents = gen.make_tree(nodes, depth, 6, shape.vocab, 62 + step, root_token=root)
        if step == 1 and nodes > 2:   # second step: plant one correct draft so that something is accepted
            probe = ov.verify(arch, ow, cache.clone(), [root], [-1])
            tokens = gen.plant_path(tokens, parents, probe["out_tokens"])
        cpu = ov.verify(arch, ow, cache, tokens, parents)
        gpu = sess.verify(tokens, parents)
        assert gpu["status"] == 0
        worst = H.compare_step(shape, gpu, cpu, tokens, parents, f"{shape.name} step {step}")
        if worst["flipped"]:
            return                # an exempt near-tie changed the path; the caches legitimately differ from here
        assert sess.length() == cache.length
        H.compare_cache(shape, sess, cache, ctx, cache.length - ctx, range(shape.n_layers), f"cache step {step}")
        root = gpu["out_tokens"][-1]


@pytest.mark.parametrize("which", [0, 1])
def test_bounded_wait_runs_out_and_the_handle_recovers(cuda_device, which):
    """Every device-side wait of the library is bounded and ends in a status code, not a hang.  The probe makes
    one such wait run out for real -- an mbarrier nobody arrives at (which = 0), an arrival counter nobody
    raises (1) -- with a limit of about a millisecond.  Expected: the kernel returns, the model reports
    ADED_ERR_TIMEOUT, a step submitted while the error is pending does nothing (accept length 0, cache
    untouched), and after the status has been read the handle works as before."""
    import time
    shape = gen.ModelShape("bf16-4x128", 2, 512, 4, 128, 1024, 1024, "bf16")
    w = H.weights_to(gen.model_weights(shape, 91), cuda_device)
    sess = H.GpuSession(shape, w, capacity=512)
    prompt = gen.zipf_tokens(70, shape.vocab, 91, 50).tolist()
    sess.append(prompt[:-1])
    tokens, parents = gen.make_tree(24, 4, 4, shape.vocab, 92, root_token=prompt[-1])
    good = sess.verify(tokens, parents, capture=False)
    assert good["status"] == 0 and good["accept_len"] >= 1
    sess.B.aded_kv_set_len(sess.kv, 0, 69)
    t0 = time.perf_counter()
    sess.B.aded_debug_wait_timeout(sess.model, which, 2_000_000)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0, "the wait did not end at its limit"
    pending = sess.verify(tokens, parents, capture=False)          # reads (and clears) the status after the call
    assert pending["status"] == 8 and pending["accept_len"] == 0 and sess.length() == 69
    assert sess.B.aded_model_poll_status(sess.model) == 0
    again = sess.verify(tokens, parents, capture=False)
    assert again["status"] == 0 and again["out_tokens"] == good["out_tokens"] and sess.length() == 69 + good["accept_len"]


def test_debug_build_runs_the_small_workloads_without_an_index_complaint(cuda_device):
    """The debug build (-DADED_DEBUG_CHECKS: index checks on slot, cache-row and bucket addressing that report
    ADED_ERR_INTERNAL through the status word; the stand-in for a memory checker) runs the fp32 workload, a
    bf16 tensor-core step and a tri-gram round trip -- each compared with the checker -- and no check fires."""
    import os
    import subprocess
    import sys
    from paper_2407_12021_b200 import build
    lib = build.build(debug=True)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, ADED_LIBRARY=lib)
    code = ("import __graft_entry__ as g, os; from paper_2407_12021_b200 import binding as B; "
            "assert B._LIB_PATH == os.environ['ADED_LIBRARY']; g.smoke()")
    res = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-2000:]
    assert "smoke ok" in res.stdout
