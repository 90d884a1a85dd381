"""GPU parity on the larger workloads: the full 32-layer 7B-shaped decode (sampled steps,
teacher-forced from the GPU's own cache), the 13B-shaped layer stack with 128-node trees, and the
ragged batches.  The CPU checker is slow, so these compare sampled steps / reduced depth; the small
workloads in test_gpu_verify.py compare everything."""
import numpy as np
import pytest
import torch

from oracle import verify as ov
from oracle.trigram import TrigramStore
from paper_2407_12021_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _oracle_cache_from_gpu(sess, arch, n_pos):
    """Teacher forcing: the checker starts from the cache contents the GPU holds."""
    cache = ov.Cache(arch)
    for l in range(arch.n_layers):
        k, v = sess.B.aded_kv_read(sess.kv, 0, l, 0, n_pos)
        cache.load(l, k, v)
    return cache


def test_c3_full_7b_decode_sampled_step(cuda_device):
    """Workload 3 at full size: 32 layers, 2048-token Zipf prompt, 64-node trees built from the GPU
    tri-gram top-4 lists, table updated every step.  Tri-gram results are compared at every lookup.
    The verification is compared at one sampled step, teacher-forced layer by layer: a random-init
    bf16 network amplifies one-ulp differences (a 1 % disagreement in attention outputs becomes a 50 %
    disagreement in SwiGLU outputs one layer on), so end-to-end logits drift apart with depth whatever
    the implementation; instead every checked layer is re-run by the checker from the hidden states and
    cache the device actually had, and the LM head from the device's final hidden states."""
    from paper_2407_12021_b200 import binding as B
    wl = gen.WORKLOADS["c3"]
    shape = wl.shape
    w = gen.model_weights(shape, 301, device=cuda_device)
    sess = H.GpuSession(shape, w, capacity=2048 + 64 * 12)
    prompt = gen.zipf_tokens(2048, shape.vocab, 301, 50)
    sess.append(prompt[:-1].tolist())
    assert sess.length() == 2047
    tg = B.aded_trigram_create(shape.vocab, log2_buckets=16, overflow_buckets=4096)
    B.aded_trigram_update(tg, prompt.to(cuda_device))
    st = TrigramStore()
    st.update(prompt.tolist())
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w)
    prev_tok, root_tok = int(prompt[-2]), int(prompt[-1])
    sampled = 2
    for step in range(4):
        def topk_gpu(a, b):
            ctx = torch.tensor([[a, b]], dtype=torch.int32, device=cuda_device)
            tok = torch.empty((1, 4), dtype=torch.int32, device=cuda_device)
            cnt = torch.empty((1, 4), dtype=torch.int32, device=cuda_device)
            B.aded_trigram_topk(tg, ctx, 4, tok, cnt)
            got = (tok[0].tolist(), cnt[0].tolist())
            assert got == st.topk(a, b, 4)            # bit-exact lists, every lookup of every step
            return got[0]
        tokens, parents, _ = gen.expand_tree_from_topk(prev_tok, root_tok, topk_gpu, 64, 6, shape.vocab, 400 + step)
        L = sess.length()
        if step == sampled:
            check_layers = [0, 1, 15, 31]
            before = {l: B.aded_kv_read(sess.kv, 0, l, 0, L) for l in check_layers}   # the cache the step starts from
            hidden = torch.empty((shape.n_layers + 1, 64, shape.d_model), dtype=torch.bfloat16, device=cuda_device)
            B.aded_debug_capture_hidden(sess.model, hidden)
        gpu = sess.verify(tokens, parents, capture=(step == sampled))
        assert gpu["status"] == 0 and gpu["accept_len"] >= 1
        if step == sampled:
            paths, depth = ov.paths_and_depths(parents)
            pos = L + np.asarray(depth)
            hid = hidden.double().cpu().numpy()
            emb = ow.embed_rows(tokens)
            assert np.array_equal(hid[0], emb)                       # embedding rows are copies
            for l in check_layers:
                kc, vc = (t.double().cpu().numpy() for t in before[l])
                h_out, k, v = ov.decoder_layer(arch, ow.layer(l), kc, vc, hid[l], paths, pos)
                err = np.abs(h_out - hid[l + 1])
                rel_max = err.max() / np.abs(h_out).max()
                rel_rms = np.sqrt((err ** 2).mean() / (h_out ** 2).mean())
                print(f"c3 layer {l}: max {rel_max:.3e} rms {rel_rms:.3e} differing {np.mean(err > 0):.3f}")
                assert rel_max <= 2e-2 and rel_rms <= 1e-2, (l, rel_max, rel_rms)
            # LM head and greedy choice from the device's own final hidden states
            lc = ov.lm_head(arch, ow, hid[shape.n_layers])
            step_cpu = {"logits": lc, "best": ov.greedy(lc)}
            step_cpu["out_tokens"] = ov.accept_walk(tokens, parents, step_cpu["best"])[1]
            step_cpu["accept_len"] = len(step_cpu["out_tokens"])
            worst = H.compare_step(shape, gpu, step_cpu, tokens, parents, "c3 LM head")
            print("c3 LM head from device hidden states:", worst)
            assert worst["logit_rel"] <= 2e-3 and worst["flipped_beyond_1e-2"] == 0
            # end to end (all 32 layers in the checker, from the device's cache): reported, loosely bounded
            cache = ov.Cache(arch)
            for l in range(shape.n_layers):
                kk, vv = (before[l] if l in before else B.aded_kv_read(sess.kv, 0, l, 0, L))
                cache.load(l, kk, vv)
            full = ov.verify(arch, ow, cache, tokens, parents)
            rel = np.max(np.abs(gpu["logits"] - full["logits"]), axis=1) / np.max(np.abs(full["logits"]), axis=1)
            print(f"c3 end-to-end logit deviation over 32 layers: max {rel.max():.3e} median {np.median(rel):.3e}; "
                  f"greedy tokens equal on {int(np.sum(gpu['best'] == full['best']))}/64 nodes")
            assert rel.max() < 0.15
        span = [prev_tok, root_tok] + gpu["out_tokens"]
        st.update(span)
        B.aded_trigram_update(tg, H.i32(span))
        chain = [root_tok] + gpu["out_tokens"]
        prev_tok, root_tok = chain[-2], chain[-1]
    torch.cuda.synchronize()
    assert B.aded_trigram_poll_status(tg) == 0
    assert B.aded_trigram_stats(tg)[0] == len(st.entries())


def test_c4_13b_shape_128_node_tree(cuda_device):
    """Workload 4's shape at reduced depth: 13B widths (d 5120, 40 heads, FFN 13824), 3 layers, cache
    pre-filled with 4096 positions, 128-node depth-8 tree with branching <= 6."""
    shape = gen.LLAMA13B.with_layers(3)
    w = gen.model_weights(shape, 311, device=cuda_device)
    sess = H.GpuSession(shape, w, capacity=4096 + 256)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w)
    cache = ov.Cache(arch)
    for l in range(shape.n_layers):
        k, v = gen.kv_normal(shape, 4096, 311, l, device=cuda_device)
        sess.B.aded_kv_load(sess.kv, 0, l, k, v)
        cache.load(l, k, v)
    tokens, parents = gen.make_tree(128, 8, 6, shape.vocab, 312)
    cpu = ov.verify(arch, ow, cache, tokens, parents)
    gpu = sess.verify(tokens, parents)
    assert gpu["status"] == 0
    worst = H.compare_step(shape, gpu, cpu, tokens, parents, "c4")
    print("c4:", worst)
    if worst["flipped"] == 0:
        H.compare_cache(shape, sess, cache, 4096, cpu["accept_len"], range(shape.n_layers), "c4 cache")


@pytest.mark.parametrize("batch", [1, 4, 16])
def test_c5_ragged_batches(cuda_device, batch):
    """Workload 5: 7B widths (one layer), ragged batch: contexts U[512, 8192], trees of 32..128 nodes
    with depth 3..8, all sequences verified in one call; sequences against the checker."""
    from paper_2407_12021_b200 import binding as B
    shape = gen.LLAMA7B_1L
    w = gen.model_weights(shape, 321, device=cuda_device)
    ctx_len = [512 + v for v in gen.randint(batch, 8192 - 512 + 1, 321 + batch, 1)]
    n_nodes = [32 + v for v in gen.randint(batch, 128 - 32 + 1, 321 + batch, 2)]
    depth = [3 + v for v in gen.randint(batch, 6, 321 + batch, 3)]
    ctx_len[0], n_nodes[0] = 8192, 128                     # the extremes are always present
    if batch > 1:
        ctx_len[1], n_nodes[1], depth[1] = 512, 32, 3
    rows = sum(n_nodes)
    model = B.aded_model_create(shape, w, max_rows=rows, max_batch=batch)
    kv = B.aded_kv_create(model, [c + 128 for c in ctx_len])
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    caches, trees = [], []
    for b in range(batch):
        k, v = gen.kv_normal(shape, ctx_len[b], 330 + b, 0, device=cuda_device)
        B.aded_kv_load(kv, b, 0, k, v)
        c = ov.Cache(arch)
        c.load(0, k, v)
        caches.append(c)
        trees.append(gen.make_tree(n_nodes[b], depth[b], 6, shape.vocab, 340 + b))
    offsets = [0]
    for b in range(batch):
        offsets.append(offsets[-1] + n_nodes[b])
    tok = H.i32([t for tr in trees for t in tr[0]])
    par = H.i32([p for tr in trees for p in tr[1]])
    out = torch.full((batch, 128), -7, dtype=torch.int32, device=cuda_device)
    out_len = torch.full((batch,), -7, dtype=torch.int32, device=cuda_device)
    logits = torch.empty((rows, shape.vocab), dtype=torch.float32, device=cuda_device)
    best = torch.empty((rows,), dtype=torch.int32, device=cuda_device)
    B.aded_debug_capture(model, logits, best)
    B.aded_verify_batch(model, kv, offsets, tok, par, out, out_len)
    torch.cuda.synchronize()
    assert B.aded_model_poll_status(model) == 0
    # a second, graph-replayed call on rolled-back caches must give the same answer
    for b in range(batch):
        B.aded_kv_set_len(kv, b, ctx_len[b])
    out2 = torch.full((batch, 128), -7, dtype=torch.int32, device=cuda_device)
    len2 = torch.full((batch,), -7, dtype=torch.int32, device=cuda_device)
    B.aded_verify_batch(model, kv, offsets, tok, par, out2, len2)
    torch.cuda.synchronize()
    assert torch.equal(out_len, len2)
    lg = logits.cpu().double().numpy()
    bs = best.cpu().numpy().astype(np.int64)
    check = range(batch) if batch <= 4 else [0, 1, 5, 11]      # the checker is slow: sample the big batch
    for b in check:
        cpu = ov.verify(arch, ow, caches[b], trees[b][0], trees[b][1])
        a = int(out_len[b])
        gpu = {"logits": lg[offsets[b]:offsets[b + 1]], "best": bs[offsets[b]:offsets[b + 1]],
               "out_tokens": out[b, :a].tolist(), "accept_len": a}
        assert out2[b, :a].tolist() == gpu["out_tokens"]
        worst = H.compare_step(shape, gpu, cpu, trees[b][0], trees[b][1], f"c5 batch {batch} seq {b}")
        print(f"c5 batch {batch} seq {b}:", worst)
        assert B.aded_kv_len(kv, b) == ctx_len[b] + a
    for b in range(batch):                                      # every sequence: the walk over its own choices
        a = int(out_len[b])
        _, walk = ov.accept_walk(trees[b][0], trees[b][1], bs[offsets[b]:offsets[b + 1]])
        assert out[b, :a].tolist() == walk and out[b, a:].tolist() == [-7] * (128 - a)
