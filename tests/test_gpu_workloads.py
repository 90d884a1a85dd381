"""GPU parity on the larger workloads at their own sizes: the full 32-layer 7B-shaped decode (three sampled
steps, one with approved drafts), the full 40-layer 13B-shaped step over a 128-node tree, a ragged batch
at full depth, and the one-layer ragged batches end to end.  The CPU checker is slow, so the full-depth
cases compare sampled layers teacher-forced from the device's own hidden states and cache plus the LM
head; the small workloads in test_gpu_verify.py compare everything end to end."""
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


def _ar_probe(sess, root_tok: int, n: int):
    """The model's own next n tokens after the committed text + root, by plain one-token-per-pass decoding
    on the device; the cache is rolled back afterwards."""
    L = sess.length()
    cur, out = root_tok, []
    for _ in range(n):
        res = sess.verify([cur], [-1], capture=False)
        assert res["status"] == 0 and res["accept_len"] == 1
        cur = res["out_tokens"][0]
        out.append(cur)
    sess.B.aded_kv_set_len(sess.kv, 0, L)
    return out


def test_c3_full_7b_decode_sampled_steps(cuda_device):
    """Workload 3 at full size: 32 layers, 2048-token Zipf prompt, 64-node trees built from the GPU
    tri-gram top-4 lists, table updated every step.  Tri-gram results are compared at every lookup.
    Three of five steps are compared with the checker, teacher-forced layer by layer (a random-init bf16
    network amplifies one-ulp differences -- a 1 % disagreement in attention outputs becomes a 50 %
    disagreement in SwiGLU outputs one layer on -- so every checked layer is re-run from the hidden states
    and cache the device actually had, and the LM head from the device's final hidden states, where the
    fixed token rule is asserted).  The second sampled step carries a planted path (the model's own next
    tokens, found by one-token decoding on the device) so that drafts are approved and their cache rows
    compacted; the compacted rows are compared with the checker's keys/values of the approved nodes, and
    the third sampled step starts from that cache."""
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
    check_layers = [0, 1, 15, 31]
    sampled, planted_step, end_to_end_step = (1, 2, 3), 2, 1
    for step in range(5):
        def topk_gpu(a, b):
            ctx = torch.tensor([[a, b]], dtype=torch.int32, device=cuda_device)
            tok = torch.empty((1, 4), dtype=torch.int32, device=cuda_device)
            cnt = torch.empty((1, 4), dtype=torch.int32, device=cuda_device)
            B.aded_trigram_topk(tg, ctx, 4, tok, cnt)
            got = (tok[0].tolist(), cnt[0].tolist())
            assert got == st.topk(a, b, 4)            # bit-exact lists, every lookup of every step
            return got[0]
        tokens, parents, _ = gen.expand_tree_from_topk(prev_tok, root_tok, topk_gpu, 64, 6, shape.vocab, 400 + step)
        probe = None
        if step == planted_step:
            # a seeded tree whose nodes 1, 2, ... form a chain, with the model's next two tokens on it
            probe = _ar_probe(sess, root_tok, 3)
            tokens, parents = gen.make_tree(64, 6, 4, shape.vocab, 400 + step, root_token=root_tok)
            tokens = gen.plant_path(tokens, parents, probe[:2])
            assert tokens[1:3] == probe[:2] and parents[1:3] == [0, 1]
        L = sess.length()
        if step in sampled:
            before = {l: B.aded_kv_read(sess.kv, 0, l, 0, L) for l in check_layers}   # the cache the step starts from
            hidden = torch.empty((shape.n_layers + 1, 64, shape.d_model), dtype=torch.bfloat16, device=cuda_device)
            B.aded_debug_capture_hidden(sess.model, hidden)
        gpu = sess.verify(tokens, parents, capture=(step in sampled))
        assert gpu["status"] == 0 and gpu["accept_len"] >= 1
        if step in sampled:
            cache_before = {l: tuple(t.double().cpu().numpy() for t in before[l]) for l in check_layers}
            res = H.layerwise_check(arch, ow, tokens, parents, L, hidden.double().cpu().numpy(), cache_before, gpu,
                                    f"c3 step {step}", shape)
            assert res["head"]["flipped_beyond_1e-2"] == 0
            if step == planted_step:
                # the planted drafts are the model's own continuation: approved unless a near-tie moved a token
                margin = ov.top2_margin(res["cpu"]["logits"])
                if all(margin[i] >= H.MARGIN_EXEMPT for i in (0, 1, 2)):
                    assert gpu["out_tokens"][:3] == probe, (gpu["out_tokens"], probe)
                    assert gpu["accept_len"] >= 3
                # compaction at full depth: rows L .. L + accept_len - 1 hold the approved nodes' keys/values
                path, _ = ov.accept_walk(tokens, parents, gpu["best"])
                a = gpu["accept_len"]
                assert len(path) == a and sess.length() == L + a
                for l in check_layers:
                    kg, vg = sess.read_kv(l, L, a)
                    k_new, v_new = res["kv_new"][l]
                    for name, got, want in (("K", kg, k_new[path].transpose(1, 0, 2)), ("V", vg, v_new[path].transpose(1, 0, 2))):
                        err = np.max(np.abs(got - want)) / np.max(np.abs(want))
                        assert err <= 2e-2, f"c3 compaction layer {l} {name}: {err:.3e}"
            if step == end_to_end_step:
                # end to end (all 32 layers in the checker, from the device's cache): reported; the logit
                # tolerance of 2e-2 is NOT met at this depth (see the docstring), only loosely bounded
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


def test_c4_full_13b_128_node_tree(cuda_device):
    """Workload 4 at full size: 40 layers of the 13B widths (d 5120, 40 heads, FFN 13824), a 4096-token
    context put in through chained appends, one verification step over a 128-node depth-8 tree with
    branching <= 6, compared teacher-forced on layers 0, 1, 20, 39 and at the LM head."""
    from paper_2407_12021_b200 import binding as B
    wl = gen.WORKLOADS["c4"]
    shape = wl.shape
    w = gen.model_weights(shape, 311, device=cuda_device)
    sess = H.GpuSession(shape, w, capacity=4096 + 256)
    prompt = gen.zipf_tokens(4096, shape.vocab, 311, 50)
    sess.append(prompt[:-1].tolist())
    L = sess.length()
    assert L == 4095 and B.aded_model_poll_status(sess.model) == 0
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w)
    tokens, parents = gen.make_tree(128, 8, 6, shape.vocab, 312, root_token=int(prompt[-1]))
    check_layers = [0, 1, 20, 39]
    before = {l: B.aded_kv_read(sess.kv, 0, l, 0, L) for l in check_layers}
    hidden = torch.empty((shape.n_layers + 1, 128, shape.d_model), dtype=torch.bfloat16, device=cuda_device)
    B.aded_debug_capture_hidden(sess.model, hidden)
    gpu = sess.verify(tokens, parents)
    assert gpu["status"] == 0 and gpu["accept_len"] >= 1
    cache_before = {l: tuple(t.double().cpu().numpy() for t in before[l]) for l in check_layers}
    res = H.layerwise_check(arch, ow, tokens, parents, L, hidden.double().cpu().numpy(), cache_before, gpu, "c4", shape)
    assert res["head"]["flipped_beyond_1e-2"] == 0
    assert sess.length() == L + gpu["accept_len"]


def test_c5_full_depth_batch4_one_sequence_layerwise(cuda_device):
    """Workload 5 at the model's full depth: 32 layers of the 7B widths, a ragged batch of 4 (contexts from
    U[512, 8192] with both extremes present, trees of 32..128 nodes), caches pre-filled with N(0,1) keys and
    values, all four sequences verified in one call; the second sequence's rows are compared teacher-forced
    on layers 0, 1, 15, 31 and at the LM head, and every sequence's emitted tokens against the walk over
    its own per-node choices."""
    from paper_2407_12021_b200 import binding as B
    shape = gen.LLAMA7B
    batch, seq = 4, 2
    w = gen.model_weights(shape, 351, device=cuda_device)
    ctx_len = [512 + v for v in gen.randint(batch, 8192 - 512 + 1, 351, 1)]
    n_nodes = [32 + v for v in gen.randint(batch, 128 - 32 + 1, 351, 2)]
    depth = [3 + v for v in gen.randint(batch, 6, 351, 3)]
    ctx_len[0], n_nodes[0] = 8192, 128
    ctx_len[1], n_nodes[1], depth[1] = 512, 32, 3
    rows = sum(n_nodes)
    model = B.aded_model_create(shape, w, max_rows=rows, max_batch=batch)
    kv = B.aded_kv_create(model, [c + 128 for c in ctx_len])
    check_layers = [0, 1, 15, 31]
    cache_before = {}
    for b in range(batch):
        for l in range(shape.n_layers):
            k, v = gen.kv_normal(shape, ctx_len[b], 360 + b, l, device=cuda_device)
            B.aded_kv_load(kv, b, l, k, v)
            if b == seq and l in check_layers:
                cache_before[l] = (k.double().cpu().numpy(), v.double().cpu().numpy())
    trees = [gen.make_tree(n_nodes[b], depth[b], 6, shape.vocab, 370 + b) for b in range(batch)]
    offsets = [0]
    for b in range(batch):
        offsets.append(offsets[-1] + n_nodes[b])
    tok = H.i32([t for tr in trees for t in tr[0]])
    par = H.i32([p for tr in trees for p in tr[1]])
    out = torch.full((batch, 128), -7, dtype=torch.int32, device=cuda_device)
    out_len = torch.full((batch,), -7, dtype=torch.int32, device=cuda_device)
    logits = torch.empty((rows, shape.vocab), dtype=torch.float32, device=cuda_device)
    best = torch.empty((rows,), dtype=torch.int32, device=cuda_device)
    hidden = torch.empty((shape.n_layers + 1, rows, shape.d_model), dtype=torch.bfloat16, device=cuda_device)
    B.aded_debug_capture(model, logits, best)
    B.aded_debug_capture_hidden(model, hidden)
    B.aded_verify_batch(model, kv, offsets, tok, par, out, out_len)
    torch.cuda.synchronize()
    assert B.aded_model_poll_status(model) == 0
    bs = best.cpu().numpy().astype(np.int64)
    for b in range(batch):
        a = int(out_len[b])
        _, walk = ov.accept_walk(trees[b][0], trees[b][1], bs[offsets[b]:offsets[b + 1]])
        assert out[b, :a].tolist() == walk and B.aded_kv_len(kv, b) == ctx_len[b] + a
    r0, r1 = offsets[seq], offsets[seq + 1]
    a = int(out_len[seq])
    gpu = {"logits": logits[r0:r1].cpu().double().numpy(), "best": bs[r0:r1], "out_tokens": out[seq, :a].tolist(), "accept_len": a}
    arch = ov.arch_from_shape(shape)
    res = H.layerwise_check(arch, ov.Weights(w), trees[seq][0], trees[seq][1], ctx_len[seq],
                            hidden[:, r0:r1].double().cpu().numpy(), cache_before, gpu, f"c5 batch 4 seq {seq}", shape)
    assert res["head"]["flipped_beyond_1e-2"] == 0


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
    # a second call on rolled-back caches must give the same answer (every sum runs in a fixed order)
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
