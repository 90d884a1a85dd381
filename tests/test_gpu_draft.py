"""GPU parity of draft-tree retrieval and of the device-resident decoding step against the CPU
checker: trees, emitted tokens, contexts and table contents bit-exact."""
import pytest
import torch

from oracle import draft as od
from oracle import verify as ov
from oracle.trigram import TrigramStore
from paper_2407_12021_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _tree_gpu(B, t, prev, root, n_nodes, max_depth, k, filler=None):
    ctx = H.i32([prev, root])
    tok = torch.full((n_nodes,), -9, dtype=torch.int32, device="cuda")
    par = torch.full((n_nodes,), -9, dtype=torch.int32, device="cuda")
    real = torch.full((1,), -9, dtype=torch.int32, device="cuda")
    B.aded_draft_tree(t, ctx, n_nodes, max_depth, k, None if filler is None else H.i32(filler), tok, par, real)
    torch.cuda.synchronize()
    return tok.tolist(), par.tolist(), int(real[0])


@pytest.mark.parametrize("vocab,corpus,seed", [(12, 600, 1), (50, 3000, 2), (4096, 10000, 3)])
def test_draft_tree_matches_checker(cuda_device, vocab, corpus, seed):
    from paper_2407_12021_b200 import binding as B
    toks = gen.zipf_tokens(corpus, vocab, seed, 1)
    st = TrigramStore()
    st.update(toks.tolist())
    t = B.aded_trigram_create(vocab, log2_buckets=14, overflow_buckets=4096)
    B.aded_trigram_update(t, toks.cuda())
    text = toks.tolist()
    starts = [(text[i], text[i + 1]) for i in range(0, 400, 37)] + [(vocab - 1, vocab - 1)]
    shapes = [(64, 6, 4), (24, 3, 3), (128, 4, 8), (7, 5, 2), (1, 3, 4), (16, 0, 4), (128, 12, 1)]
    filler = gen.zipf_tokens(4 * 128, vocab, seed, 9).tolist()
    for (prev, root) in starts:
        for (n_nodes, max_depth, k) in shapes:
            want = od.draft_tree(st, prev, root, n_nodes, max_depth, k)
            got = _tree_gpu(B, t, prev, root, n_nodes, max_depth, k)
            pad = n_nodes - want[2]
            assert got == (want[0] + [-1] * pad, want[1] + [-1] * pad, want[2]), (prev, root, n_nodes, max_depth, k)
            try:
                want = od.draft_tree(st, prev, root, n_nodes, max_depth, k, filler=filler[:4 * n_nodes])
            except ValueError:
                want = None
            got = _tree_gpu(B, t, prev, root, n_nodes, max_depth, k, filler=filler[:4 * n_nodes])
            if want is None:      # no room (depth 0, or a chain that is full): reported, root marked invalid
                assert got[0][0] == -1 and B.aded_trigram_poll_status(t) == 1
            else:
                assert got == want, (prev, root, n_nodes, max_depth, k)
    assert B.aded_trigram_poll_status(t) == 0


def test_filler_edge_cases(cuda_device):
    from paper_2407_12021_b200 import binding as B
    t = B.aded_trigram_create(64, log2_buckets=8, overflow_buckets=64)
    empty = TrigramStore()
    assert _tree_gpu(B, t, 0, 1, 6, 2, 2, [5, 5, 6, 7, 8, 9, 10]) == od.draft_tree(empty, 0, 1, 6, 2, 2, [5, 5, 6, 7, 8, 9, 10])
    assert _tree_gpu(B, t, 0, 1, 4, 1, 3, [5, 5, 5, 6, 7]) == ([1, 5, 6, 7], [-1, 0, 0, 0], 1)
    assert B.aded_trigram_poll_status(t) == 0
    # the filler runs out / a token outside the vocabulary / no node has room: reported, tree marked invalid
    for args in ((4, 1, 3, [5, 5, 5, 6]), (4, 1, 3, [5, 64, 6, 7]), (6, 1, 2, list(range(10, 40)))):
        tok, par, real = _tree_gpu(B, t, 0, 1, *args)
        assert tok[0] == -1 and real == 1
        assert B.aded_trigram_poll_status(t) == 1
    # host-side argument checks
    from paper_2407_12021_b200.binding import AdedError
    for bad in ((0, 2, 2), (129, 2, 2), (8, -1, 2), (8, 2, 0), (8, 2, 9)):
        with pytest.raises(AdedError):
            _tree_gpu(B, t, 0, 1, *bad)


def _decode_setup(cuda_device, seed):
    shape = gen.TINY
    w = gen.model_weights(shape, seed)
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=512)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    prompt = gen.zipf_tokens(64, shape.vocab, seed, 50).tolist()
    cache = ov.Cache(arch)
    ov.append(arch, ow, cache, prompt[:-1])
    sess.append(prompt[:-1])
    # the checker's own continuation: a table that has seen it proposes drafts the model accepts
    probe = cache.clone()
    cur, ar = prompt[-1], []
    for _ in range(40):
        cur = ov.verify(arch, ow, probe, [cur], [-1])["out_tokens"][0]
        ar.append(cur)
    return shape, arch, ow, cache, sess, prompt, ar


@pytest.mark.parametrize("host", [False, True])
def test_decode_steps_match_checker(cuda_device, host):
    """Ten steps of draft -> verify -> table update -> next context, device-resident, against the same
    loop built from the checker's parts."""
    from paper_2407_12021_b200 import binding as B
    shape, arch, ow, cache, sess, prompt, ar = _decode_setup(cuda_device, seed=31)
    n_nodes, max_depth, k = 16, 4, 3
    seen_text = prompt + ar[:25]              # the table knows the first 25 tokens of the continuation
    st = TrigramStore()
    st.update(seen_text)
    t = B.aded_trigram_create(shape.vocab, log2_buckets=12, overflow_buckets=1024)
    B.aded_trigram_update(t, H.i32(seen_text))
    ctx = H.i32(prompt[-2:])
    prev, root = prompt[-2], prompt[-1]
    out = torch.full((n_nodes,), -7, dtype=torch.int32, device="cuda")
    alen = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    real = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    out_h = torch.full((n_nodes,), -7, dtype=torch.int32).pin_memory()
    alen_h = torch.full((1,), -7, dtype=torch.int32).pin_memory()
    emitted, lens = [], []
    for step in range(10):
        filler = gen.zipf_tokens(4 * n_nodes, shape.vocab, 31, 1000 + step).tolist()
        tokens, parents, from_table = od.draft_tree(st, prev, root, n_nodes, max_depth, k, filler=filler)
        cpu = ov.verify(arch, ow, cache, tokens, parents)
        st.update([prev, root] + cpu["out_tokens"])
        prev, root = od.decode_context(prev, root, cpu["out_tokens"])
        if host:
            B.aded_decode_step_host(sess.model, sess.kv, t, ctx, n_nodes, max_depth, k,
                                    torch.tensor(filler, dtype=torch.int32).pin_memory(), out_h, alen_h)
            a, got = int(alen_h[0]), out_h.tolist()
        else:
            B.aded_decode_step(sess.model, sess.kv, t, ctx, n_nodes, max_depth, k, H.i32(filler), out, alen, real)
            torch.cuda.synchronize()
            a, got = int(alen[0]), out.tolist()
            assert int(real[0]) == from_table
        assert B.aded_model_poll_status(sess.model) == 0 and B.aded_trigram_poll_status(t) == 0
        assert a == cpu["accept_len"] and got[:a] == cpu["out_tokens"], f"step {step}"
        assert ctx.tolist() == [prev, root]
        assert sess.length() == cache.length
        emitted += got[:a]
        lens.append(a)
    m = min(len(emitted), len(ar))
    assert emitted[:m] == ar[:m]                  # greedy speculative decoding emits the autoregressive text
    assert max(lens) >= 3                         # drafts were accepted where the table knew the text
    # the table learned the emitted text: every stored tri-gram of the checker, bit-exact
    for (a_, b_, c_), n in st.entries().items():
        assert B.aded_trigram_get(t, a_, b_, c_) == n
    assert B.aded_trigram_stats(t)[0] == len(st.entries())


def test_failed_step_changes_nothing(cuda_device):
    from paper_2407_12021_b200 import binding as B
    shape, arch, ow, cache, sess, prompt, ar = _decode_setup(cuda_device, seed=32)
    t = B.aded_trigram_create(shape.vocab, log2_buckets=10, overflow_buckets=64)
    B.aded_trigram_update(t, H.i32(prompt))
    before = B.aded_trigram_stats(t)
    ctx = H.i32(prompt[-2:])
    out = torch.full((16,), -7, dtype=torch.int32, device="cuda")
    alen = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    B.aded_decode_step(sess.model, sess.kv, t, ctx, 16, 4, 3, H.i32([5]), out, alen)     # filler too short
    torch.cuda.synchronize()
    assert int(alen[0]) == 0 and ctx.tolist() == prompt[-2:] and sess.length() == 63
    assert B.aded_trigram_poll_status(t) == 1 and B.aded_model_poll_status(sess.model) != 0
    assert B.aded_trigram_stats(t) == before
    # and the next step works
    filler = gen.zipf_tokens(64, shape.vocab, 32, 7).tolist()
    B.aded_decode_step(sess.model, sess.kv, t, ctx, 16, 4, 3, H.i32(filler), out, alen)
    torch.cuda.synchronize()
    assert int(alen[0]) >= 1 and B.aded_model_poll_status(sess.model) == 0 and sess.length() == 63 + int(alen[0])
