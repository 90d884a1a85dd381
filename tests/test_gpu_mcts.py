"""GPU parity of the draft maker's tree search against the CPU checker: prefix tree, ranked sentences
and their scores."""
import numpy as np
import pytest
import torch

from oracle import mcts as om
from oracle.trigram import TrigramStore
from paper_2407_12021_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _compare(B, t, st, prev, root, iters, length, n, k, u, c1=32.0, c2=8.0):
    want = om.mcts_draft(st, prev, root, iters, length, n, k, u.reshape(iters, length).tolist(), c1=c1, c2=c2)
    got = B.aded_mcts_draft(t, H.i32([prev, root]), iters, length, n, k, torch.tensor(u, dtype=torch.float32, device="cuda"), c1, c2)
    assert got[0] == want[0] and got[1] == want[1], (prev, root, iters, length, n, k)
    assert [s for s, _ in got[2]] == [s for s, _ in want[2]]
    assert [sc for _, sc in got[2]] == [sc for _, sc in want[2]]          # the same doubles, bit for bit
    return want


@pytest.mark.parametrize("vocab,corpus,seed", [(12, 800, 1), (60, 4000, 2), (4096, 20000, 3)])
def test_search_equals_the_checker(cuda_device, vocab, corpus, seed):
    from paper_2407_12021_b200 import binding as B
    toks = gen.zipf_tokens(corpus, vocab, seed, 1)
    text = toks.tolist()
    st = TrigramStore()
    st.update(text)
    t = B.aded_trigram_create(vocab, log2_buckets=15, overflow_buckets=8192)
    B.aded_trigram_update(t, toks.cuda())
    sizes = []
    for case, (iters, length, n, k) in enumerate([(150, 4, 24, 8), (40, 4, 24, 4), (160, 8, 12, 3), (25, 1, 24, 8), (7, 3, 5, 1)]):
        for start in (5, 123, 400):
            u = gen.uniform01(iters * length, seed, 100 + case).numpy().astype(np.float32)
            want = _compare(B, t, st, text[start], text[start + 1], iters, length, n, k, u)
            sizes.append(len(want[0]))
    assert max(sizes) > 8                              # real trees, not only roots
    # the other constant of the paper (Figures 4a, 5) as the float32 the C interface takes
    u = gen.uniform01(600, seed, 200).numpy().astype(np.float32)
    _compare(B, t, st, text[50], text[51], 150, 4, 24, 8, u, c1=float(np.float32(2.414)), c2=8.0)
    # unknown context: the root alone, no sentence
    assert B.aded_mcts_draft(t, H.i32([vocab - 1, vocab - 1]), 10, 4, 24, 4, torch.zeros(40, device="cuda")) == \
        om.mcts_draft(st, vocab - 1, vocab - 1, 10, 4, 24, 4, [[0.0] * 4] * 10)
    assert B.aded_trigram_poll_status(t) == 0


def test_hot_context_with_a_long_chain_and_bad_arguments(cuda_device):
    from paper_2407_12021_b200 import binding as B
    vocab = 400
    # context (1, 2) is followed by every token: its chain is longer than the kernel's in-memory list
    text = []
    for c in range(vocab):
        text += [1, 2, c] * (1 + c % 5)
    st = TrigramStore()
    st.update(text)
    t = B.aded_trigram_create(vocab, log2_buckets=12, overflow_buckets=4096)
    B.aded_trigram_update(t, H.i32(text))
    u = gen.uniform01(150 * 4, 9, 1).numpy().astype(np.float32)
    _compare(B, t, st, 1, 2, 150, 4, 24, 8, u)
    from paper_2407_12021_b200.binding import AdedError
    for bad in ((0, 4, 24, 8), (161, 4, 24, 8), (10, 0, 24, 8), (10, 9, 4, 8), (10, 4, 0, 8), (10, 4, 32, 8), (10, 4, 24, 9)):
        with pytest.raises(AdedError):
            B.aded_mcts_draft(t, H.i32([1, 2]), bad[0], bad[1], bad[2], bad[3], torch.zeros(2000, device="cuda"))


def test_drafts_feed_the_verification_step(cuda_device):
    """The merged prefix tree is a valid draft tree: the verification step of workload 1's model takes it
    and emits what the checker emits for the same tree."""
    from oracle import verify as ov
    from paper_2407_12021_b200 import binding as B
    shape = gen.TINY
    w = gen.model_weights(shape, 51)
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=256)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    prompt = gen.zipf_tokens(64, 40, 51, 50).tolist()          # a small alphabet, so that contexts repeat
    cache = ov.Cache(arch)
    ov.append(arch, ow, cache, prompt[:-1])
    sess.append(prompt[:-1])
    st = TrigramStore()
    st.update(prompt)
    t = B.aded_trigram_create(shape.vocab, log2_buckets=12, overflow_buckets=1024)
    B.aded_trigram_update(t, H.i32(prompt))
    u = gen.uniform01(600, 51, 7).numpy().astype(np.float32)
    # start from a context inside the prompt so that the table has continuations for it
    tok, par, sent = B.aded_mcts_draft(t, H.i32(prompt[20:22]), 150, 4, 24, 8, torch.tensor(u, device="cuda"))
    assert (tok, par) == om.mcts_draft(st, prompt[20], prompt[21], 150, 4, 24, 8, u.reshape(150, 4).tolist())[:2]
    assert len(tok) >= 3
    tok[0] = prompt[-1]                                        # the tree's root must be the last committed token
    cpu = ov.verify(arch, ow, cache, tok, par)
    gpu = sess.verify(tok, par)
    H.compare_step(shape, gpu, cpu, tok, par, "mcts tree")


def _mcts_tree_cpu(st, prev, root, n_nodes, iters, length, n, k, u, filler):
    from oracle import draft as od
    tok, par, _ = om.mcts_draft(st, prev, root, iters, length, n, k, u.reshape(iters, length).tolist())
    tok, par = tok[:n_nodes], par[:n_nodes]          # breadth-first numbering: a prefix is a tree
    return od.fill_tree(tok, par, n_nodes, length, k, filler)


def test_completed_tree_and_decode_steps(cuda_device):
    """The paper's loop on the device: tree search over the table -> prefix tree completed to a fixed
    shape -> verification -> the emitted tokens raise the table's counts -> next context."""
    from oracle import draft as od
    from oracle import verify as ov
    from paper_2407_12021_b200 import binding as B
    shape = gen.TINY
    w = gen.model_weights(shape, 61)
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=400)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    prompt = gen.zipf_tokens(96, 24, 61, 50).tolist()          # a small alphabet, so that contexts repeat
    cache = ov.Cache(arch)
    ov.append(arch, ow, cache, prompt[:-1])
    sess.append(prompt[:-1])
    st = TrigramStore()
    st.update(prompt)
    t = B.aded_trigram_create(shape.vocab, log2_buckets=12, overflow_buckets=1024)
    B.aded_trigram_update(t, H.i32(prompt))
    iters, length, n, k, n_nodes = 60, 4, 8, 4, 24
    # the completed tree alone, for a context the table knows
    u = gen.uniform01(iters * length, 61, 1).numpy().astype(np.float32)
    filler = gen.zipf_tokens(4 * n_nodes, shape.vocab, 61, 2).tolist()
    got = B.aded_mcts_draft(t, H.i32(prompt[30:32]), iters, length, n, k, torch.tensor(u, device="cuda"), n_nodes_target=n_nodes,
                            filler_dev=H.i32(filler))
    want = _mcts_tree_cpu(st, prompt[30], prompt[31], n_nodes, iters, length, n, k, u, filler)
    assert (got[0], got[1]) == want and len(got[0]) == n_nodes
    assert len(om.mcts_draft(st, prompt[30], prompt[31], iters, length, n, k, u.reshape(iters, length).tolist())[0]) > 3
    # decoding steps
    ctx = H.i32(prompt[-2:])
    prev, root = prompt[-2], prompt[-1]
    out = torch.full((n_nodes,), -7, dtype=torch.int32, device="cuda")
    alen = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    for step in range(5):
        u = gen.uniform01(iters * length, 61, 10 + step).numpy().astype(np.float32)
        filler = gen.zipf_tokens(4 * n_nodes, shape.vocab, 61, 20 + step).tolist()
        tokens, parents = _mcts_tree_cpu(st, prev, root, n_nodes, iters, length, n, k, u, filler)
        cpu = ov.verify(arch, ow, cache, tokens, parents)
        st.update([prev, root] + cpu["out_tokens"])
        prev, root = od.decode_context(prev, root, cpu["out_tokens"])
        B.aded_decode_step_mcts(sess.model, sess.kv, t, ctx, n_nodes, iters, length, n, k, torch.tensor(u, device="cuda"),
                                H.i32(filler), out, alen)
        torch.cuda.synchronize()
        assert B.aded_model_poll_status(sess.model) == 0 and B.aded_trigram_poll_status(t) == 0
        a = int(alen[0])
        assert a == cpu["accept_len"] and out[:a].tolist() == cpu["out_tokens"], f"step {step}"
        assert ctx.tolist() == [prev, root] and sess.length() == cache.length
    for (a_, b_, c_), cnt in st.entries().items():
        assert B.aded_trigram_get(t, a_, b_, c_) == cnt
