"""GPU parity of sampling-mode verification: the drawing rule bit-exact against the CPU checker on
seeded logits, and the verification step with sampled tokens against the checker's step."""
import numpy as np
import pytest
import torch

from oracle import sample as osmp
from oracle import verify as ov
from paper_2407_12021_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _draw_gpu(B, logits: np.ndarray, temp, top_p, u: np.ndarray):
    lg = torch.tensor(logits, dtype=torch.float32, device="cuda").contiguous()
    uu = torch.tensor(u, dtype=torch.float32, device="cuda")
    out = torch.full((logits.shape[0],), -5, dtype=torch.int32, device="cuda")
    B.aded_sample_tokens(lg, temp, top_p, uu, out)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.int64)


@pytest.mark.parametrize("vocab,rows", [(7, 64), (1000, 48), (4096, 32), (32000, 12), (32768, 4), (1, 3)])
def test_draws_equal_the_checker(cuda_device, vocab, rows):
    from paper_2407_12021_b200 import binding as B
    for case, (std, temp, top_p) in enumerate([(1.0, 1.0, 1.0), (2.0, 0.7, 0.9), (0.5, 2.0, 0.5), (3.0, 0.3, 0.95),
                                               (1.0, 1.0, 2.0 ** -16), (1.0, 0.05, 1.0)]):
        logits = gen.normal([rows, vocab], std, 70 + case, vocab).numpy().astype(np.float32)
        u = gen.uniform01(rows, 71 + case, vocab).numpy().astype(np.float32)
        got = _draw_gpu(B, logits, temp, top_p, u)
        want = osmp.sample_rows(logits, temp, top_p, u)
        assert np.array_equal(got, want), (vocab, case, np.nonzero(got != want)[0][:5])


def test_ties_extremes_and_bad_arguments(cuda_device):
    from paper_2407_12021_b200 import binding as B
    rows, vocab = 16, 3000
    u = gen.uniform01(rows, 80, 1).numpy().astype(np.float32)
    u[0], u[1] = 0.0, np.float32(1.0 - 2.0 ** -24)
    # many equal logits: the nucleus edge falls inside a run of ties, which enter in id order
    coarse = np.round(gen.normal([rows, vocab], 1.0, 81, 1).numpy() * 2) / 2
    flat = np.zeros((rows, vocab), dtype=np.float32)
    spread = gen.normal([rows, vocab], 30.0, 82, 1).numpy()            # most weights underflow to zero
    holes = gen.normal([rows, vocab], 1.0, 83, 1).numpy()
    holes[:, ::3] = -np.inf
    for logits in (coarse, flat, spread, holes):
        logits = logits.astype(np.float32)
        for temp, top_p in ((1.0, 0.9), (0.5, 0.3), (1.3, 1.0)):
            got = _draw_gpu(B, logits, temp, top_p, u)
            want = osmp.sample_rows(logits, temp, top_p, u)
            assert np.array_equal(got, want)
    from paper_2407_12021_b200.binding import AdedError
    lg = torch.zeros((2, 8), dtype=torch.float32, device="cuda")
    uu = torch.zeros(2, dtype=torch.float32, device="cuda")
    out = torch.zeros(2, dtype=torch.int32, device="cuda")
    for temp, top_p in ((0.0, 1.0), (-1.0, 1.0), (1.0, 0.0), (1.0, 1.5), (float("nan"), 1.0)):
        with pytest.raises(AdedError):
            B.aded_sample_tokens(lg, temp, top_p, uu, out)
    with pytest.raises(AdedError):
        B.aded_sample_tokens(torch.zeros((1, 40000), dtype=torch.float32, device="cuda"), 1.0, 1.0, uu, out)


def test_sampled_verification_steps(cuda_device):
    """Workload 1's model with sampled approval: per-node draws, emitted tokens and cache against the
    checker.  A low temperature keeps the draws away from the boundaries that a 1e-4 logit difference
    could move; a node whose draw changes when u moves by 2e-3 is exempt from the per-node comparison."""
    from paper_2407_12021_b200 import binding as B
    shape = gen.TINY
    w = gen.model_weights(shape, 21)
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=256)
    arch = ov.arch_from_shape(shape)
    ow = ov.Weights(w, keep=True)
    prompt = gen.zipf_tokens(64, shape.vocab, 21, 50).tolist()
    cache = ov.Cache(arch)
    ov.append(arch, ow, cache, prompt[:-1])
    sess.append(prompt[:-1])
    temp, top_p, n = 0.05, 0.9, 16
    root = prompt[-1]
    not_greedy = fragile = 0
    for step in range(6):
        tokens, parents = gen.make_tree(n, 4, 4, shape.vocab, 300 + step, root_token=root)
        u = gen.uniform01(n, 21, 400 + step).numpy().astype(np.float32)
        if step >= 2:      # plant the checker's own draws on the deep chain so that drafts get approved
            probe = ov.verify(arch, ow, cache.clone(), tokens, parents, choose=osmp.chooser(temp, top_p, u))
            tokens = gen.plant_path(tokens, parents, [int(probe["best"][0])])
        cpu = ov.verify(arch, ow, cache, tokens, parents, choose=osmp.chooser(temp, top_p, u))
        out = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        alen = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        best = torch.empty((n,), dtype=torch.int32, device="cuda")
        B.aded_debug_capture(sess.model, None, best)
        B.aded_verify_sampled(sess.model, sess.kv, H.i32(tokens), H.i32(parents), temp, top_p,
                              torch.tensor(u, device="cuda"), out, alen)
        torch.cuda.synchronize()
        assert B.aded_model_poll_status(sess.model) == 0
        gbest = best.cpu().numpy().astype(np.int64)
        lg32 = cpu["logits"].astype(np.float32)
        for i in range(n):
            if gbest[i] != cpu["best"][i]:
                near = {osmp.sample(lg32[i], temp, top_p, float(np.clip(u[i] + d, 0, 1 - 2.0 ** -24))) for d in (-2e-3, 2e-3)}
                assert int(gbest[i]) in near, f"step {step} node {i}: {gbest[i]} vs {cpu['best'][i]}"
                fragile += 1
        not_greedy += int(np.sum(cpu["best"] != ov.greedy(cpu["logits"])))
        # the emitted sequence is the checker's walk over the GPU's own draws; equal draws give the checker's step
        path, want_out = ov.accept_walk(tokens, parents, gbest)
        a = int(alen[0])
        assert a == len(want_out) and out[:a].tolist() == want_out
        if np.array_equal(gbest, cpu["best"]):
            assert want_out == cpu["out_tokens"]
            assert sess.length() == cache.length
            H.compare_cache(shape, sess, cache, cache.length - a, a, range(shape.n_layers), f"sampled step {step}")
            root = want_out[-1]
        else:
            pytest.skip("a fragile draw changed the accepted path; the remaining steps would compare different texts")
    assert not_greedy >= 3, "the temperature is so low that sampling never left the greedy token"
    assert fragile <= 2


def test_sampled_step_on_the_tensor_core_path(cuda_device):
    """bf16 model (projections and LM head on the tensor-core GEMM, logits gathered from its partial
    tiles): the tokens the sampled step drew equal the library's stand-alone drawing call on the step's
    own logits (that call is checked bit for bit against the checker on seeded logits above), and the
    emitted sequence is the approval walk over those draws."""
    from paper_2407_12021_b200 import binding as B
    shape = gen.ModelShape("bf16-4x64", 2, 256, 4, 64, 384, 1024, "bf16")
    w = gen.model_weights(shape, 91)
    sess = H.GpuSession(shape, H.weights_to(w, cuda_device), capacity=400)
    prompt = gen.zipf_tokens(90, shape.vocab, 91, 50).tolist()
    sess.append(prompt[:-1])
    n = 40
    for step, (temp, top_p) in enumerate([(1.0, 0.9), (0.3, 1.0), (2.0, 0.5)]):
        tokens, parents = gen.make_tree(n, 5, 4, shape.vocab, 92 + step, root_token=prompt[-1])
        u = torch.tensor(gen.uniform01(n, 93, step).numpy().astype(np.float32), device="cuda")
        logits = torch.empty((n, shape.vocab), dtype=torch.float32, device="cuda")
        best = torch.empty((n,), dtype=torch.int32, device="cuda")
        out = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        alen = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        length_before = sess.length()
        B.aded_debug_capture(sess.model, logits, best)
        B.aded_verify_sampled(sess.model, sess.kv, H.i32(tokens), H.i32(parents), temp, top_p, u, out, alen)
        torch.cuda.synchronize()
        assert B.aded_model_poll_status(sess.model) == 0
        again = torch.full((n,), -5, dtype=torch.int32, device="cuda")
        B.aded_sample_tokens(logits, temp, top_p, u, again)
        torch.cuda.synchronize()
        assert torch.equal(again, best)
        path, want_out = ov.accept_walk(tokens, parents, best.cpu().numpy().astype(np.int64))
        a = int(alen[0])
        assert a == len(want_out) and out[:a].tolist() == want_out
        assert sess.length() == length_before + a
        B.aded_kv_set_len(sess.kv, 0, length_before)
