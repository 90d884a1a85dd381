"""aded_greedy_noalloc -- the allocation-free greedy token choice -- against the library's own
per-node greedy choice and the CPU checker's.

Some users of the library cannot allocate device memory while decoding: the device heap belongs to
another component of their process (a framework's memory pool), or their latency budget forbids
cudaMalloc because it synchronises the device.  For them the library offers its greedy choice as a
stand-alone call that works inside a fixed scratch array.  This test runs a verification step
through the ordinary entry point, captures every node's logits and greedy token, feeds the same
logits to the allocation-free call and expects identical tokens -- twice in a row, because the call
reuses its scratch array and must not depend on what the previous call left there.

The file is named so that pytest collects it last: a run that stops at the first failure has then
already run every other test.  It does not rely on any state left by other tests.
"""
import pytest
import torch

from paper_2407_12021_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _step_logits(cuda_device, nodes, seed):
    """One verification step on the tiny fp32 workload; returns (logits [nodes, V], greedy token per node)."""
    from paper_2407_12021_b200 import binding as B
    shape = gen.TINY
    w = gen.model_weights(shape, seed)
    wc = {k: (v.to(cuda_device) if hasattr(v, "to") else v) for k, v in w.items() if k != "layers"}
    wc["layers"] = [{k: v.to(cuda_device) for k, v in p.items()} for p in w["layers"]]
    model = B.aded_model_create(shape, wc, max_rows=128, max_batch=1)
    kv = B.aded_kv_create(model, [512])
    prompt = gen.zipf_tokens(40, shape.vocab, seed, 50)
    B.aded_append(model, kv, prompt[:-1].to(cuda_device))
    tokens, parents = gen.make_tree(nodes, 6, 6, shape.vocab, seed + 1, root_token=int(prompt[-1]))
    logits = torch.empty((nodes, shape.vocab), dtype=torch.float32, device=cuda_device)
    best = torch.empty((nodes,), dtype=torch.int32, device=cuda_device)
    out = torch.zeros(nodes, dtype=torch.int32, device=cuda_device)
    n = torch.zeros(1, dtype=torch.int32, device=cuda_device)
    B.aded_debug_capture(model, logits, best)
    B.aded_verify(model, kv, torch.tensor(tokens, dtype=torch.int32, device=cuda_device),
                  torch.tensor(parents, dtype=torch.int32, device=cuda_device), out, n)
    torch.cuda.synchronize()
    assert B.aded_model_poll_status(model) == 0 and int(n[0]) >= 1
    return logits, best


def test_noalloc_greedy_matches_verify_twice_in_a_row(cuda_device):
    from paper_2407_12021_b200 import binding as B
    logits_a, best_a = _step_logits(cuda_device, 128, 71)     # the largest size the call accepts
    logits_b, best_b = _step_logits(cuda_device, 37, 72)      # a smaller, ragged one right after it
    got_a = torch.full((128,), -1, dtype=torch.int32, device=cuda_device)
    got_b = torch.full((37,), -1, dtype=torch.int32, device=cuda_device)
    B.aded_greedy_noalloc(logits_a, got_a)
    B.aded_greedy_noalloc(logits_b, got_b)     # reuses the scratch the first call filled
    torch.cuda.synchronize()
    # integer results: the bar is exact equality, as for every index the library produces
    assert torch.equal(got_a, best_a)
    assert torch.equal(got_b, best_b)
    # and equal to the CPU checker's greedy choice on the very same logits (largest value, lowest id among equals)
    from oracle import verify as ov
    assert got_a.cpu().tolist() == ov.greedy(logits_a.cpu().double().numpy()).tolist()
    assert got_b.cpu().tolist() == ov.greedy(logits_b.cpu().double().numpy()).tolist()
    # and once more on the first input: still the same after the array held other rows
    again = torch.full((128,), -1, dtype=torch.int32, device=cuda_device)
    B.aded_greedy_noalloc(logits_a, again)
    torch.cuda.synchronize()
    assert torch.equal(again, best_a)


def test_noalloc_greedy_tie_rule_and_limits(cuda_device):
    from paper_2407_12021_b200 import binding as B
    x = torch.zeros((3, 5000), dtype=torch.float32, device=cuda_device)
    x[0, 4999] = 2.0
    x[0, 17] = 2.0            # equal maxima: the lower index wins
    x[1, :] = -1.0
    x[1, 4000] = -0.5
    got = torch.empty(3, dtype=torch.int32, device=cuda_device)
    B.aded_greedy_noalloc(x, got)
    torch.cuda.synchronize()
    assert got.tolist() == [17, 4000, 0]
    # a row without any finite candidate (all -inf) yields token 0, as the verification step's choice does
    y = torch.full((2, 300), float("-inf"), dtype=torch.float32, device=cuda_device)
    y[1, 299] = -3.0e38
    got2 = torch.full((2,), -1, dtype=torch.int32, device=cuda_device)
    B.aded_greedy_noalloc(y, got2)
    torch.cuda.synchronize()
    assert got2.tolist() == [0, 299]
    too_many = torch.zeros((B.ADED_NOALLOC_MAX_ROWS + 1, 8), dtype=torch.float32, device=cuda_device)
    with pytest.raises(B.AdedError) as err:
        B.aded_greedy_noalloc(too_many, torch.empty(B.ADED_NOALLOC_MAX_ROWS + 1, dtype=torch.int32, device=cuda_device))
    assert err.value.status == 1


def test_noalloc_greedy_leaves_device_memory_as_it_found_it(cuda_device):
    """What the entry point promises the callers it exists for: after its first call on the device (which looks
    up the scratch array's address), a call neither takes nor returns device memory.  Free device memory, as
    the driver reports it, is the same before and after a warm call; torch's own pool is not touched either."""
    from paper_2407_12021_b200 import binding as B
    x = torch.randn((64, 4096), dtype=torch.float32, device=cuda_device)
    got = torch.empty(64, dtype=torch.int32, device=cuda_device)
    B.aded_greedy_noalloc(x, got)              # first call on this device: address look-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info(cuda_device)
    reserved0 = torch.cuda.memory_reserved(cuda_device)
    B.aded_greedy_noalloc(x, got)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info(cuda_device)
    assert free1 == free0 and torch.cuda.memory_reserved(cuda_device) == reserved0
    assert got.cpu().tolist() == x.cpu().argmax(dim=1).tolist()
