"""The tensor-core projection GEMM alone, through the C ABI, against a float64 matrix product of the
same bf16 inputs (the plain definition of the contraction)."""
import numpy as np
import pytest
import torch

from paper_2407_12021_b200 import inputs as gen

pytestmark = pytest.mark.gpu

SMALL16 = gen.ModelShape("gemm-small", 1, 512, 4, 128, 1408, 1024, "bf16")


def _model(shape, dev, seed, max_rows=128):
    from paper_2407_12021_b200 import binding as B
    w = gen.model_weights(shape, seed, device=dev)
    return B, w, B.aded_model_create(shape, w, max_rows=max_rows, max_batch=1)


def _check(B, model, w, which, rows, seed):
    mats = {0: w["layers"][0]["wqkv"], 1: w["layers"][0]["wo"], 2: w["layers"][0]["wgu"], 3: w["layers"][0]["wd"],
            4: w["lm_head"]}
    W = mats[which]
    k = W.shape[1]
    x = gen.normal((rows, k), 1.0, seed, 500 + which, device=W.device, dtype=torch.bfloat16)
    y = B.aded_debug_gemm(model, 0, which, x)
    y2 = B.aded_debug_gemm(model, 0, which, x)
    torch.cuda.synchronize()
    assert B.aded_model_poll_status(model) == 0
    assert torch.equal(y, y2), "the split-tile reduction must not depend on timing"
    want = x.double().cpu().numpy() @ W.double().cpu().numpy().T
    got = y.double().cpu().numpy()
    err = np.max(np.abs(got - want)) / np.max(np.abs(want))
    assert err < 2e-5, (which, rows, err)
    # element-wise: every output within fp32 accumulation error of its own magnitude scale
    bound = 4e-6 * (np.abs(x.double().cpu().numpy()) @ np.abs(W.double().cpu().numpy()).T) + 1e-12
    assert np.all(np.abs(got - want) <= bound), (which, rows)


@pytest.mark.parametrize("rows", [1, 16, 17, 64, 100, 128])
def test_small_shapes_all_projections(cuda_device, rows):
    B, w, model = _model(SMALL16, cuda_device, 41)
    for which in range(5):
        _check(B, model, w, which, rows, 41 + rows)


@pytest.mark.parametrize("rows", [64, 128, 3])
def test_7b_shapes(cuda_device, rows):
    B, w, model = _model(gen.LLAMA7B_1L, cuda_device, 42)
    for which in range(5):
        _check(B, model, w, which, rows, 42 + rows)


def test_more_rows_than_one_pass(cuda_device):
    """Calls with more than 128 rows run as passes of up to 256 rows over the weights (one accumulator of 256
    tensor-memory columns): a single wide pass with a ragged tail (129, 256), two passes (300), five (1228)."""
    B, w, model = _model(SMALL16, cuda_device, 43, max_rows=1228)
    for which in (0, 3):
        _check(B, model, w, which, 300, 43)
        _check(B, model, w, which, 129, 44)
        _check(B, model, w, which, 256, 45)
    _check(B, model, w, 4, 1228, 46)


def test_7b_shape_wide_pass(cuda_device):
    B, w, model = _model(gen.LLAMA7B_1L, cuda_device, 47, max_rows=416)
    for which in (0, 1, 2, 3):
        _check(B, model, w, which, 416, 47)
