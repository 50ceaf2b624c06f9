"""GPU parity for the inverse-transform kernels that write their tiles by TMA (large forwards; float32 k = 32 .. 256,
bfloat16 k = 64 .. 256, p a multiple of 32 or a divisor of it with whole tiles; short blocks, one thread per transform:
float32 k = 4 .. 16, bfloat16 k = 8, 16, p a multiple of 128): bias and ReLU, float32 and bfloat16
outputs, odd batches, Y that comes as several copies with real and imaginary parts apart (after the row-streaming
contraction), and agreement with the load-based kernels."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, scale_rel_err, to_device

pytestmark = pytest.mark.gpu


def _run(case, allow_tma, variant=circ.CIRC_VARIANT_AUTO):
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        if case.bias is not None:
            circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, int(case.relu))
        code = circ.CIRC_BF16 if case.bf16_io else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        circ.circ_set_variant(h, variant)
        circ.circ_debug_set_transforms(h, 1, allow_tma)
        x = to_device(case.x, case.bf16_io)
        y = torch.full((case.batch, case.m), float("nan"), device="cuda", dtype=torch.bfloat16 if case.bf16_io else torch.float32)
        circ.circ_fc_forward(h, x, y, case.batch)
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        return y.float().cpu().numpy().astype(np.float64), circ.circ_debug_last_kernels(h)
    finally:
        circ.circ_destroy(h)


def _rows(B):
    half = (B + 1) // 2
    return sorted({0, 1, half - 1, half, half + 1, B - 2, B - 1, B // 3})   # both members of the first and last pairs


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("k,p,q,batch", [
    (64, 32, 8, 3000),     # one tile = the 32 row blocks of a pair
    (64, 16, 8, 6000),     # tiles of two pairs
    (64, 64, 8, 1601),     # two tiles per pair; odd batch: the last pair's second sample does not exist
    (256, 8, 8, 12000),    # 16 threads per transform in the second pass
    (128, 64, 4, 700),     # float32 FMA contraction feeds the same kernel
    (32, 32, 8, 4000),
    (64, 16, 8, 6002),     # 3001 pairs: a tile of two pairs would be partial -> the other kernels
    (64, 24, 8, 4000),     # p neither a multiple nor a divisor of 32 -> the other kernels
])
def test_tma_written_inverse_transforms(k, p, q, batch, bf16):
    case = synth.fc_case(f"outtma_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=True, bf16_io=bf16)
    got, kernels = _run(case, 1)
    bho = (batch + 1) // 2
    served = k >= (64 if bf16 else 32) and (p % 32 == 0 or (p % 4 == 0 and 32 % p == 0 and bho % (32 // p) == 0))
    assert (kernels[2] == circ.CIRC_KERNEL_S3_TMA) == served, kernels
    assert not np.isnan(got).any()
    rows = _rows(batch)
    ref = oracle.fc(case.w, case.x[rows], bias=case.bias, relu=case.relu)
    assert scale_rel_err(got[rows], ref) <= (TOL_BF16 if bf16 else TOL_F32)
    if served:
        old, kernels_old = _run(case, 0)
        assert kernels_old[2] != circ.CIRC_KERNEL_S3_TMA
        assert scale_rel_err(got, old) <= (2e-2 if bf16 else 2e-5)     # the same transform, another order of operations


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("k,p,q,batch", [
    (4, 128, 8, 600),      # one complex problem; one tile per pair
    (4, 256, 16, 301),     # two tiles per pair, odd batch
    (8, 128, 8, 400),
    (16, 384, 8, 255),     # three tiles per pair, seven complex problems, odd batch
    (16, 128, 16, 2000),   # more tiles than resident thread blocks: the double buffers are reused many times
    (8, 192, 8, 500),      # p not a multiple of 128 -> the other kernels
])
def test_tma_written_inverse_transforms_of_short_blocks(k, p, q, batch, bf16):
    case = synth.fc_case(f"outtma_small_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=True, bf16_io=bf16)
    got, kernels = _run(case, 1, circ.CIRC_VARIANT_TENSOR)
    served = p % 128 == 0 and k >= (8 if bf16 else 4)
    assert (kernels[2] == circ.CIRC_KERNEL_S3_TMA) == served, kernels
    assert not np.isnan(got).any()
    rows = _rows(batch)
    ref = oracle.fc(case.w, case.x[rows], bias=case.bias, relu=case.relu)
    assert scale_rel_err(got[rows], ref) <= (TOL_BF16 if bf16 else TOL_F32)
    if served:
        old, kernels_old = _run(case, 0, circ.CIRC_VARIANT_TENSOR)
        assert kernels_old[2] != circ.CIRC_KERNEL_S3_TMA
        assert scale_rel_err(got, old) <= (2e-2 if bf16 else 2e-5)


@pytest.mark.parametrize("bf16", [False, True])
def test_copies_of_y_after_the_row_streaming_contraction_take_the_load_based_kernel(bf16):
    # 512 row blocks, 60 columns: the contraction writes several copies of Y with real and imaginary parts apart, which
    # the load-based inverse transforms add up (little to transform at so few columns)
    case = synth.fc_case("outtma_rows", 512 * 64, 8 * 64, 64, 60, w_var=1.0 / 512, x_dist="uniform", bias_var=0.01, relu=True,
                         bf16_io=bf16)
    got, kernels = _run(case, 1, circ.CIRC_VARIANT_TENSOR)
    assert kernels[1] == circ.CIRC_KERNEL_S2_ROWS_TWIN and kernels[2] == circ.CIRC_KERNEL_S3_LOADS, kernels
    ref = oracle.fc(case.w, case.x, bias=case.bias, relu=True)
    assert scale_rel_err(got, ref) <= (TOL_BF16 if bf16 else TOL_F32)


def test_tma_written_output_is_repeatable_bitwise():
    case = synth.fc_case("outtma_repeat", 32 * 64, 8 * 64, 64, 3000, w_var=1.0 / 512, x_dist="normal")
    a, _ = _run(case, 1)
    b, _ = _run(case, 1)
    assert np.array_equal(a, b)
