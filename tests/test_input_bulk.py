"""GPU parity for the input-transform kernel that stages its tiles by TMA (large forwards, float32 k = 32 .. 256,
bfloat16 k = 64 .. 256, q a multiple or a divisor of 32): float32 and bfloat16 inputs, all three operand formats (float32 for the FMA contraction, split and
plain bfloat16 for the tensor cores, with and without twin column groups), ragged last tile, odd batches, and
agreement with the load-based kernel."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, scale_rel_err, to_device

pytestmark = pytest.mark.gpu


def _run(case, allow_bulk, variant=circ.CIRC_VARIANT_AUTO):
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        if case.bias is not None:
            circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, int(case.relu))
        code = circ.CIRC_BF16 if case.bf16_io else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        circ.circ_set_variant(h, variant)
        circ.circ_debug_set_transforms(h, allow_bulk, 1)
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
    (64, 16, 8, 6002),     # split bfloat16 operand (tensor cores); tiles of four rows of x, the last one half empty
    (64, 8, 32, 1601),     # one tile = 32 column blocks of a row; odd batch: the last pair has no second sample
    (256, 6, 8, 15000),    # 16 threads per transform in the first pass
    (128, 5, 4, 20000),    # q = 4: bfloat16 runs padded to 8 entries, written by the load-based kernel
    (32, 8, 16, 8000),
    (128, 3, 64, 700),     # two tiles per row
    (16, 40, 8, 10001),    # below the kernel's block sizes: the load-based kernel
    (64, 4, 24, 3000),     # q neither a multiple nor a divisor of 32: the load-based kernel
])
def test_bulk_staged_input_transforms(k, p, q, batch, bf16):
    case = synth.fc_case(f"inbulk_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=True, bf16_io=bf16)
    got, kernels = _run(case, 1)
    served = k >= (64 if bf16 else 32) and (q % 32 == 0 or (32 % q == 0 and q % 8 == 0))
    assert kernels[0] == (circ.CIRC_KERNEL_S1_BULK if served else circ.CIRC_KERNEL_S1_LOADS), kernels
    assert not np.isnan(got).any()
    rows = _rows(batch)
    ref = oracle.fc(case.w, case.x[rows], bias=case.bias, relu=case.relu)
    assert scale_rel_err(got[rows], ref) <= (TOL_BF16 if bf16 else TOL_F32)
    old, kernels_old = _run(case, 0)
    assert kernels_old[0] == circ.CIRC_KERNEL_S1_LOADS
    assert scale_rel_err(got, old) <= (1e-2 if bf16 else 2e-5)     # the same transform, another order of operations


def test_bulk_staged_input_transforms_with_twin_columns():
    # many row blocks, 400 columns: weights stored once, X written as two column groups
    case = synth.fc_case("inbulk_twin", 1024 * 64, 64 * 64, 64, 400, w_var=1.0 / 4096, x_dist="uniform")
    got, kernels = _run(case, 1, circ.CIRC_VARIANT_TENSOR)
    assert kernels[0] == circ.CIRC_KERNEL_S1_BULK and kernels[1] == circ.CIRC_KERNEL_S2_TENSOR_TWIN, kernels
    rows = _rows(case.batch)
    ref = oracle.fc(case.w, case.x[rows])
    assert scale_rel_err(got[rows], ref) <= TOL_F32


def test_bulk_staged_input_is_repeatable_bitwise():
    case = synth.fc_case("inbulk_repeat", 16 * 64, 8 * 64, 64, 6002, w_var=1.0 / 512, x_dist="normal")
    a, _ = _run(case, 1)
    b, _ = _run(case, 1)
    assert np.array_equal(a, b)
