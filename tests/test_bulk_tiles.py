"""GPU parity for the inverse-transform kernel that fetches its tiles by bulk copies (large forwards, 16 <= k <= 256):
bias and ReLU, a ragged last tile, float32 and bfloat16 outputs, and the fall-back when the runs are not 16-byte
aligned (an odd number of transforms)."""
import numpy as np
import pytest

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, run_fc, scale_rel_err

pytestmark = pytest.mark.gpu


def _check(case, tol, want_s3):
    got, used = run_fc(case, kernels=(kernels := []))
    assert kernels[2] == want_s3, kernels          # the inverse-transform kernel under test really served the call
    assert not np.isnan(got).any()
    B = case.batch
    half = (B + 1) // 2
    rows = sorted({0, 1, half - 1, half, half + 1, B - 2, B - 1, B // 3})   # both members of the first and last pairs
    ref = oracle.fc(case.w, case.x[rows], bias=case.bias, relu=case.relu)
    assert scale_rel_err(got[rows], ref) <= tol
    return used


@pytest.mark.parametrize("k,p,q,batch", [
    (64, 16, 8, 6002),     # 48016 transforms: even, last tile of 32 half full
    (16, 40, 8, 4000),     # one lane per transform
    (256, 6, 8, 15000),    # 16 lanes per transform, 45000 transforms
    (128, 5, 3, 20000),    # q % 4 != 0: the fp32 FMA contraction feeds the same kernel
])
def test_bulk_tiles_float32(k, p, q, batch):
    case = synth.fc_case(f"bulk_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=True)
    used = _check(case, TOL_F32, circ.CIRC_KERNEL_S3_BULK)
    assert used == (circ.CIRC_VARIANT_TENSOR if q % 4 == 0 else circ.CIRC_VARIANT_STAGED)


def test_bulk_tiles_bfloat16():
    case = synth.fc_case("bulk_bf16", 16 * 64, 8 * 64, 64, 6002, w_var=1.0 / 512, x_dist="uniform", bias_var=0.01, relu=True,
                         bf16_io=True)
    _check(case, TOL_BF16, circ.CIRC_KERNEL_S3_BULK)


def test_odd_transform_count_falls_back():
    # 3001 pairs x 15 row blocks = 45015 transforms: the runs of Y are not 16-byte aligned, the load-based kernel runs
    case = synth.fc_case("bulk_odd", 15 * 64, 8 * 64, 64, 6001, w_var=1.0 / 512, x_dist="normal", bias_var=0.01, relu=True)
    _check(case, TOL_F32, circ.CIRC_KERNEL_S3_LOADS)


def test_repeatable_bitwise_large():
    case = synth.fc_case("bulk_repeat", 16 * 64, 8 * 64, 64, 6002, w_var=1.0 / 512, x_dist="normal")
    a, _ = run_fc(case)
    b, _ = run_fc(case)
    assert np.array_equal(a, b)
