"""GPU parity of the strided convolution (every stride-th output position of Eq. 6) against the oracle: strides 2, 3, 4,
filters 1 x 1 to 7 x 7, padding 0 .. r - 1, float32 and bfloat16, images wider than one tile, odd image counts, extents
that do not divide by the stride; agreement with the stride-1 result subsampled; error paths."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, scale_rel_err, to_device

pytestmark = pytest.mark.gpu


def _run(case, stride):
    h = circ.circ_conv_create(case.c_out, case.c_in, case.r, case.pad, case.k, case.w)
    try:
        if case.bias is not None:
            circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, int(case.relu))
        dt = circ.CIRC_BF16 if case.bf16_io else circ.CIRC_F32
        circ.circ_set_io_dtype(h, dt, dt)
        circ.circ_conv_set_stride(h, stride)
        x = to_device(case.x, case.bf16_io)
        Ho = (case.H + 2 * case.pad - case.r) // stride + 1
        Wo = (case.W + 2 * case.pad - case.r) // stride + 1
        y = torch.full((case.N, Ho, Wo, case.c_out), float("nan"), device="cuda", dtype=torch.bfloat16 if case.bf16_io else torch.float32)
        circ.circ_conv_forward(h, x, y, case.N, case.H, case.W)
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        assert circ.circ_last_variant(h) == circ.CIRC_VARIANT_TENSOR
        return y.float().cpu().numpy().astype(np.float64)
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("r,pad,stride,p,q,k,N,H,W,bf16", [
    (3, 1, 2, 2, 8, 4, 2, 9, 10, False),     # four phase sub-tiles; 10 columns -> 5
    (3, 1, 2, 2, 8, 4, 2, 9, 10, True),
    (3, 0, 2, 3, 8, 16, 3, 11, 8, False),    # no padding, odd image count, 11 rows -> 5
    (3, 1, 2, 4, 4, 16, 2, 28, 28, True),    # q = 4: padded runs; 14 x 14 outputs
    (3, 1, 2, 4, 4, 16, 2, 28, 28, False),
    (5, 2, 2, 2, 8, 4, 1, 13, 12, False),    # 5 x 5: shifts 0, 1, 2 inside a phase
    (7, 3, 2, 1, 8, 4, 1, 23, 20, True),     # 7 x 7, shifts up to 3 (bfloat16: 49 taps' weight tiles of float32 hi + lo do not fit a stage)
    (3, 1, 4, 1, 8, 4, 1, 23, 20, False),    # stride 4 > r: nine phases, no shift, input pixels that no tap reads
    (3, 1, 3, 2, 8, 4, 2, 10, 10, False),    # stride 3 = r: nine phases, no shift
    (1, 0, 2, 2, 16, 8, 2, 7, 9, False),     # 1 x 1: pure subsampling of the channels' product
    (2, 0, 2, 2, 8, 4, 1, 8, 8, True),       # 2 x 2, stride 2: non-overlapping windows
    (3, 1, 2, 2, 8, 4, 1, 5, 300, False),    # 150 output columns: two tiles across, halo over the tile border
    (3, 2, 2, 2, 8, 4, 1, 6, 6, False),      # padding 2 = r - 1
])
def test_strided_conv_matches_the_oracle(r, pad, stride, p, q, k, N, H, W, bf16):
    case = synth.conv_case(f"stride_{r}_{pad}_{stride}_{p}_{q}_{k}_{N}_{H}_{W}", p * k, q * k, r, pad, k, N, H, W,
                           w_var=1.0 / (r * r * q * k), bf16_io=bf16, bias_var=0.01, relu=(N % 2 == 0))
    got = _run(case, stride)
    ref = oracle.conv(case.w, case.x, case.pad, bias=case.bias, relu=case.relu, stride=stride)
    assert got.shape == ref.shape and not np.isnan(got).any()
    assert scale_rel_err(got, ref) <= (TOL_BF16 if bf16 else TOL_F32)


def test_strided_result_is_the_subsampled_stride_one_result():
    case = synth.conv_case("stride_sub", 32, 64, 3, 1, 8, 2, 12, 14, w_var=1.0 / (9 * 64), bf16_io=False)
    full = _run(case, 1)
    half = _run(case, 2)
    assert scale_rel_err(half, full[:, ::2, ::2, :]) <= 2e-6      # the same products in the same order within a pixel


def test_stride_error_paths():
    case = synth.conv_case("stride_err", 16, 12, 3, 1, 4, 1, 6, 6, w_var=0.01, bf16_io=False)      # q = 3: no tensor-core contraction
    h = circ.circ_conv_create(case.c_out, case.c_in, case.r, case.pad, case.k, case.w)
    f = circ.circ_fc_create(16, 16, 4, np.zeros((4, 4, 4), dtype=np.float32))
    try:
        for bad in (0, 5):
            with pytest.raises(circ.CircError) as e:
                circ.circ_conv_set_stride(h, bad)
            assert e.value.code == circ.CIRC_ERR_SHAPE
        with pytest.raises(circ.CircError) as e:
            circ.circ_conv_set_stride(f, 2)
        assert e.value.code == circ.CIRC_ERR_ARG
        circ.circ_set_io_dtype(h, circ.CIRC_F32, circ.CIRC_F32)
        circ.circ_conv_set_stride(h, 2)
        x = torch.from_numpy(case.x).cuda()
        y = torch.empty((1, 3, 3, 16), device="cuda")
        with pytest.raises(circ.CircError) as e:
            circ.circ_conv_forward(h, x, y, 1, 6, 6)
        assert e.value.code == circ.CIRC_ERR_UNSUPPORTED
        g = torch.zeros((1, 3, 3, 16), device="cuda")
        gx = torch.zeros((1, 6, 6, 12), device="cuda")
        with pytest.raises(circ.CircError) as e:
            circ.circ_conv_backward_input(h, g, gx, 1, 6, 6)
        assert e.value.code == circ.CIRC_ERR_UNSUPPORTED
    finally:
        circ.circ_destroy(h)
        circ.circ_destroy(f)
