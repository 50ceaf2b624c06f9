"""GPU parity of the pooling layer (Sec. 2.1; the peripheral computing block of Sec. 4.2) against the plain-loop oracle:
max, mean and L2 norm, float32 and bfloat16, the window / stride pairs of the networks the paper names (3 x 3 stride 2,
2 x 2 stride 2), overlapping and non-overlapping windows, channel counts with and without 16-byte groups, windows
that do not fit (dropped), and the error paths of the call."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, scale_rel_err

pytestmark = pytest.mark.gpu

MODES = [(circ.CIRC_POOL_MAX, oracle.POOL_MAX), (circ.CIRC_POOL_AVG, oracle.POOL_AVG), (circ.CIRC_POOL_L2, oracle.POOL_L2)]


def _pool(x_np, window, stride, mode, bf16, offset=0):
    N, H, W, C = x_np.shape
    dt = torch.bfloat16 if bf16 else torch.float32
    xb = torch.zeros(x_np.size + offset, device="cuda", dtype=dt)
    x = xb[offset:]
    x.copy_(torch.from_numpy(x_np).cuda().to(dt).reshape(-1))
    Ho, Wo = (H - window) // stride + 1, (W - window) // stride + 1
    y = torch.full((N, Ho, Wo, C), float("nan"), device="cuda", dtype=dt)
    circ.circ_pool_forward(x, y, N, H, W, C, window, stride, mode, circ.CIRC_BF16 if bf16 else circ.CIRC_F32, torch.cuda.current_stream())
    torch.cuda.synchronize()
    return y.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("N,H,W,C,window,stride", [
    (2, 55, 55, 96, 3, 2),     # the first pooling layer of the ImageNet network whose FC shapes the benchmark uses
    (2, 27, 27, 256, 3, 2),
    (4, 13, 13, 256, 3, 2),
    (8, 28, 28, 32, 2, 2),     # 2 x 2, stride 2 (the MNIST network)
    (1, 9, 11, 7, 3, 1),       # 7 channels: element-wise path; overlapping windows
    (3, 10, 7, 12, 4, 3),      # 12 channels: 16-byte groups for float32 only; the last rows and columns do not fit a window
    (1, 6, 6, 8, 6, 1),        # one window covers the image
    (2, 5, 5, 16, 1, 2),       # 1 x 1 window: subsampling alone
])
def test_pool_matches_the_oracle(N, H, W, C, window, stride, bf16):
    x = synth.normal((N, H, W, C), 1.0, synth.stream_id(f"pool_{N}_{H}_{W}_{C}", "x"))
    if bf16:
        x = synth.round_to_bf16(x)
    for mode, omode in MODES:
        got = _pool(x, window, stride, mode, bf16)
        ref = oracle.pool(x, window, stride, omode)
        assert got.shape == ref.shape and not np.isnan(got).any()
        if mode == circ.CIRC_POOL_MAX:
            assert np.array_equal(got, ref)                     # a maximum of representable values is exact in any precision
        else:
            assert scale_rel_err(got, ref) <= (TOL_BF16 if bf16 else TOL_F32)


def test_pool_of_negative_values_and_unaligned_buffers():
    x = -np.abs(synth.normal((2, 8, 8, 8), 1.0, synth.stream_id("pool_neg", "x"))) - 1.0
    got = _pool(x, 2, 2, circ.CIRC_POOL_MAX, False, offset=1)      # x starts 4 bytes past a 16-byte boundary: element-wise path
    assert np.array_equal(got, oracle.pool(x, 2, 2, oracle.POOL_MAX)) and (got < 0).all()


def test_pool_follows_a_convolution():
    # the layout the convolution writes is the layout the pooling reads: CONV (bias, ReLU) -> 2 x 2 max pooling
    case = synth.conv_case("pool_after_conv", 64, 32, 3, 1, 8, 2, 12, 12, w_var=1.0 / (9 * 32), bf16_io=False, bias_var=0.01, relu=True)
    h = circ.circ_conv_create(case.c_out, case.c_in, case.r, case.pad, case.k, case.w)
    try:
        circ.circ_set_io_dtype(h, circ.CIRC_F32, circ.CIRC_F32)
        circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, 1)
        x = torch.from_numpy(case.x).cuda()
        a = torch.empty((2, 12, 12, 64), device="cuda")
        y = torch.full((2, 6, 6, 64), float("nan"), device="cuda")
        st = torch.cuda.current_stream()
        circ.circ_conv_forward(h, x, a, 2, 12, 12, st)
        circ.circ_pool_forward(a, y, 2, 12, 12, 64, 2, 2, circ.CIRC_POOL_MAX, circ.CIRC_F32, st)
        torch.cuda.synchronize()
        circ.circ_device_status(h)
    finally:
        circ.circ_destroy(h)
    ref = oracle.pool(oracle.conv(case.w, case.x, case.pad, bias=case.bias, relu=True), 2, 2, oracle.POOL_MAX)
    assert scale_rel_err(y.cpu().numpy().astype(np.float64), ref) <= TOL_F32


def test_pool_error_paths():
    x = torch.zeros(2 * 4 * 4 * 4, device="cuda")
    y = torch.zeros(2 * 4 * 4 * 4, device="cuda")
    args = dict(N=2, H=4, W=4, C=4, window=2, stride=2, mode=circ.CIRC_POOL_MAX, dtype=circ.CIRC_F32)

    def call(**kw):
        a = dict(args, **kw)
        circ.circ_pool_forward(a.get("x", x), a.get("y", y), a["N"], a["H"], a["W"], a["C"], a["window"], a["stride"], a["mode"], a["dtype"])

    call()
    for bad, code in ((dict(window=5), circ.CIRC_ERR_SHAPE), (dict(window=0), circ.CIRC_ERR_SHAPE), (dict(stride=0), circ.CIRC_ERR_SHAPE),
                      (dict(N=0), circ.CIRC_ERR_SHAPE), (dict(mode=3), circ.CIRC_ERR_ARG), (dict(dtype=7), circ.CIRC_ERR_ARG),
                      (dict(x=0), circ.CIRC_ERR_ARG)):
        with pytest.raises(circ.CircError) as e:
            call(**bad)
        assert e.value.code == code, bad
