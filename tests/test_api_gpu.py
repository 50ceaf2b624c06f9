"""GPU tests of the C-ABI's companion calls: host-pointer forwards, workspace reservation, timing aids,
stream handling, error codes that need a device."""
import numpy as np
import pytest
import torch

import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, oracle_conv, oracle_fc, scale_rel_err

pytestmark = pytest.mark.gpu


def _fc_handle(case):
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    if case.bias is not None:
        circ.circ_set_bias(h, case.bias)
    circ.circ_set_activation(h, int(case.relu))
    return h


@pytest.mark.parametrize("batch", [3, 40])
def test_fc_forward_host_matches_oracle(batch):
    case = synth.fc_case(f"host_{batch}", 512, 384, 32, batch, w_var=1.0 / 384, x_dist="uniform", bias_var=0.01, relu=True)
    h = _fc_handle(case)
    try:
        x = torch.from_numpy(case.x).pin_memory()
        y = torch.empty(batch, case.m).pin_memory()
        s = torch.cuda.Stream()
        circ.circ_fc_forward_host(h, x, y, batch, s)
        s.synchronize()
        assert scale_rel_err(y.numpy().astype(np.float64), oracle_fc(case)) <= TOL_F32
        circ.circ_fc_forward_host(h, case.x, y, batch, s)          # pageable numpy input works too
        s.synchronize()
        assert scale_rel_err(y.numpy().astype(np.float64), oracle_fc(case)) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_conv_forward_host_matches_oracle():
    cc = synth.conv_case("host_conv", 64, 128, 3, 1, 16, 2, 6, 5, w_var=1.0 / (9 * 128))
    h = circ.circ_conv_create(cc.c_out, cc.c_in, cc.r, cc.pad, cc.k, cc.w)
    try:
        x = torch.from_numpy(cc.x).to(torch.bfloat16).pin_memory()
        y = torch.empty(cc.N, cc.H, cc.W, cc.c_out, dtype=torch.bfloat16).pin_memory()
        circ.circ_conv_forward_host(h, x, y, cc.N, cc.H, cc.W, torch.cuda.current_stream())
        torch.cuda.synchronize()
        assert scale_rel_err(y.float().numpy().astype(np.float64), oracle_conv(cc)) <= TOL_BF16
    finally:
        circ.circ_destroy(h)


def test_reserve_then_forward_allocates_nothing():
    case = synth.fc_case("reserve", 256, 256, 16, 64, w_var=1.0 / 256, x_dist="uniform")
    h = _fc_handle(case)
    try:
        assert circ.circ_workspace_bytes(h) == 0
        circ.circ_reserve(h, 64)
        ws = circ.circ_workspace_bytes(h)
        assert ws >= 4 * 65 * (256 + 256)
        x = torch.from_numpy(case.x).cuda()
        y = torch.empty(64, 256, device="cuda")
        for b in (64, 33, 9):
            circ.circ_fc_forward(h, x[:b].contiguous(), y[:b], b, torch.cuda.current_stream())
        torch.cuda.synchronize()
        assert circ.circ_workspace_bytes(h) == ws
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("variant,batch", [(circ.CIRC_VARIANT_FUSED, 4), (circ.CIRC_VARIANT_TENSOR, 48), (circ.CIRC_VARIANT_STAGED, 48)])
def test_repeated_stage_leaves_results_unchanged(variant, batch):
    case = synth.fc_case(f"repeat_{variant}", 512, 512, 64, batch, w_var=1.0 / 512, x_dist="normal", bias_var=0.01, relu=True)
    h = _fc_handle(case)
    try:
        circ.circ_set_variant(h, variant)
        x = torch.from_numpy(case.x).cuda()
        y0 = torch.empty(batch, case.m, device="cuda")
        y1 = torch.empty(batch, case.m, device="cuda")
        s = torch.cuda.current_stream()
        circ.circ_fc_forward(h, x, y0, batch, s)                     # the first forward also builds the stored form it reads
        l0 = circ.circ_debug_launch_count()
        circ.circ_fc_forward(h, x, y0, batch, s)
        per_forward = circ.circ_debug_launch_count() - l0
        assert per_forward == (1 if variant == circ.CIRC_VARIANT_FUSED else 3)
        stages = [circ.CIRC_STAGE_FUSED] if variant == circ.CIRC_VARIANT_FUSED else [0, 1, 2]
        for st in stages:
            l0 = circ.circ_debug_launch_count()
            circ.circ_debug_forward_repeat(h, x, y1, batch, 1, 1, st, 3, s)
            assert circ.circ_debug_launch_count() - l0 == per_forward + 2
            torch.cuda.synchronize()
            assert torch.equal(y0, y1)                               # bitwise: every kernel rewrites the same values
        assert scale_rel_err(y1.cpu().numpy().astype(np.float64), oracle_fc(case)) <= TOL_F32
        with pytest.raises(circ.CircError):
            circ.circ_debug_forward_repeat(h, x, y1, batch, 1, 1, 7, 2, s)
        if variant != circ.CIRC_VARIANT_FUSED:
            want = (circ.CIRC_KERNEL_S2_TENSOR, circ.CIRC_KERNEL_S2_TENSOR_TWIN) if variant == circ.CIRC_VARIANT_TENSOR else (circ.CIRC_KERNEL_S2_FMA,)
            assert circ.circ_debug_last_kernels(h)[1] in want
    finally:
        circ.circ_destroy(h)


def test_growing_the_workspace_inside_a_capture_is_refused_up_front():
    case = synth.fc_case("capture_grow", 256, 256, 16, 64, w_var=1.0 / 256, x_dist="uniform")
    h = _fc_handle(case)
    try:
        x = torch.from_numpy(case.x).cuda()
        y = torch.empty(64, 256, device="cuda")
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            with pytest.raises(circ.CircError) as e:
                circ.circ_fc_forward(h, x, y, 64, torch.cuda.current_stream())      # no workspace yet
            assert e.value.code == circ.CIRC_ERR_UNSUPPORTED
        circ.circ_reserve(h, 64)
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=side):
            circ.circ_fc_forward(h, x, y, 64, torch.cuda.current_stream())
        g2.replay()
        torch.cuda.synchronize()
        assert scale_rel_err(y.cpu().numpy().astype(np.float64), oracle_fc(case)) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_forward_on_a_side_stream_and_weights_from_device_memory():
    case = synth.fc_case("stream", 128, 256, 8, 20, w_var=1.0 / 256, x_dist="uniform")
    w_dev = torch.from_numpy(case.w).cuda()
    h = circ.circ_fc_create(case.m, case.n, case.k, w_dev)           # device pointer for w
    try:
        side = torch.cuda.Stream()
        x = torch.from_numpy(case.x).cuda()
        y = torch.empty(20, 128, device="cuda")
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            circ.circ_fc_forward(h, x, y, 20, side)
        side.synchronize()
        assert scale_rel_err(y.cpu().numpy().astype(np.float64), oracle_fc(case)) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_device_side_argument_errors():
    case = synth.fc_case("errs", 64, 64, 16, 4, w_var=1.0 / 64, x_dist="uniform")
    h = _fc_handle(case)
    try:
        x = torch.zeros(4, 64, device="cuda")
        y = torch.zeros(4, 64, device="cuda")
        with pytest.raises(circ.CircError) as e:
            circ.circ_fc_forward(h, x, x, 4)                         # aliasing
        assert e.value.code == circ.CIRC_ERR_ARG
        with pytest.raises(circ.CircError) as e:
            circ.circ_fc_forward(h, x.data_ptr() + 4, y, 1)          # misaligned
        assert e.value.code == circ.CIRC_ERR_ARG
        with pytest.raises(circ.CircError) as e:
            circ.circ_fc_forward(h, x, y, 0)
        assert e.value.code == circ.CIRC_ERR_SHAPE
        with pytest.raises(circ.CircError) as e:
            circ.circ_conv_forward(h, x, y, 1, 2, 2)                 # FC handle in the CONV call
        assert e.value.code == circ.CIRC_ERR_ARG
        circ.circ_device_status(h)
    finally:
        circ.circ_destroy(h)
