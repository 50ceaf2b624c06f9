"""GPU parity of the FC backward pass (Algorithm 2) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_F32, scale_rel_err

pytestmark = pytest.mark.gpu


def run_backward(w, x, g, k, convention=0, want_gx=True, want_gw=True):
    p, q, _ = w.shape
    batch = x.shape[0]
    h = circ.circ_fc_create(p * k, q * k, k, w)
    try:
        circ.circ_set_convention(h, convention)
        xd, gd = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
        gx = torch.full((batch, q * k), float("nan"), device="cuda") if want_gx else None
        gw = torch.full((p, q, k), float("nan"), device="cuda") if want_gw else None
        circ.circ_fc_backward(h, xd, gd, gx, gw, batch, torch.cuda.current_stream())
        circ.circ_fc_backward(h, xd, gd, gx, gw, batch, torch.cuda.current_stream())   # second call: everything cached
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        return (None if gx is None else gx.cpu().numpy().astype(np.float64),
                None if gw is None else gw.cpu().numpy().astype(np.float64))
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("k", [4, 16, 64, 256])
@pytest.mark.parametrize("p,q,batch", [(1, 1, 1), (2, 3, 2), (3, 2, 5), (5, 8, 17), (16, 8, 40), (9, 24, 130)])
def test_backward_small(k, p, q, batch):
    name = f"bwd_{k}_{p}_{q}_{batch}"
    w = synth.normal((p, q, k), 1.0 / (q * k), synth.stream_id(name, "w"))
    x = synth.normal((batch, q * k), 1.0, synth.stream_id(name, "x"))
    g = synth.normal((batch, p * k), 1.0, synth.stream_id(name, "g"))
    gx, gw = run_backward(w, x, g, k)
    ref_gx, ref_gw = oracle.fc_backward(w, x, g)
    assert not np.isnan(gx).any() and not np.isnan(gw).any()
    assert scale_rel_err(gx, ref_gx) <= TOL_F32
    assert scale_rel_err(gw, ref_gw) <= TOL_F32


def test_backward_convention_1_and_partial_outputs():
    k, p, q, batch = 16, 4, 8, 11
    w = synth.normal((p, q, k), 0.01, 1)
    x = synth.normal((batch, q * k), 1.0, 2)
    g = synth.normal((batch, p * k), 1.0, 3)
    gx, gw = run_backward(w, x, g, k, convention=1)
    ref_gx, ref_gw = oracle.fc_backward(w, x, g, convention=1)
    assert scale_rel_err(gx, ref_gx) <= TOL_F32 and scale_rel_err(gw, ref_gw) <= TOL_F32
    ref0_gx, ref0_gw = oracle.fc_backward(w, x, g, convention=0)
    assert scale_rel_err(gx, ref0_gx) > 1e-2 and scale_rel_err(gw, ref0_gw) > 1e-2    # the flag is observable
    only_gx, none_gw = run_backward(w, x, g, k, want_gw=False)
    assert none_gw is None and scale_rel_err(only_gx, ref0_gx) <= TOL_F32
    none_gx, only_gw = run_backward(w, x, g, k, want_gx=False)
    assert none_gx is None and scale_rel_err(only_gw, ref0_gw) <= TOL_F32


def test_backward_config2_shape():
    # 4096 x 4096, k = 64, batch 256: gradients of L = sum(g * a); oracle on all of dL/dw and sampled rows of dL/dx
    case = synth.config2(256)
    g = synth.normal((256, 4096), 1.0, synth.stream_id("cfg2_bwd", "g"))
    gx, gw = run_backward(case.w, case.x, g, 64)
    ref_gx, ref_gw = oracle.fc_backward(case.w, case.x, g)
    assert scale_rel_err(gw, ref_gw) <= TOL_F32
    assert scale_rel_err(gx, ref_gx) <= TOL_F32


@pytest.mark.parametrize("r,pad,p,q,k,N,H,W", [(3, 1, 2, 2, 4, 2, 5, 6), (3, 1, 8, 3, 16, 3, 7, 5), (1, 0, 2, 8, 8, 2, 3, 3),
                                               (3, 0, 8, 2, 4, 1, 5, 4), (5, 2, 2, 8, 4, 1, 6, 5), (3, 2, 8, 8, 4, 2, 3, 3),
                                               (3, 1, 16, 16, 16, 2, 28, 28)])
@pytest.mark.parametrize("bf16", [False, True])
def test_conv_backward_input(r, pad, p, q, k, N, H, W, bf16):
    name = f"cbwd_{r}_{pad}_{p}_{q}_{k}_{N}_{H}_{W}"
    w = synth.normal((r, r, p, q, k), 1.0 / (r * r * p * k), synth.stream_id(name, "w"))
    Ho, Wo = H + 2 * pad - r + 1, W + 2 * pad - r + 1
    g = synth.normal((N, Ho, Wo, p * k), 1.0, synth.stream_id(name, "g"))
    if bf16:
        g = synth.round_to_bf16(g)
    dt = torch.bfloat16 if bf16 else torch.float32
    h = circ.circ_conv_create(p * k, q * k, r, pad, k, w)
    try:
        code = circ.CIRC_BF16 if bf16 else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        gd = torch.from_numpy(g).cuda().to(dt)
        gx = torch.full((N, H, W, q * k), float("nan"), device="cuda", dtype=dt)
        circ.circ_conv_backward_input(h, gd, gx, N, H, W, torch.cuda.current_stream())
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        got = gx.float().cpu().numpy().astype(np.float64)
        assert not np.isnan(got).any()
        ref = oracle.conv_backward_input(w, g, pad, H, W)
        assert scale_rel_err(got, ref) <= (2e-2 if bf16 else TOL_F32)
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("r,pad,p,q,k,N,H,W", [(3, 1, 2, 2, 4, 2, 5, 6), (3, 1, 8, 3, 16, 3, 7, 5), (1, 0, 2, 8, 8, 2, 3, 3),
                                               (3, 0, 8, 2, 4, 1, 5, 4), (5, 2, 2, 8, 4, 1, 6, 5), (3, 2, 8, 8, 4, 2, 3, 3),
                                               (2, 1, 3, 5, 4, 3, 4, 40), (7, 3, 1, 2, 8, 1, 9, 8), (3, 1, 20, 18, 4, 2, 6, 35),
                                               (3, 1, 16, 16, 16, 4, 28, 28)])
@pytest.mark.parametrize("bf16,convention", [(False, 0), (False, 1), (True, 0)])
def test_conv_backward_weight(r, pad, p, q, k, N, H, W, bf16, convention):
    # gradient of L = sum(g * conv(w, x)) with respect to the defining vectors; odd image counts, odd tap counts
    # (the last tap has no partner in the paired inverse transforms), rows wider than one staged segment, p, q > 16
    name = f"cbww_{r}_{pad}_{p}_{q}_{k}_{N}_{H}_{W}"
    w = synth.normal((r, r, p, q, k), 1.0 / (r * r * q * k), synth.stream_id(name, "w"))
    Ho, Wo = H + 2 * pad - r + 1, W + 2 * pad - r + 1
    x = synth.normal((N, H, W, q * k), 1.0, synth.stream_id(name, "x"))
    g = synth.normal((N, Ho, Wo, p * k), 1.0, synth.stream_id(name, "g"))
    if bf16:
        x, g = synth.round_to_bf16(x), synth.round_to_bf16(g)
    dt = torch.bfloat16 if bf16 else torch.float32
    h = circ.circ_conv_create(p * k, q * k, r, pad, k, w)
    try:
        code = circ.CIRC_BF16 if bf16 else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        circ.circ_set_convention(h, convention)
        xd = torch.from_numpy(x).cuda().to(dt)
        gd = torch.from_numpy(g).cuda().to(dt)
        gw = torch.full((r, r, p, q, k), float("nan"), device="cuda", dtype=torch.float32)
        for _ in range(2):   # the second call must overwrite, not accumulate
            circ.circ_conv_backward_weight(h, xd, gd, gw, N, H, W, torch.cuda.current_stream())
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        got = gw.cpu().numpy().astype(np.float64)
        assert not np.isnan(got).any()
        ref = oracle.conv_backward_weight(x, g, r, pad, k, convention=convention)
        assert scale_rel_err(got, ref) <= TOL_F32   # inputs rounded to bfloat16 are exact in the float32 arithmetic
    finally:
        circ.circ_destroy(h)


def test_conv_backward_weight_rejects_bad_arguments():
    w = synth.normal((3, 3, 1, 1, 4), 1.0, 3)
    h = circ.circ_conv_create(4, 4, 3, 1, 4, w)
    hf = circ.circ_fc_create(4, 4, 4, w[0, 0])
    try:
        x = torch.zeros(1, 4, 4, 4, device="cuda")
        gw = torch.zeros(3, 3, 1, 1, 4, device="cuda")
        with pytest.raises(circ.CircError) as e:
            circ.circ_conv_backward_weight(h, x, None, gw, 1, 4, 4)
        assert e.value.code == circ.CIRC_ERR_ARG
        with pytest.raises(circ.CircError) as e:
            circ.circ_conv_backward_weight(hf, x, x, gw, 1, 4, 4)
        assert e.value.code == circ.CIRC_ERR_ARG
        with pytest.raises(circ.CircError) as e:
            circ.circ_conv_backward_weight(h, x, x, gw, 0, 4, 4)
        assert e.value.code == circ.CIRC_ERR_SHAPE
    finally:
        circ.circ_destroy(h)
        circ.circ_destroy(hf)
