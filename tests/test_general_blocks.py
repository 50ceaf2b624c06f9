"""GPU parity for block sizes that are not powers of two (and for k = 1, 2).

A circular convolution of length k is the linear convolution of the zero-padded vectors folded back,
a[t] = c[t] + c[t + k]; the library runs such layers on the next power-of-two transform that holds 2k - 1
points and folds in the inverse-transform kernel.  The oracle is the dense definition at the caller's k."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, oracle_conv, oracle_fc, run_conv, run_fc, scale_rel_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("k", [1, 2, 3, 5, 6, 12, 24, 48, 96, 100, 200, 255, 257, 384, 500, 512 - 1])
@pytest.mark.parametrize("p,q,batch", [(1, 1, 1), (3, 2, 3), (2, 5, 16), (2, 8, 33), (5, 16, 6)])
def test_fc_any_block_size(k, p, q, batch):
    case = synth.fc_case(f"gen_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=(batch % 2 == 0))
    got, used = run_fc(case)
    assert used == (circ.CIRC_VARIANT_TENSOR if q % 4 == 0 else circ.CIRC_VARIANT_STAGED)
    assert not np.isnan(got).any()
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


def test_k1_is_a_dense_layer():
    # k = 1: every block is a scalar, the layer is an ordinary dense matrix (the paper's degenerate case)
    case = synth.fc_case("gen_dense", 24, 40, 1, 7, w_var=1.0 / 40, x_dist="normal")
    got, _ = run_fc(case)
    dense = case.w.reshape(24, 40).astype(np.float64)
    assert scale_rel_err(got, case.x.astype(np.float64) @ dense.T) <= TOL_F32


@pytest.mark.parametrize("k", [3, 12, 100])
def test_convention_and_bf16(k):
    case = synth.fc_case(f"gen_conv1_{k}", 2 * k, 8 * k, k, 10, w_var=1.0 / (8 * k), x_dist="uniform")
    got, _ = run_fc(case, convention=1)
    assert scale_rel_err(got, oracle_fc(case, 1)) <= TOL_F32
    cb = synth.fc_case(f"gen_bf16_{k}", 2 * k, 8 * k, k, 10, w_var=1.0 / (8 * k), x_dist="uniform", bf16_io=True)
    got, _ = run_fc(cb)
    assert scale_rel_err(got, oracle_fc(cb)) <= TOL_BF16


@pytest.mark.parametrize("k,c_in,c_out", [(12, 96, 48), (3, 24, 9), (20, 160, 40)])
def test_conv_any_block_size(k, c_in, c_out):
    case = synth.conv_case(f"gen_conv_{k}", c_out, c_in, 3, 1, k, 3, 9, 7, w_var=1.0 / (9 * c_in), bias_var=0.01, relu=True)
    got, _ = run_conv(case)
    assert scale_rel_err(got, oracle_conv(case)) <= TOL_BF16


@pytest.mark.parametrize("k,batch", [(6, 12), (100, 12), (12, 40), (3, 33)])
@pytest.mark.parametrize("convention", [0, 1])
def test_gradients_any_block_size(k, batch, convention):
    # batch >= 32 takes the tensor-core batch product, smaller ones the fp32 FMA one
    p, q = 3, 8
    case = synth.fc_case(f"gen_bwd_{k}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal")
    g = synth.normal((batch, p * k), 1.0, synth.stream_id(case.name, "g"))
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        circ.circ_set_convention(h, convention)
        gd = torch.from_numpy(g).cuda()
        gx = torch.full((batch, case.n), float("nan"), device="cuda")
        gw = torch.full((p, q, k), float("nan"), device="cuda")
        circ.circ_fc_backward(h, torch.from_numpy(case.x).cuda(), gd, gx, gw, batch)
        torch.cuda.synchronize()
        ref_x, ref_w = oracle.fc_backward(case.w, case.x, g, convention=convention)
        assert scale_rel_err(gx.cpu().numpy(), ref_x) <= TOL_F32
        assert scale_rel_err(gw.cpu().numpy(), ref_w) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_conv_gradients_any_block_size():
    k, c_in, c_out = 12, 48, 24
    case = synth.conv_case("gen_conv_bwd", c_out, c_in, 3, 1, k, 2, 6, 5, w_var=1.0 / (9 * c_in), bf16_io=False)
    g = synth.normal((case.N, case.H, case.W, c_out), 1.0, synth.stream_id(case.name, "g"))
    h = circ.circ_conv_create(c_out, c_in, 3, 1, k, case.w)
    try:
        circ.circ_set_io_dtype(h, circ.CIRC_F32, circ.CIRC_F32)
        x = torch.from_numpy(case.x).cuda()
        gd = torch.from_numpy(g).cuda()
        gx = torch.full(case.x.shape, float("nan"), device="cuda")
        gw = torch.full(case.w.shape, float("nan"), device="cuda")
        circ.circ_conv_backward_input(h, gd, gx, case.N, case.H, case.W)
        circ.circ_conv_backward_weight(h, x, gd, gw, case.N, case.H, case.W)
        torch.cuda.synchronize()
        assert scale_rel_err(gx.cpu().numpy(), oracle.conv_backward_input(case.w, g, case.pad, case.H, case.W)) <= TOL_F32
        assert scale_rel_err(gw.cpu().numpy(), oracle.conv_backward_weight(case.x, g, 3, case.pad, k)) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_stack_any_block_size():
    # embedded layers are not relayed: the boundary goes through the stack's activation buffer
    dims, k, batch = [96, 48, 24], 12, 20
    cases = [synth.fc_case(f"gen_stack_{i}", dims[i + 1], dims[i], k, batch, w_var=1.0 / dims[i], x_dist="absnormal") for i in range(2)]
    hs = [circ.circ_fc_create(c.m, c.n, c.k, c.w) for c in cases]
    try:
        circ.circ_set_activation(hs[0], 1)
        st = circ.circ_stack_create(hs)
        x = torch.from_numpy(cases[0].x).cuda()
        y = torch.full((batch, dims[-1]), float("nan"), device="cuda")
        circ.circ_stack_forward(st, x, y, batch)
        torch.cuda.synchronize()
        assert circ.circ_stack_relayed(st) == 0
        a = oracle.fc(cases[0].w, cases[0].x, relu=True)
        ref = oracle.fc(cases[1].w, a.astype(np.float32))
        assert scale_rel_err(y.cpu().numpy(), ref) <= TOL_F32
        circ.circ_stack_destroy(st)
    finally:
        for h in hs:
            circ.circ_destroy(h)


def test_fused_refused_and_limit():
    case = synth.fc_case("gen_fused", 24, 36, 12, 2, w_var=1.0 / 36, x_dist="normal")
    with pytest.raises(circ.CircError) as err:
        run_fc(case, circ.CIRC_VARIANT_FUSED)
    assert err.value.code == circ.CIRC_ERR_UNSUPPORTED
    w = np.zeros(513, dtype=np.float32)
    with pytest.raises(circ.CircError) as err:           # 2 * 513 - 1 points do not fit the largest transform
        circ.circ_fc_create(513, 513, 513, w)
    assert err.value.code == circ.CIRC_ERR_SHAPE


def test_hand_cases_k2_k3():
    # the hand-computed fixtures below the power-of-two range: Fig. 1's shape (m=6, n=3, k=3) and the k=2 row-sum case
    w = np.array([[[1, 2, 3]], [[4, 5, 6]]], dtype=np.float32)
    for conv, x, y in [(0, [1, 1, 1], [6, 6, 6, 15, 15, 15]), (0, [1, 0, 0], [1, 2, 3, 4, 5, 6]), (1, [1, 0, 0], [1, 3, 2, 4, 6, 5])]:
        case = synth.FcCase("hand3", 6, 3, 3, 1, w, np.array([x], dtype=np.float32))
        got, _ = run_fc(case, convention=conv)
        np.testing.assert_allclose(got[0], y, atol=1e-5)
    w2 = np.array([[[1, 2], [3, 4]]], dtype=np.float32)
    case = synth.FcCase("hand2", 2, 4, 2, 1, w2, np.array([[1, 0, 0, 1]], dtype=np.float32))
    got, _ = run_fc(case)
    np.testing.assert_allclose(got[0], [5, 5], atol=1e-5)
