"""Layers whose number of column blocks is a multiple of 4 but not of 8 (q = 4, 12, 20): the bfloat16 operands of the
tensor-core contraction keep their contraction runs a multiple of 8 entries long, so these layers store zero entries
at the end of every run (weights) and write them with every forward (X).  Parity against the oracle for FC and CONV,
float32 and bfloat16, embedded block sizes, stacks whose relay kernel writes such an operand, both conventions, and
the input gradient (a forward of the transposed layer, whose own q is this layer's p)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, oracle_conv, oracle_fc, run_conv, run_fc, scale_rel_err

pytestmark = pytest.mark.gpu
T = circ.CIRC_VARIANT_TENSOR


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("k,p,q,batch", [
    (256, 4, 4, 64),       # the 1024 x 1024, k = 256 point of the sweep
    (256, 4, 4, 1024),
    (16, 12, 12, 33),      # odd batch, 12 -> 16 entries per run
    (64, 3, 20, 200),      # 20 -> 24
    (4, 8, 4, 9),
    (8, 20, 12, 3000),     # large enough for the tiles staged by asynchronous copies on the output side
])
def test_fc_runs_padded_to_eight(k, p, q, batch, bf16):
    case = synth.fc_case(f"pad_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=True, bf16_io=bf16)
    ids = []
    got, used = run_fc(case, kernels=ids)
    assert used == T and ids[1] in (circ.CIRC_KERNEL_S2_TENSOR, circ.CIRC_KERNEL_S2_ROWS), (used, ids)   # never the twin form
    assert not np.isnan(got).any()
    assert scale_rel_err(got, oracle_fc(case)) <= (TOL_BF16 if bf16 else TOL_F32)


def test_stale_workspace_does_not_leak_into_the_padding():
    # a forward at a larger batch leaves arbitrary bits where the next, smaller forward's padding entries lie
    big = synth.fc_case("pad_big", 4 * 64, 4 * 64, 64, 400, w_var=1.0 / 256, x_dist="normal")
    small = synth.fc_case("pad_small", 4 * 64, 4 * 64, 64, 37, w_var=1.0 / 256, x_dist="normal")
    h = circ.circ_fc_create(big.m, big.n, big.k, big.w)
    try:
        circ.circ_set_variant(h, T)
        for case in (big, small, big, small):
            x = torch.from_numpy(case.x).cuda() * 1e30            # huge values: their low bfloat16 parts are anything but zero
            y = torch.empty(case.batch, case.m, device="cuda")
            circ.circ_fc_forward(h, x, y, case.batch, torch.cuda.current_stream())
            x = torch.from_numpy(case.x).cuda()
            y = torch.full((case.batch, case.m), float("nan"), device="cuda")
            circ.circ_fc_forward(h, x, y, case.batch, torch.cuda.current_stream())
            torch.cuda.synchronize()
            got = y.cpu().numpy().astype(np.float64)
            assert scale_rel_err(got, oracle.fc(big.w, case.x)) <= TOL_F32
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("k", [12, 100])
def test_embedded_block_sizes_with_padded_runs(k):
    case = synth.fc_case(f"pad_emb_{k}", 3 * k, 4 * k, k, 21, w_var=1.0 / (4 * k), x_dist="uniform", bias_var=0.01)
    for conv in (0, 1):
        got, used = run_fc(case, convention=conv)
        assert used == T
        assert scale_rel_err(got, oracle_fc(case, conv)) <= TOL_F32


@pytest.mark.parametrize("bf16", [False, True])
def test_conv_runs_padded_to_eight(bf16):
    # 64 input channels in blocks of 16: q = 4
    case = synth.conv_case("pad_conv", 32, 64, 3, 1, 16, 3, 9, 10, w_var=1.0 / (9 * 64), bf16_io=bf16, bias_var=0.01, relu=True)
    got, used = run_conv(case)
    assert used == T and not np.isnan(got).any()
    assert scale_rel_err(got, oracle_conv(case)) <= (TOL_BF16 if bf16 else TOL_F32)


def test_stack_relays_into_a_padded_operand():
    # 512 -> 256 -> 128 with k = 64: the second layer has q = 4, and the relay kernel writes its X
    l0 = synth.fc_case("pad_stack0", 256, 512, 64, 40, w_var=1.0 / 512, x_dist="normal", relu=True)
    l1 = synth.fc_case("pad_stack1", 128, 256, 64, 40, w_var=1.0 / 256, x_dist="normal")
    hs = []
    for l in (l0, l1):
        h = circ.circ_fc_create(l.m, l.n, l.k, l.w)
        circ.circ_set_activation(h, int(l.relu))
        hs.append(h)
    st = circ.circ_stack_create(hs)
    try:
        x = torch.from_numpy(l0.x).cuda()
        y = torch.full((40, 128), float("nan"), device="cuda")
        circ.circ_stack_forward(st, x, y, 40, torch.cuda.current_stream())
        torch.cuda.synchronize()
        assert circ.circ_stack_relayed(st) == 1
        a = oracle.fc(l0.w, l0.x, relu=True)
        assert scale_rel_err(y.cpu().numpy().astype(np.float64), oracle.fc(l1.w, a)) <= TOL_F32
    finally:
        circ.circ_stack_destroy(st)
        for h in hs:
            circ.circ_destroy(h)


def test_input_gradient_of_a_layer_with_four_row_blocks():
    # dL/dx is a forward of the transposed layer, whose q is this layer's p = 4
    case = synth.fc_case("pad_back", 4 * 32, 8 * 32, 32, 50, w_var=1.0 / 256, x_dist="normal")
    g = synth.normal((50, case.m), 1.0, synth.stream_id("pad_back", "g"))
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        gx = torch.full((50, case.n), float("nan"), device="cuda")
        gw = torch.full(case.w.shape, float("nan"), device="cuda")
        circ.circ_fc_backward(h, torch.from_numpy(case.x).cuda(), torch.from_numpy(g).cuda(), gx, gw, 50, torch.cuda.current_stream())
        torch.cuda.synchronize()
        rgx, rgw = oracle.fc_backward(case.w, case.x, g)
        assert scale_rel_err(gx.cpu().numpy().astype(np.float64), rgx) <= TOL_F32
        assert scale_rel_err(gw.cpu().numpy().astype(np.float64), rgw) <= TOL_F32
    finally:
        circ.circ_destroy(h)
