"""GPU parity for block sizes above 256 (k = 512, 1024): the larger transform is the same in-register
transform with more cross-lane butterfly levels (the recursive construction of Sec. 4.1), so every
staged kernel is checked again at these sizes against the fp64 dense oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, oracle_fc, run_fc, scale_rel_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("k", [512, 1024])
@pytest.mark.parametrize("p,q,batch", [(1, 1, 1), (2, 3, 2), (3, 2, 5), (5, 4, 17), (2, 8, 40), (3, 16, 33), (9, 8, 130)])
def test_fc_large_blocks(k, p, q, batch):
    # q % 4 == 0 runs the tensor-core contraction (runs padded to 8 entries), other q the fp32 FMA one; odd batches leave a half-filled pair
    case = synth.fc_case(f"large_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=(batch % 2 == 0))
    got, used = run_fc(case)
    assert used == (circ.CIRC_VARIANT_TENSOR if q % 4 == 0 else circ.CIRC_VARIANT_STAGED)
    assert not np.isnan(got).any()
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


@pytest.mark.parametrize("k", [512, 1024])
def test_single_circulant_limit(k):
    # p = q = 1: the whole weight matrix is one circulant block (the single-circulant baseline the paper generalises)
    case = synth.fc_case(f"single_{k}", k, k, k, 6, w_var=1.0 / k, x_dist="uniform")
    got, _ = run_fc(case)
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32
    got1, _ = run_fc(case, convention=1)
    assert scale_rel_err(got1, oracle_fc(case, 1)) <= TOL_F32


@pytest.mark.parametrize("k", [512, 1024])
def test_forced_fma_and_fused_refusal(k):
    case = synth.fc_case(f"large_fma_{k}", 2 * k, 8 * k, k, 4, w_var=1.0 / (8 * k), x_dist="normal")
    got, used = run_fc(case, circ.CIRC_VARIANT_STAGED)
    assert used == circ.CIRC_VARIANT_STAGED
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32
    with pytest.raises(circ.CircError) as err:      # the one-launch kernel stops at k = 256
        run_fc(case, circ.CIRC_VARIANT_FUSED)
    assert err.value.code == circ.CIRC_ERR_UNSUPPORTED
    got, used = run_fc(case)                        # the planner falls through to the staged kernels at small batch
    assert used == circ.CIRC_VARIANT_TENSOR
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


@pytest.mark.parametrize("k", [512, 1024])
def test_bf16_io_large_blocks(k):
    case = synth.fc_case(f"large_bf16_{k}", 2 * k, 8 * k, k, 24, w_var=1.0 / (8 * k), x_dist="uniform", bf16_io=True)
    got, _ = run_fc(case)
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_BF16


@pytest.mark.parametrize("k", [512, 1024])
def test_backward_large_blocks(k):
    p, q, batch = 2, 3, 10
    case = synth.fc_case(f"large_bwd_{k}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal")
    g = synth.normal((batch, p * k), 1.0, synth.stream_id(case.name, "g"))
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        x = torch.from_numpy(case.x).cuda()
        gd = torch.from_numpy(g).cuda()
        gx = torch.full((batch, case.n), float("nan"), device="cuda")
        gw = torch.full((p, q, k), float("nan"), device="cuda")
        circ.circ_fc_backward(h, x, gd, gx, gw, batch)
        torch.cuda.synchronize()
        ref_x, ref_w = oracle.fc_backward(case.w, case.x, g)
        assert scale_rel_err(gx.cpu().numpy(), ref_x) <= TOL_F32
        assert scale_rel_err(gw.cpu().numpy(), ref_w) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_stack_large_blocks():
    # 4096 -> 2048 -> 1024 with k = 512: the relay kernel at a block size above 256
    dims, k, batch = [4096, 2048, 1024], 512, 12
    cases = [synth.fc_case(f"large_stack_{i}", dims[i + 1], dims[i], k, batch, w_var=1.0 / dims[i], x_dist="absnormal",
                           relu=(i == 0)) for i in range(2)]
    hs = [circ.circ_fc_create(c.m, c.n, c.k, c.w) for c in cases]
    try:
        circ.circ_set_activation(hs[0], 1)
        st = circ.circ_stack_create(hs)
        x = torch.from_numpy(cases[0].x).cuda()
        y = torch.full((batch, dims[-1]), float("nan"), device="cuda")
        circ.circ_stack_forward(st, x, y, batch)
        torch.cuda.synchronize()
        assert circ.circ_stack_relayed(st) == 1
        a = oracle.fc(cases[0].w, cases[0].x, relu=True)
        ref = oracle.fc(cases[1].w, a.astype(np.float32), relu=False)
        assert scale_rel_err(y.cpu().numpy(), ref) <= TOL_F32
        circ.circ_stack_destroy(st)
    finally:
        for h in hs:
            circ.circ_destroy(h)


def test_block_size_limit():
    w = np.zeros(2048, dtype=np.float32)
    with pytest.raises(circ.CircError) as err:
        circ.circ_fc_create(2048, 2048, 2048, w)
    assert err.value.code == circ.CIRC_ERR_SHAPE
