"""GPU parity: the CUDA fully-connected path against the fp64 dense oracle, element by element."""
import numpy as np
import pytest

import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, oracle_fc, run_fc, scale_rel_err

pytestmark = pytest.mark.gpu

VARIANTS = [circ.CIRC_VARIANT_STAGED, circ.CIRC_VARIANT_FUSED]


@pytest.mark.parametrize("variant", VARIANTS)
def test_hand_cases_on_gpu(variant, golden_dir):
    # the k=4 hand fixtures (k=2, 3 are below the library's block-size range)
    w = np.array([1, 2, 3, 4], dtype=np.float32).reshape(1, 1, 4)
    for conv, x, y in [(0, [1, 2, 3, 4], [26, 28, 26, 20]), (1, [1, 2, 3, 4], [30, 24, 22, 24]),
                       (0, [0, 1, 0, 0], [4, 1, 2, 3]), (1, [0, 1, 0, 0], [2, 1, 4, 3])]:
        case = synth.FcCase("hand", 4, 4, 4, 1, w, np.array([x], dtype=np.float32))
        got, _ = run_fc(case, variant, convention=conv)
        np.testing.assert_allclose(got[0], y, atol=1e-5)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("k", [4, 8, 16, 32, 64, 128, 256])
@pytest.mark.parametrize("p,q,batch", [(1, 1, 1), (2, 3, 2), (3, 2, 3), (5, 7, 17), (3, 3, 64), (9, 11, 8), (40, 3, 5)])
def test_small_shapes_all_block_sizes(variant, k, p, q, batch):
    case = synth.fc_case(f"small_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=(batch % 2 == 0))
    if variant == circ.CIRC_VARIANT_FUSED and batch > 8:
        with pytest.raises(circ.CircError) as err:      # the one-launch kernel serves batch <= 8 only
            run_fc(case, variant)
        assert err.value.code == circ.CIRC_ERR_UNSUPPORTED
        return
    got, used = run_fc(case, variant)
    assert used == variant
    assert not np.isnan(got).any()
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


@pytest.mark.parametrize("variant", VARIANTS)
def test_convention_flag(variant):
    case = synth.fc_case("conv_flag", 64, 96, 16, 3, w_var=0.01, x_dist="normal")
    g0, _ = run_fc(case, variant, convention=0)
    g1, _ = run_fc(case, variant, convention=1)
    assert scale_rel_err(g0, oracle_fc(case, 0)) <= TOL_F32
    assert scale_rel_err(g1, oracle_fc(case, 1)) <= TOL_F32
    assert scale_rel_err(g0, oracle_fc(case, 1)) > 1e-2     # the flag is observable


def _run_fused_split(case, slices):
    import torch
    from gpu_helpers import to_device
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, 1)
        code = circ.CIRC_BF16 if case.bf16_io else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        circ.circ_set_variant(h, circ.CIRC_VARIANT_FUSED)
        circ.circ_debug_set_fused_split(h, slices)
        x = to_device(case.x, case.bf16_io)
        y = torch.full((case.batch, case.m), float("nan"), device="cuda", dtype=torch.bfloat16 if case.bf16_io else torch.float32)
        circ.circ_fc_forward(h, x, y, case.batch)
        torch.cuda.synchronize()
        return y.float().cpu().numpy().astype(np.float64), circ.circ_debug_last_kernels(h)
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("k,p,q,batch", [(64, 4, 64, 1), (256, 2, 16, 3), (16, 8, 128, 8), (4, 16, 1024, 5), (128, 64, 8, 2),
                                         (32, 300, 24, 7), (256, 64, 64, 1), (64, 256, 256, 2), (8, 3, 40, 4)])
def test_one_launch_kernel_with_split_columns(k, p, q, batch, bf16):
    # the columns split over the 1, 2, 4 or 8 thread blocks of a cluster, partial spectra added up through distributed
    # shared memory: odd row counts, all pair counts, both storage types, bias + ReLU, every split that divides q
    case = synth.fc_case(f"split_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=True, bf16_io=bf16)
    ref = oracle_fc(case)
    for slices in (1, 2, 4, 8):
        if q % slices:
            continue
        got, kernels = _run_fused_split(case, slices)
        assert kernels[0] == circ.CIRC_KERNEL_S4_FUSED and kernels[1] == slices
        assert not np.isnan(got).any()
        assert scale_rel_err(got, ref) <= (TOL_BF16 if bf16 else TOL_F32)
        again, _ = _run_fused_split(case, slices)
        assert np.array_equal(got, again)         # fixed-order sums: bitwise repeatable


def test_one_launch_planner_splits_wide_layers_with_few_rows():
    case = synth.fc_case("split_plan", 16384, 16384, 256, 1, w_var=1.0 / 16384, x_dist="uniform")
    kernels = []
    run_fc(case, circ.CIRC_VARIANT_FUSED, kernels=kernels)
    assert kernels[0] == circ.CIRC_KERNEL_S4_FUSED and kernels[1] > 1 and kernels[1] * -(-64 // kernels[2]) >= 100, kernels


def test_config1():
    case = synth.config1()
    got, _ = run_fc(case)
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


@pytest.mark.parametrize("batch", [1, 16, 256])
def test_config2(batch):
    case = synth.config2(batch)
    got, used = run_fc(case)
    assert used == (circ.CIRC_VARIANT_FUSED if batch == 1 else used)
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("batch", [1, 2, 7, 8])
def test_config2_small_batches_both_variants(variant, batch):
    case = synth.config2(batch)
    got, used = run_fc(case, variant)
    assert used == variant
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


def test_config3_stack():
    layers = synth.config3_layers(128)
    x = layers[0].x
    for c in layers:
        c.x = x
        got, _ = run_fc(c)
        ref = oracle_fc(c)
        assert scale_rel_err(got, ref) <= TOL_F32
        x = got.astype(np.float32)   # feed the GPU activations forward, as a real stack does


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("k,p,q,batch", [(16, 4, 4, 5), (64, 2, 2, 8), (4, 8, 8, 3)])
def test_bf16_io(variant, k, p, q, batch):
    case = synth.fc_case(f"bf16_{k}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="uniform", bf16_io=True)
    got, _ = run_fc(case, variant)
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_BF16
    got32, _ = run_fc(case, variant, y_bf16=False)     # bf16 in, float32 out: only the input was rounded
    assert scale_rel_err(got32, oracle_fc(case)) <= TOL_F32


def test_repeatable_bitwise():
    case = synth.config2(16)
    a, _ = run_fc(case)
    b, _ = run_fc(case)
    assert np.array_equal(a, b)


def test_very_large_batch_fma_path():
    # q = 2 is not a multiple of 8, so this runs the float32 FMA contraction: 50,001 samples, ragged tiles everywhere
    case = synth.fc_case("fma_bigbatch", 48, 32, 16, 50001, w_var=1.0 / 32, x_dist="normal", bias_var=0.01, relu=True)
    got, used = run_fc(case)
    assert used == circ.CIRC_VARIANT_STAGED
    rows = [0, 25000, 25001, 50000]
    import oracle
    assert scale_rel_err(got[rows], oracle.fc(case.w, case.x[rows], bias=case.bias, relu=True)) <= TOL_F32
