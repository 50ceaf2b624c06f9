"""GPU parity of the tensor-core (tcgen05) contraction path against the fp64 dense oracle."""
import numpy as np
import pytest

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, oracle_conv, oracle_fc, run_conv, run_fc, scale_rel_err

pytestmark = pytest.mark.gpu
T = circ.CIRC_VARIANT_TENSOR


@pytest.mark.parametrize("k", [4, 16, 64, 256])
@pytest.mark.parametrize("p,q,batch", [(2, 8, 1), (5, 16, 3), (40, 8, 17), (3, 24, 64), (9, 8, 200), (130, 16, 130), (7, 40, 300)])
def test_fc_tensor_small(k, p, q, batch):
    # spans one and several 128-column tiles, ragged tails in columns, rows and the contraction length
    case = synth.fc_case(f"tc_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=(batch % 2 == 1))
    got, used = run_fc(case, T)
    assert used == T and not np.isnan(got).any()
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


def test_fc_tensor_needs_q_multiple_of_8():
    case = synth.fc_case("tc_bad", 64, 48, 16, 4, w_var=0.1, x_dist="normal")
    with pytest.raises(circ.CircError) as err:
        run_fc(case, T)
    assert err.value.code == circ.CIRC_ERR_UNSUPPORTED


def test_fc_tensor_wide_rows():
    # more than 256 weight rows per problem: several row tiles
    case = synth.fc_case("tc_wide", 2048, 256, 8, 96, w_var=1.0 / 256, x_dist="uniform")
    got, used = run_fc(case, T)
    assert used == T
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


@pytest.mark.parametrize("k,p,q,batch", [(16, 4, 8, 40), (64, 2, 16, 130)])
def test_fc_tensor_bf16(k, p, q, batch):
    case = synth.fc_case(f"tcbf_{k}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="uniform", bf16_io=True)
    got, used = run_fc(case, T)
    assert used == T
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_BF16


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("k,p,q,batch,conv", [(4, 256, 64, 64, 0), (16, 64, 16, 30, 0), (64, 32, 8, 15, 1), (128, 16, 8, 7, 0),
                                              (8, 2048, 24, 100, 0), (32, 48, 8, 1, 1), (16, 448, 16, 200, 0)])
def test_fc_tensor_twin_columns(k, p, q, batch, conv, bf16):
    # many row blocks, few columns: every complex weight is stored once and multiplies two column groups of X,
    # (Zr, -Zi) for the real parts of the result and (Zi, Zr) for the imaginary parts
    case = synth.fc_case(f"twin_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=(batch % 2 == 1), bf16_io=bf16)
    kernels = []
    got, used = run_fc(case, T, convention=conv, kernels=kernels)
    assert used == T and kernels[1] in (circ.CIRC_KERNEL_S2_TENSOR_TWIN, circ.CIRC_KERNEL_S2_ROWS_TWIN), kernels
    assert not np.isnan(got).any()
    assert scale_rel_err(got, oracle_fc(case, conv)) <= (TOL_BF16 if bf16 else TOL_F32)


def test_twin_and_embedded_forms_agree_and_store_half_the_weights():
    import torch
    case = synth.fc_case("twin_vs_embed", 64 * 64, 16 * 64, 64, 24, w_var=1.0 / 1024, x_dist="uniform")
    outs, sizes = [], []
    for allow in (1, 0):
        h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
        try:
            base = circ.circ_weight_bytes(h)
            assert base == 4 * case.m * case.n // case.k                  # the packed spectra and nothing else
            circ.circ_set_variant(h, T)
            circ.circ_debug_set_contraction(h, allow, 0)
            x = torch.from_numpy(case.x).cuda()
            y = torch.empty(case.batch, case.m, device="cuda")
            circ.circ_fc_forward(h, x, y, case.batch)
            torch.cuda.synchronize()
            want = circ.CIRC_KERNEL_S2_TENSOR_TWIN if allow else circ.CIRC_KERNEL_S2_TENSOR
            assert circ.circ_debug_last_kernels(h)[1] == want
            outs.append(y.cpu().numpy().astype(np.float64))
            sizes.append(circ.circ_weight_bytes(h) - base)
        finally:
            circ.circ_destroy(h)
    assert scale_rel_err(outs[0], outs[1]) <= 1e-5
    assert scale_rel_err(outs[0], oracle_fc(case)) <= TOL_F32
    assert sizes[0] < 0.6 * sizes[1]                                       # one copy of every complex value against two


ROWS_SHAPES = [(64, 128, 8, 9), (16, 512, 16, 64), (256, 32, 8, 30), (4, 2048, 64, 100), (64, 256, 8, 64), (16, 520, 24, 128),
               (32, 300, 8, 1), (8, 1100, 40, 17)]


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("k,p,q,batch", ROWS_SHAPES)
def test_fc_tensor_row_streaming(k, p, q, batch, bf16):
    # many row blocks, at most 256 columns: weight rows on the 128-row side of the MMA, all columns in one tile;
    # ragged last row tile, ragged contraction tail, odd batches, with and without twin columns
    case = synth.fc_case(f"rows_{k}_{p}_{q}_{batch}", p * k, q * k, k, batch, w_var=1.0 / (q * k), x_dist="normal",
                         bias_var=0.01, relu=(batch % 2 == 0), bf16_io=bf16)
    ref = oracle_fc(case)
    import torch
    from gpu_helpers import to_device
    for allow_twin in (1, 0):
        h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
        try:
            circ.circ_set_bias(h, case.bias)
            circ.circ_set_activation(h, int(case.relu))
            code = circ.CIRC_BF16 if bf16 else circ.CIRC_F32
            circ.circ_set_io_dtype(h, code, code)
            circ.circ_set_variant(h, T)
            circ.circ_debug_set_contraction(h, allow_twin, 1)
            x = to_device(case.x, bf16)
            y = torch.full((batch, case.m), float("nan"), device="cuda", dtype=torch.bfloat16 if bf16 else torch.float32)
            circ.circ_fc_forward(h, x, y, batch)
            torch.cuda.synchronize()
            circ.circ_device_status(h)
            kern = circ.circ_debug_last_kernels(h)[1]
            assert kern in (circ.CIRC_KERNEL_S2_ROWS, circ.CIRC_KERNEL_S2_ROWS_TWIN), kern
            if not allow_twin:
                assert kern == circ.CIRC_KERNEL_S2_ROWS
            got = y.float().cpu().numpy().astype(np.float64)
            assert not np.isnan(got).any()
            assert scale_rel_err(got, ref) <= (TOL_BF16 if bf16 else TOL_F32)
        finally:
            circ.circ_destroy(h)


def test_stored_forms_are_built_on_first_use():
    import torch
    case = synth.fc_case("lazy_forms", 4096, 4096, 4, 1, w_var=1.0 / 4096, x_dist="uniform")
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        alg = 4 * case.m * case.n // case.k
        x = torch.from_numpy(case.x).cuda()
        y = torch.empty(1, case.m, device="cuda")
        circ.circ_fc_forward(h, x, y, 1)                                   # the one-launch kernel reads the packed spectra
        torch.cuda.synchronize()
        assert circ.circ_last_variant(h) == circ.CIRC_VARIANT_FUSED
        assert circ.circ_weight_bytes(h) + circ.circ_workspace_bytes(h) <= 1.1 * alg
        assert scale_rel_err(y.cpu().numpy().astype(np.float64), oracle_fc(case)) <= TOL_F32
        xb = torch.from_numpy(np.tile(case.x, (40, 1))).cuda()
        yb = torch.empty(40, case.m, device="cuda")
        circ.circ_fc_forward(h, xb, yb, 40)                                # the tensor path builds its own form now
        torch.cuda.synchronize()
        assert circ.circ_weight_bytes(h) > alg
        assert torch.allclose(yb[0], y[0], rtol=0, atol=1e-4 * float(y.abs().max()))
    finally:
        circ.circ_destroy(h)


def test_config2_b256_uses_tensor_cores():
    case = synth.config2(256)
    got, used = run_fc(case)
    assert used == T
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32


def test_convention_1_tensor():
    case = synth.fc_case("tc_conv1", 128, 128, 16, 33, w_var=0.01, x_dist="normal")
    got, _ = run_fc(case, T, convention=1)
    assert scale_rel_err(got, oracle_fc(case, 1)) <= TOL_F32


@pytest.mark.parametrize("r,pad,p,q,k,N,H,W", [(3, 1, 2, 8, 4, 2, 5, 6), (3, 1, 3, 8, 16, 3, 7, 5), (1, 0, 2, 16, 8, 2, 3, 3),
                                               (3, 0, 1, 8, 4, 1, 4, 4), (5, 2, 2, 8, 4, 1, 6, 5), (3, 1, 4, 8, 4, 2, 13, 30),
                                               (3, 2, 2, 8, 4, 1, 3, 3), (3, 1, 2, 8, 4, 1, 3, 150)])
@pytest.mark.parametrize("bf16", [False, True])
def test_conv_tensor_small(r, pad, p, q, k, N, H, W, bf16):
    case = synth.conv_case(f"tcconv_{r}_{pad}_{p}_{q}_{k}_{N}_{H}_{W}", p * k, q * k, r, pad, k, N, H, W,
                           w_var=1.0 / (r * r * q * k), bf16_io=bf16, bias_var=0.01, relu=(N % 2 == 0))
    got, used = run_conv(case, T)
    assert used == T and not np.isnan(got).any()
    assert scale_rel_err(got, oracle_conv(case)) <= (TOL_BF16 if bf16 else TOL_F32)


def test_config4_uses_tensor_cores():
    case = synth.config4()
    got, used = run_conv(case)
    assert used == T
    rng = np.random.default_rng(44)
    pix = [(n, h, w) for n in (0, 15, 16, 31) for (h, w) in ((0, 0), (0, 27), (27, 0), (27, 27), (3, 27), (4, 0), (14, 13))]
    pix += [(int(rng.integers(32)), int(rng.integers(28)), int(rng.integers(28))) for _ in range(100)]
    ref = oracle.conv_pixels(case.w, case.x, case.pad, pix)
    sel = np.stack([got[n, h, w] for (n, h, w) in pix])
    assert scale_rel_err(sel, ref) <= TOL_BF16


def test_very_large_batch_small_layer():
    # many columns, few rows: 70,001 samples through a 128 x 128 layer (547 column tiles, ragged last one, odd batch)
    case = synth.fc_case("tc_bigbatch", 128, 128, 16, 70001, w_var=1.0 / 128, x_dist="uniform")
    got, used = run_fc(case)
    assert used == T and not np.isnan(got).any()
    rows = [0, 1, 35000, 35001, 69999, 70000]
    assert scale_rel_err(got[rows], oracle.fc(case.w, case.x[rows])) <= TOL_F32


def test_conv_wide_image_several_column_tiles():
    # 300-pixel rows: three tiles across, one-row tiles, halo crossing tile and image borders
    case = synth.conv_case("tcconv_wide", 32, 32, 3, 1, 4, 1, 5, 300, w_var=1.0 / (9 * 32), bf16_io=False)
    got, used = run_conv(case, T)
    assert used == T
    assert scale_rel_err(got, oracle_conv(case)) <= TOL_F32


@pytest.mark.parametrize("p,q,r,bf16", [(16, 16, 3, False), (16, 8, 3, False), (24, 8, 1, False), (48, 8, 1, True), (16, 16, 5, True)])
def test_conv_tensor_narrow_row_tiles(p, q, r, bf16):
    # many taps (or a small grid) make the planner cut the weight rows into tiles narrower than the 32-column
    # chunks the epilogue reads from tensor memory: neighbouring row tiles must not overwrite each other
    k = 16
    case = synth.conv_case(f"tcconv_rows_{p}_{q}_{r}_{bf16}", p * k, q * k, r, r // 2, k, 2, 9, 28,
                           w_var=1.0 / (r * r * q * k), bf16_io=bf16)
    got, used = run_conv(case, T)
    assert used == T
    assert scale_rel_err(got, oracle_conv(case)) <= (TOL_BF16 if bf16 else TOL_F32)


def test_fc_tensor_row_tiles_not_multiple_of_32():
    # 2p = 96 rows with a small grid: row tiles of 48
    case = synth.fc_case("tc_rows48", 48 * 8, 64, 8, 40, w_var=1.0 / 64, x_dist="normal")
    got, used = run_fc(case, T)
    assert used == T
    assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32
