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
