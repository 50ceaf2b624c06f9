"""GPU parity: the CUDA convolution path against the fp64 dense oracle."""
import numpy as np
import pytest

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, oracle_conv, run_conv, scale_rel_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("r,pad,p,q,k,N,H,W", [(3, 1, 2, 2, 4, 2, 5, 6), (3, 1, 3, 2, 16, 3, 7, 5), (1, 0, 2, 3, 8, 2, 3, 3),
                                               (3, 0, 1, 2, 4, 1, 4, 4), (5, 2, 2, 1, 32, 1, 6, 5), (2, 1, 1, 1, 8, 4, 4, 3),
                                               (3, 2, 2, 2, 4, 1, 3, 3)])
@pytest.mark.parametrize("bf16", [False, True])
def test_small_conv(r, pad, p, q, k, N, H, W, bf16):
    case = synth.conv_case(f"conv_{r}_{pad}_{p}_{q}_{k}_{N}", p * k, q * k, r, pad, k, N, H, W,
                           w_var=1.0 / (r * r * q * k), bf16_io=bf16, bias_var=0.01, relu=(N % 2 == 0))
    got, _ = run_conv(case)
    assert not np.isnan(got).any()
    assert scale_rel_err(got, oracle_conv(case)) <= (TOL_BF16 if bf16 else TOL_F32)


def test_conv_convention_flag():
    case = synth.conv_case("conv_flag", 32, 32, 3, 1, 16, 2, 4, 4, w_var=0.01, bf16_io=False)
    g1, _ = run_conv(case, convention=1)
    assert scale_rel_err(g1, oracle_conv(case, 1)) <= TOL_F32
    assert scale_rel_err(g1, oracle_conv(case, 0)) > 1e-2


def test_config4_sampled():
    # full benchmark size; the oracle evaluates every channel of a sample of output pixels that covers
    # image corners, edges, the interior, the first / last image and both halves of the image pairing
    case = synth.config4()
    got, _ = run_conv(case)
    rng = np.random.default_rng(4)
    pix = [(n, h, w) for n in (0, 15, 16, 31) for (h, w) in ((0, 0), (0, 27), (27, 0), (27, 27), (13, 14), (0, 9), (20, 27))]
    pix += [(int(rng.integers(32)), int(rng.integers(28)), int(rng.integers(28))) for _ in range(100)]
    ref = oracle.conv_pixels(case.w, case.x, case.pad, pix)
    sel = np.stack([got[n, h, w] for (n, h, w) in pix])
    assert scale_rel_err(sel, ref) <= TOL_BF16
    assert not np.isnan(got).any()


def test_config4_small_full():
    case = synth.config4(N=3, H=6, W=7)
    got, _ = run_conv(case)
    assert scale_rel_err(got, oracle_conv(case)) <= TOL_BF16
