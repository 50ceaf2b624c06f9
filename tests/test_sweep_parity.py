"""GPU parity at the full sizes of the square-layer sweep (n x k x batch, float32 and bfloat16-input).

The oracle evaluates all n outputs of a few sampled batch rows (first, last, both sides of the
pair split and of a 128-column tile boundary): the layer treats batch rows independently, so a
sampled row checks the whole pipeline for that row.  All 72 points run (about half a minute).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, TOL_F32, scale_rel_err

pytestmark = pytest.mark.gpu

ALL = [(n, k, b, bf) for n in synth.SWEEP_N for k in synth.SWEEP_K for b in synth.SWEEP_B for bf in (False, True)]
POINTS = ALL


def sampled_rows(batch):
    half = (batch + 1) // 2
    rows = {0, batch - 1, half - 1, min(half, batch - 1), min(63, batch - 1), min(64, batch - 1), min(127, batch - 1), min(128, batch - 1)}
    return sorted(rows)


@pytest.mark.parametrize("n,k,batch,bf16", POINTS)
def test_sweep_point(n, k, batch, bf16):
    case = synth.sweep_point(n, k, batch, bf16)
    h = circ.circ_fc_create(n, n, k, case.w)
    try:
        code = circ.CIRC_BF16 if bf16 else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        x = torch.from_numpy(case.x).cuda()
        x = x.to(torch.bfloat16) if bf16 else x
        y = torch.full((batch, n), float("nan"), device="cuda", dtype=torch.bfloat16 if bf16 else torch.float32)
        circ.circ_fc_forward(h, x, y, batch, torch.cuda.current_stream())
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        rows = sampled_rows(batch)
        got = y[rows].float().cpu().numpy().astype(np.float64)
        assert not torch.isnan(y.float()).any()
        ref = oracle.fc(case.w, case.x[rows])
        assert scale_rel_err(got, ref) <= (TOL_BF16 if bf16 else TOL_F32)
    finally:
        circ.circ_destroy(h)
