"""Failure paths that need a device but fault nothing: a bounded device-side wait that runs out (the producer
issues no copy, so nothing is in flight, the waiting thread block gives up after a few thousand polls, frees
what it holds and returns), and device allocations that fail (an injected failure, before the runtime is asked).
After each failure the same handle serves a correct forward."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_F32, oracle_fc, scale_rel_err

pytestmark = pytest.mark.gpu


def _forward(h, case):
    x = torch.from_numpy(case.x).cuda()
    y = torch.full((case.batch, case.m), float("nan"), device="cuda")
    circ.circ_fc_forward(h, x, y, case.batch, torch.cuda.current_stream())
    torch.cuda.synchronize()
    return y.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("shape", ["large_batch", "row_streaming"])
def test_tensor_contraction_wait_runs_out_and_the_handle_recovers(shape):
    if shape == "large_batch":
        case = synth.fc_case("timeout_tc", 512, 512, 64, 300, w_var=1.0 / 512, x_dist="uniform")
    else:
        case = synth.fc_case("timeout_rows", 128 * 64, 512, 64, 20, w_var=1.0 / 512, x_dist="uniform")
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        circ.circ_set_variant(h, circ.CIRC_VARIANT_TENSOR)
        circ.circ_debug_inject(h, circ.CIRC_INJECT_TENSOR_NO_COPY)
        _forward(h, case)                                   # returns: every wait is bounded
        with pytest.raises(circ.CircError) as e:
            circ.circ_device_status(h)
        assert e.value.code == circ.CIRC_ERR_DEVICE_TIMEOUT
        circ.circ_device_status(h)                          # the word was cleared
        circ.circ_debug_inject(h, circ.CIRC_INJECT_NONE)
        got = _forward(h, case)
        circ.circ_device_status(h)
        rows_kernel = circ.circ_debug_last_kernels(h)[1] in (circ.CIRC_KERNEL_S2_ROWS, circ.CIRC_KERNEL_S2_ROWS_TWIN)
        assert rows_kernel == (shape == "row_streaming")
        assert scale_rel_err(got, oracle_fc(case)) <= TOL_F32
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("m,n,k,batch", [(16 * 64, 8 * 64, 64, 6000), (16 * 64, 8 * 64, 64, 6002), (128 * 4, 8 * 4, 4, 600)])
def test_bulk_fed_inverse_transform_wait_runs_out_and_the_handle_recovers(m, n, k, batch):
    # large enough for the kernels that stage their tiles by asynchronous copies: k = 64, 3000 pairs x 16 row blocks (whole
    # tiles of two pairs: the TMA kernel; 3001 pairs: the bulk-copy kernel); k = 4, 300 pairs x 128 row blocks (the TMA
    # kernel for short blocks)
    case = synth.fc_case(f"timeout_bulk_{k}", m, n, k, batch, w_var=1.0 / n, x_dist="normal")
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        circ.circ_debug_inject(h, circ.CIRC_INJECT_BULK_NO_COPY)
        _forward(h, case)
        assert circ.circ_debug_last_kernels(h)[2] in (circ.CIRC_KERNEL_S3_BULK, circ.CIRC_KERNEL_S3_TMA)
        with pytest.raises(circ.CircError) as e:
            circ.circ_device_status(h)
        assert e.value.code == circ.CIRC_ERR_DEVICE_TIMEOUT
        circ.circ_debug_inject(h, circ.CIRC_INJECT_NONE)
        got = _forward(h, case)
        circ.circ_device_status(h)
        half = (batch + 1) // 2
        rows = [0, 1, half - 1, half, batch - 1]
        ref = oracle.fc(case.w, case.x[rows])
        assert scale_rel_err(got[rows], ref) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_injected_allocation_failures_give_alloc_errors():
    case = synth.fc_case("alloc_fail", 256, 256, 16, 40, w_var=1.0 / 256, x_dist="uniform")
    try:
        circ.circ_debug_fail_alloc_after(1)                 # the copy of the defining vectors
        with pytest.raises(circ.CircError) as e:
            circ.circ_fc_create(case.m, case.n, case.k, case.w)
        assert e.value.code == circ.CIRC_ERR_ALLOC
        circ.circ_debug_fail_alloc_after(2)                 # the packed spectra
        with pytest.raises(circ.CircError) as e:
            circ.circ_fc_create(case.m, case.n, case.k, case.w)
        assert e.value.code == circ.CIRC_ERR_ALLOC
    finally:
        circ.circ_debug_fail_alloc_after(0)
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        circ.circ_set_variant(h, circ.CIRC_VARIANT_STAGED)
        x = torch.from_numpy(case.x).cuda()
        y = torch.empty(case.batch, case.m, device="cuda")
        circ.circ_debug_fail_alloc_after(1)                 # the workspace
        with pytest.raises(circ.CircError) as e:
            circ.circ_fc_forward(h, x, y, case.batch, torch.cuda.current_stream())
        assert e.value.code == circ.CIRC_ERR_ALLOC and circ.circ_workspace_bytes(h) == 0
        circ.circ_debug_fail_alloc_after(2)                 # the stored form of the staged path (built on first use)
        weights = circ.circ_weight_bytes(h)
        with pytest.raises(circ.CircError) as e:
            circ.circ_fc_forward(h, x, y, case.batch, torch.cuda.current_stream())
        assert e.value.code == circ.CIRC_ERR_ALLOC and circ.circ_weight_bytes(h) == weights
        circ.circ_debug_fail_alloc_after(0)
        assert scale_rel_err(_forward(h, case), oracle_fc(case)) <= TOL_F32
    finally:
        circ.circ_debug_fail_alloc_after(0)
        circ.circ_destroy(h)
