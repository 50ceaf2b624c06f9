"""The allocation-free entry point gives the same answers as the regular one.

``circ_fc_forward_noalloc`` exists for callers that cannot call ``cudaMalloc`` while serving (tight
latency loops, processes whose memory another allocator owns, plug-ins with fixed buffers): its
scratch is a fixed array inside the library instead of an allocated workspace.  This file is named
so that pytest collects it last; it must pass alone in a fresh process and after every other test.
"""
import numpy as np
import pytest
import torch

import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_F32, oracle_fc, scale_rel_err

pytestmark = pytest.mark.gpu


def _layer(case):
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    if case.bias is not None:
        circ.circ_set_bias(h, case.bias)
    circ.circ_set_activation(h, int(case.relu))
    return h


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    big = synth.fc_case("noalloc_a", 1024, 768, 64, 24, w_var=1.0 / 768, x_dist="uniform", bias_var=0.01, relu=True)
    small = synth.fc_case("noalloc_b", 1024, 768, 64, 7, w_var=1.0 / 768, x_dist="normal", bias_var=0.01, relu=True)
    small.w, small.bias = big.w, big.bias            # same layer, a second and smaller batch
    h = _layer(big)
    try:
        circ.circ_set_variant(h, circ.CIRC_VARIANT_STAGED)   # the path the allocation-free call takes
        stream = torch.cuda.current_stream()
        for case in (big, small):                    # two calls in a row share the scratch array
            x = torch.from_numpy(case.x).cuda()
            y_ref = torch.full((case.batch, case.m), float("nan"), device="cuda")
            y_new = torch.full((case.batch, case.m), float("nan"), device="cuda")
            circ.circ_fc_forward(h, x, y_ref, case.batch, stream)
            torch.cuda.synchronize()
            ws_before = circ.circ_workspace_bytes(h)
            free_before = torch.cuda.mem_get_info()[0]
            circ.circ_fc_forward_noalloc(h, x, y_new, case.batch, stream)
            torch.cuda.synchronize()
            assert circ.circ_workspace_bytes(h) == ws_before        # it did not touch the handle's workspace
            assert torch.cuda.mem_get_info()[0] == free_before      # and took no device memory of its own
            ref = y_ref.cpu().numpy().astype(np.float64)
            new = y_new.cpu().numpy().astype(np.float64)
            assert not np.isnan(new).any()
            assert scale_rel_err(new, ref) <= TOL_F32
            assert scale_rel_err(new, oracle_fc(case)) <= TOL_F32
    finally:
        circ.circ_destroy(h)


def test_noalloc_rejects_requests_beyond_its_fixed_scratch():
    limit = circ.circ_noalloc_max_bytes()
    assert limit == 32 * 1024 * 1024
    case = synth.fc_case("noalloc_big", 4096, 4096, 64, 1, w_var=1.0 / 4096, x_dist="uniform")
    h = _layer(case)
    try:
        batch = 2048                                  # 4 * 2048 * (4096 + 4096) bytes = 64 MiB > 32 MiB
        x = torch.zeros(batch, case.n, device="cuda")
        y = torch.zeros(batch, case.m, device="cuda")
        with pytest.raises(circ.CircError) as err:    # nothing prepared yet: it refuses rather than allocate
            circ.circ_fc_forward_noalloc(h, x, y, 256, torch.cuda.current_stream())
        assert err.value.code == circ.CIRC_ERR_UNSUPPORTED
        circ.circ_set_variant(h, circ.CIRC_VARIANT_STAGED)   # the documented preparation, while allocation is allowed
        circ.circ_reserve(h, 256)
        with pytest.raises(circ.CircError) as err:
            circ.circ_fc_forward_noalloc(h, x, y, batch, torch.cuda.current_stream())
        assert err.value.code == circ.CIRC_ERR_SHAPE
        assert str(limit) in str(err.value)
        circ.circ_fc_forward_noalloc(h, x, y, 256, torch.cuda.current_stream())   # 8 MiB fits
        torch.cuda.synchronize()
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("k,bf16", [(12, False), (64, True), (100, True)])
def test_noalloc_embedded_block_sizes_and_bfloat16(k, bf16):
    # block sizes that run on a larger transform (k = 12 on 32 points, k = 100 on 256) size the scratch by the
    # transform size; bfloat16 tensors take the same path
    case = synth.fc_case(f"noalloc_k{k}", 6 * k, 10 * k, k, 9, w_var=1.0 / (10 * k), x_dist="normal", bias_var=0.01, relu=True,
                         bf16_io=bf16)
    h = _layer(case)
    try:
        code = circ.CIRC_BF16 if bf16 else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        circ.circ_set_variant(h, circ.CIRC_VARIANT_STAGED)
        circ.circ_reserve(h, case.batch)
        dt = torch.bfloat16 if bf16 else torch.float32
        x = torch.from_numpy(case.x).cuda().to(dt)
        outs = []
        for call in (circ.circ_fc_forward, circ.circ_fc_forward_noalloc, circ.circ_fc_forward_noalloc):
            y = torch.full((case.batch, case.m), float("nan"), device="cuda", dtype=dt)
            call(h, x, y, case.batch, torch.cuda.current_stream())
            torch.cuda.synchronize()
            outs.append(y.float().cpu().numpy().astype(np.float64))
        assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[1], outs[2])   # the same kernels on the same operands
        assert scale_rel_err(outs[1], oracle_fc(case)) <= (2e-2 if bf16 else TOL_F32)
    finally:
        circ.circ_destroy(h)
