"""Helpers shared by the GPU parity tests: run a case through the C ABI, compare with the oracle."""
import numpy as np
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth

TOL_F32 = 1e-4    # max |gpu - oracle| / max |oracle|, float32 path
TOL_BF16 = 2e-2   # bfloat16-input, float32-accumulate path


def scale_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """E = max_t |g_t - o_t| / max_t |o_t| over the whole tensor."""
    denom = float(np.max(np.abs(ref)))
    if denom == 0.0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got.astype(np.float64) - ref)) / denom)


def floored_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """The secondary, element-wise figure: max_t |g_t - o_t| / max(|o_t|, 1e-3 rms(o)).  Reported, not a pass criterion:
    it divides by each element's own magnitude (floored), so it is larger than E wherever small outputs carry the
    absolute error of large sums."""
    ref = ref.astype(np.float64)
    floor = 1e-3 * float(np.sqrt(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), floor if floor > 0.0 else 1.0)
    return float(np.max(np.abs(got.astype(np.float64) - ref) / den))


def to_device(a: np.ndarray, bf16: bool) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if bf16 else t


def run_fc(case: synth.FcCase, variant=circ.CIRC_VARIANT_AUTO, convention=0, y_bf16=None, stream=None, kernels=None):
    """Returns (y as float64 numpy [B][m], variant used); ``kernels``: a list that receives the S1 / S2 / S3 kernel ids."""
    y_bf16 = case.bf16_io if y_bf16 is None else y_bf16
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        if case.bias is not None:
            circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, int(case.relu))
        circ.circ_set_io_dtype(h, circ.CIRC_BF16 if case.bf16_io else circ.CIRC_F32,
                               circ.CIRC_BF16 if y_bf16 else circ.CIRC_F32)
        circ.circ_set_convention(h, convention)
        circ.circ_set_variant(h, variant)
        x = to_device(case.x, case.bf16_io)
        y = torch.full((case.batch, case.m), float("nan"), device="cuda",
                       dtype=torch.bfloat16 if y_bf16 else torch.float32)
        circ.circ_fc_forward(h, x, y, case.batch, stream)
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        used = circ.circ_last_variant(h)
        if kernels is not None:
            kernels.extend(circ.circ_debug_last_kernels(h))
        return y.float().cpu().numpy().astype(np.float64), used
    finally:
        circ.circ_destroy(h)


def run_conv(case: synth.ConvCase, variant=circ.CIRC_VARIANT_AUTO, convention=0):
    h = circ.circ_conv_create(case.c_out, case.c_in, case.r, case.pad, case.k, case.w)
    try:
        if case.bias is not None:
            circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, int(case.relu))
        dt = circ.CIRC_BF16 if case.bf16_io else circ.CIRC_F32
        circ.circ_set_io_dtype(h, dt, dt)
        circ.circ_set_convention(h, convention)
        circ.circ_set_variant(h, variant)
        x = to_device(case.x, case.bf16_io)
        Ho, Wo = case.H + 2 * case.pad - case.r + 1, case.W + 2 * case.pad - case.r + 1
        y = torch.full((case.N, Ho, Wo, case.c_out), float("nan"), device="cuda",
                       dtype=torch.bfloat16 if case.bf16_io else torch.float32)
        circ.circ_conv_forward(h, x, y, case.N, case.H, case.W)
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        used = circ.circ_last_variant(h)
        return y.float().cpu().numpy().astype(np.float64), used
    finally:
        circ.circ_destroy(h)


def oracle_fc(case: synth.FcCase, convention=0, rows=None):
    x = case.x if rows is None else case.x[rows]
    return oracle.fc(case.w, x, bias=case.bias, relu=case.relu, convention=convention)


def oracle_conv(case: synth.ConvCase, convention=0):
    return oracle.conv(case.w, case.x, case.pad, bias=case.bias, relu=case.relu, convention=convention)
