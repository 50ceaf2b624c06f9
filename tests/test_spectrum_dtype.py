"""bfloat16 weight spectra for the small-batch streaming kernel (the 16-bit spectrum storage of Sec. 4.3)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_BF16, scale_rel_err, to_device

pytestmark = pytest.mark.gpu


def spectrally_rounded(w: np.ndarray) -> np.ndarray:
    """The defining vectors whose spectra are the bfloat16 roundings of the spectra of ``w`` (numpy float64 FFT)."""
    W = np.fft.fft(w.astype(np.float64), axis=-1)
    Wr = synth.round_to_bf16(W.real.astype(np.float32)).astype(np.float64)
    Wi = synth.round_to_bf16(W.imag.astype(np.float32)).astype(np.float64)
    return np.fft.ifft(Wr + 1j * Wi, axis=-1).real


def forward(case, spectrum_dtype, convention=0):
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        if case.bias is not None:
            circ.circ_set_bias(h, case.bias)
        circ.circ_set_activation(h, int(case.relu))
        code = circ.CIRC_BF16 if case.bf16_io else circ.CIRC_F32
        circ.circ_set_io_dtype(h, code, code)
        circ.circ_set_spectrum_dtype(h, spectrum_dtype)   # before the convention: the switch must refresh the rounded copy
        circ.circ_set_convention(h, convention)
        x = to_device(case.x, case.bf16_io)
        y = torch.full((case.batch, case.m), float("nan"), device="cuda", dtype=torch.bfloat16 if case.bf16_io else torch.float32)
        circ.circ_fc_forward(h, x, y, case.batch)
        torch.cuda.synchronize()
        circ.circ_device_status(h)
        assert circ.circ_last_variant(h) == circ.CIRC_VARIANT_FUSED
        return y.float().cpu().numpy().astype(np.float64)
    finally:
        circ.circ_destroy(h)


@pytest.mark.parametrize("m,n,k,batch", [(256, 256, 16, 1), (512, 384, 4, 3), (1024, 2048, 64, 8), (768, 512, 256, 2),
                                         (4096, 4096, 8, 5), (2048, 1024, 128, 1), (96, 160, 32, 7)])
@pytest.mark.parametrize("convention", [0, 1])
def test_bf16_spectra_match_the_layer_of_the_rounded_spectra(m, n, k, batch, convention):
    case = synth.fc_case(f"specbf16_{m}_{n}_{k}_{batch}", m, n, k, batch, w_var=1.0 / n, x_dist="uniform",
                         bias_var=0.01, relu=True)
    got = forward(case, circ.CIRC_BF16, convention)
    exact = oracle.fc(case.w, case.x, bias=case.bias, relu=True, convention=convention)
    rounded = oracle.fc(spectrally_rounded(case.w), case.x, bias=case.bias, relu=True, convention=convention)
    assert scale_rel_err(got, exact) <= TOL_BF16                     # accuracy class of the reduced-precision path
    assert scale_rel_err(got, rounded) <= 2e-4                       # float32 arithmetic on exactly those spectra
    assert scale_rel_err(rounded, exact) > 1e-5                      # the case can tell the two apart ...
    assert scale_rel_err(got, rounded) < 0.2 * scale_rel_err(got, exact)   # ... and the kernel sits on the rounded side


def test_switching_back_restores_float32_spectra():
    case = synth.fc_case("specbf16_back", 512, 512, 16, 2, w_var=1.0 / 512, x_dist="uniform")
    h = circ.circ_fc_create(case.m, case.n, case.k, case.w)
    try:
        x = to_device(case.x, False)
        ys = []
        for dt in (circ.CIRC_F32, circ.CIRC_BF16, circ.CIRC_F32):
            circ.circ_set_spectrum_dtype(h, dt)
            y = torch.empty(case.batch, case.m, device="cuda")
            circ.circ_fc_forward(h, x, y, case.batch)
            torch.cuda.synchronize()
            ys.append(y.cpu().numpy())
        assert np.array_equal(ys[0], ys[2]) and not np.array_equal(ys[0], ys[1])
        assert scale_rel_err(ys[0].astype(np.float64), oracle.fc(case.w, case.x)) <= 1e-4
        with pytest.raises(circ.CircError) as e:
            circ.circ_set_spectrum_dtype(h, 7)
        assert e.value.code == circ.CIRC_ERR_ARG
    finally:
        circ.circ_destroy(h)


def test_bf16_spectra_with_bf16_activations():
    case = synth.fc_case("specbf16_io", 1024, 1024, 16, 4, w_var=1.0 / 1024, x_dist="uniform", bf16_io=True)
    got = forward(case, circ.CIRC_BF16)
    assert scale_rel_err(got, oracle.fc(case.w, case.x)) <= TOL_BF16
