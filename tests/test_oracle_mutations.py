"""The pins have teeth: plausible mistakes planted in a COPY of the oracle source make them fail.

Each mutation is a one-token edit of ``oracle/circ_oracle.c`` compiled to a temporary library
(CPU only); the original file and library are never touched.
"""
import ctypes
import subprocess
from pathlib import Path

import numpy as np
import pytest

SRC = Path(__file__).resolve().parent.parent / "oracle" / "circ_oracle.c"
_dp = ctypes.POINTER(ctypes.c_double)

MUTATIONS = {
    "swapped_shift_direction": ("convention == 0 ? r - c : c - r", "convention == 0 ? c - r : r - c"),
    "dropped_column_blocks": ("for (int j = 0; j < q; ++j) {\n                    const double* wij",
                              "for (int j = 0; j < 1; ++j) {\n                    const double* wij"),
    "wrong_block_stride": ("w + ((size_t)i * q + j) * k;\n                    const double* xj",
                           "w + ((size_t)j * p + i) * k;\n                    const double* xj"),
    "flipped_tap": ("int hi = ho + ti - pad;", "int hi = ho - ti + pad;"),
    "transposed_taps": ("((((size_t)ti * r + tj) * p + ib) * q + jb) * k", "((((size_t)tj * r + ti) * p + ib) * q + jb) * k"),
    "relu_on_wrong_side": ("if (relu && acc < 0.0) acc = 0.0;\n                y[", "if (relu && acc > 0.0) acc = 0.0;\n                y["),
}


def _build(tmp_path, name):
    old, new = MUTATIONS[name]
    text = SRC.read_text()
    assert text.count(old) >= 1, f"mutation anchor for {name} not found"
    out = tmp_path / f"{name}.c"
    out.write_text(text.replace(old, new, 1))
    lib = tmp_path / f"{name}.so"
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(lib), str(out), "-lm"], check=True)
    return ctypes.CDLL(str(lib))


def _fc(lib, w, x, bias=None, relu=False, conv=0):
    p, q, k = w.shape
    x = np.ascontiguousarray(np.atleast_2d(x), dtype=np.float64)
    w = np.ascontiguousarray(w, dtype=np.float64)
    y = np.empty((x.shape[0], p * k))
    lib.circ_oracle_fc(p * k, q * k, k, conv, w.ctypes.data_as(_dp), x.ctypes.data_as(_dp),
                       None if bias is None else bias.ctypes.data_as(_dp), int(relu), ctypes.c_long(x.shape[0]),
                       y.ctypes.data_as(_dp))
    return y


def _conv(lib, w, x, pad):
    r, _, p, q, k = w.shape
    N, H, W, C = x.shape
    y = np.empty((N, H + 2 * pad - r + 1, W + 2 * pad - r + 1, p * k))
    lib.circ_oracle_conv(p * k, C, r, pad, k, 0, w.ctypes.data_as(_dp), x.ctypes.data_as(_dp), None, 0, N, H, W,
                         y.ctypes.data_as(_dp))
    return y


def _pins_hold(lib) -> bool:
    """A reduced copy of the pins: hand cases, a 2x3-block library product, ReLU sign, one conv tap."""
    import scipy.linalg
    rng = np.random.default_rng(5)
    ok = True
    ok &= np.array_equal(_fc(lib, np.array([1., 2, 3, 4]).reshape(1, 1, 4), np.array([1., 2, 3, 4]))[0], [26, 28, 26, 20])
    ok &= np.array_equal(_fc(lib, np.array([1., 2, 3, 4]).reshape(1, 2, 2), np.array([1., 0, 0, 1]))[0], [5, 5])
    w = rng.standard_normal((2, 3, 4))
    x = rng.standard_normal((2, 12))
    dense = np.block([[scipy.linalg.circulant(w[i, j]) for j in range(3)] for i in range(2)])
    ok &= np.allclose(_fc(lib, w, x), x @ dense.T, atol=1e-12)
    ok &= np.allclose(_fc(lib, w, x, relu=True), np.maximum(x @ dense.T, 0), atol=1e-12)
    wc = np.zeros((3, 3, 1, 1, 1))
    wc[0, 2] = 1.0
    xc = rng.standard_normal((1, 5, 6, 1))
    ok &= np.array_equal(_conv(lib, wc, xc, 0)[0, :, :, 0], xc[0, 0:3, 2:6, 0])
    wc = np.zeros((3, 3, 1, 1, 1))
    wc[2, 1] = 1.0
    ok &= np.array_equal(_conv(lib, wc, xc, 0)[0, :, :, 0], xc[0, 2:5, 1:5, 0])
    return bool(ok)


def test_unmutated_copy_passes(tmp_path):
    text = SRC.read_text()
    (tmp_path / "plain.c").write_text(text)
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(tmp_path / "plain.so"), str(tmp_path / "plain.c"), "-lm"],
                   check=True)
    assert _pins_hold(ctypes.CDLL(str(tmp_path / "plain.so")))


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(tmp_path, name):
    assert not _pins_hold(_build(tmp_path, name)), f"pins did not notice mutation {name}"


# ---- the backward functions: mistakes planted there must break the finite-difference pins -----------------------
BACKWARD_MUTATIONS = {
    "fc_gx_transposed_block": ("acc += gi[r] * block_entry(wij, k, convention, r, c);", "acc += gi[r] * block_entry(wij, k, convention, c, r);"),
    "fc_gw_swapped_operands": ("out[d] += gi[r] * xj[c];", "out[d] += gi[c] * xj[r];"),
    "conv_gx_unflipped_tap": ("const int ho = h - ti + pad;", "const int ho = h + ti - pad;"),
    "conv_gx_wrong_block": ("acc += block_entry(wv, k, convention, rr, c) * gp[(size_t)ib * k + rr];",
                            "acc += block_entry(wv, k, convention, c, rr) * gp[(size_t)ib * k + rr];"),
    "conv_gw_flipped_tap": ("const int h = ho + ti - pad;", "const int h = ho - ti + pad;"),
    "conv_gw_wrong_diagonal": ("int d = convention == 0 ? rr - cc : cc - rr;", "int d = convention == 0 ? cc - rr : rr - cc;"),
    "conv_gw_dropped_image": ("for (int nn = 0; nn < N; ++nn)\n                    for (int ho", "for (int nn = 0; nn < 1; ++nn)\n                    for (int ho"),
}


def _build_backward(tmp_path, name):
    old, new = BACKWARD_MUTATIONS[name]
    text = SRC.read_text()
    assert text.count(old) == 1, f"mutation anchor for {name} must be unique"
    out = tmp_path / f"{name}.c"
    out.write_text(text.replace(old, new, 1))
    lib = tmp_path / f"{name}.so"
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(lib), str(out), "-lm"], check=True)
    return ctypes.CDLL(str(lib))


def _backward_pins_hold(lib) -> bool:
    """Directional derivatives of L = sum(g * forward) (linear in x and in w, so central differences are exact)."""
    rng = np.random.default_rng(11)
    ok = True
    # fully-connected
    p, q, k, B = 2, 3, 4, 3
    w, x, g = rng.standard_normal((p, q, k)), rng.standard_normal((B, q * k)), rng.standard_normal((B, p * k))
    gx, gw = np.empty((B, q * k)), np.empty((p, q, k))
    lib.circ_oracle_fc_backward(p * k, q * k, k, 0, w.ctypes.data_as(_dp), x.ctypes.data_as(_dp), g.ctypes.data_as(_dp),
                                ctypes.c_long(B), gx.ctypes.data_as(_dp), gw.ctypes.data_as(_dp))
    dx, dw = rng.standard_normal(x.shape), rng.standard_normal(w.shape)
    ok &= np.isclose((g * (_fc(lib, w, x + dx) - _fc(lib, w, x - dx))).sum() / 2, (gx * dx).sum(), atol=1e-9)
    ok &= np.isclose((g * (_fc(lib, w + dw, x) - _fc(lib, w - dw, x))).sum() / 2, (gw * dw).sum(), atol=1e-9)
    # convolution
    r, pad, p, q, k, N, H, W = 3, 1, 2, 2, 4, 2, 4, 3
    w, x, g = rng.standard_normal((r, r, p, q, k)), rng.standard_normal((N, H, W, q * k)), rng.standard_normal((N, H, W, p * k))
    gx, gw = np.empty(x.shape), np.empty(w.shape)
    lib.circ_oracle_conv_backward_input(p * k, q * k, r, pad, k, 0, w.ctypes.data_as(_dp), g.ctypes.data_as(_dp), N, H, W,
                                        gx.ctypes.data_as(_dp))
    lib.circ_oracle_conv_backward_weight(p * k, q * k, r, pad, k, 0, x.ctypes.data_as(_dp), g.ctypes.data_as(_dp), N, H, W,
                                         gw.ctypes.data_as(_dp))
    dx, dw = rng.standard_normal(x.shape), rng.standard_normal(w.shape)
    ok &= np.isclose((g * (_conv(lib, w, x + dx, pad) - _conv(lib, w, x - dx, pad))).sum() / 2, (gx * dx).sum(), atol=1e-9)
    ok &= np.isclose((g * (_conv(lib, w + dw, x, pad) - _conv(lib, w - dw, x, pad))).sum() / 2, (gw * dw).sum(), atol=1e-9)
    return bool(ok)


def test_unmutated_copy_passes_backward_pins(tmp_path):
    (tmp_path / "plain.c").write_text(SRC.read_text())
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(tmp_path / "plain.so"), str(tmp_path / "plain.c"), "-lm"],
                   check=True)
    assert _backward_pins_hold(ctypes.CDLL(str(tmp_path / "plain.so")))


@pytest.mark.parametrize("name", sorted(BACKWARD_MUTATIONS))
def test_planted_backward_mistake_is_caught(tmp_path, name):
    assert not _backward_pins_hold(_build_backward(tmp_path, name)), f"pins did not notice mutation {name}"


# ---- the pooling function: mistakes planted there must break its hand cases ------------------------------------------
POOL_MUTATIONS = {
    "pool_min_instead_of_max": ("acc = v > acc ? v : acc;", "acc = v < acc ? v : acc;"),
    "pool_max_starts_at_zero": ("double acc = mode == 0 ? -INFINITY : 0.0;", "double acc = 0.0;"),
    "pool_stride_ignored_on_rows": ("(size_t)(stride * i + a)) * W", "(size_t)(i + a)) * W"),
    "pool_rows_and_columns_swapped": ("(size_t)(stride * i + a)) * W + (size_t)(stride * j + b)", "(size_t)(stride * j + b)) * W + (size_t)(stride * i + a)"),
    "pool_mean_divides_by_window": ("acc /= (double)(window * window);", "acc /= (double)window;"),
    "pool_window_one_short": ("for (int b = 0; b < window; ++b) {\n                            const double v", "for (int b = 0; b < window - 1; ++b) {\n                            const double v"),
    "pool_l2_without_root": ("if (mode == 2) acc = sqrt(acc);", "if (mode == 2) acc = acc;"),
    "pool_channels_mixed": ("* C + c];\n                            if (mode == 0)", "* C + (C - 1 - c)];\n                            if (mode == 0)"),
}


def _pool_pins_hold(lib) -> bool:
    golden = Path(__file__).resolve().parent / "golden" / "pool_cases.txt"
    ok = True
    for line in golden.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, shape, xs, ys = [part.split() for part in line.split("|")]
        mode, window, stride = (int(v) for v in head)
        H, W, C = (int(v) for v in shape)
        x = np.array(xs, dtype=np.float64)
        want = np.array(ys, dtype=np.float64)
        y = np.full(want.shape, np.nan)
        lib.circ_oracle_pool(mode, window, stride, 1, H, W, C, x.ctypes.data_as(_dp), y.ctypes.data_as(_dp))
        ok &= bool(np.allclose(y, want, rtol=0, atol=1e-12))
    return bool(ok)


def test_unmutated_copy_passes_the_pool_pins(tmp_path):
    (tmp_path / "plain.c").write_text(SRC.read_text())
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(tmp_path / "plain.so"), str(tmp_path / "plain.c"), "-lm"], check=True)
    assert _pool_pins_hold(ctypes.CDLL(str(tmp_path / "plain.so")))


@pytest.mark.parametrize("name", sorted(POOL_MUTATIONS))
def test_planted_pool_mistake_is_caught(tmp_path, name):
    old, new = POOL_MUTATIONS[name]
    text = SRC.read_text()
    assert text.count(old) == 1, f"mutation anchor for {name} must be unique"
    out = tmp_path / f"{name}.c"
    out.write_text(text.replace(old, new, 1))
    lib = tmp_path / f"{name}.so"
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(lib), str(out), "-lm"], check=True)
    assert not _pool_pins_hold(ctypes.CDLL(str(lib))), f"pins did not notice mutation {name}"


# ---- the strided convolution: mistakes planted there must break its hand case -----------------------------------------
STRIDE_MUTATIONS = {
    "stride_ignored_on_columns": ("nn, stride * ho, stride * wo,", "nn, stride * ho, wo,"),
    "stride_rows_and_columns_swapped": ("nn, stride * ho, stride * wo,", "nn, stride * wo, stride * ho,"),
    "stride_extent_without_division": ("const int Ho = (H + 2 * pad - r) / stride + 1, Wo = (W + 2 * pad - r) / stride + 1;\n#pragma omp parallel for collapse(3) schedule(static)\n    for (int nn = 0; nn < N; ++nn)\n        for (int ho = 0; ho < Ho; ++ho)\n            for (int wo = 0; wo < Wo; ++wo)\n                conv_pixel(c_out, c_in, r, pad, k, convention, w, x, bias, relu, H, W, nn, stride * ho",
                                       "const int Ho = (H + 2 * pad - r) / stride + 1, Wo = (W + 2 * pad - r) / stride + 1;\n#pragma omp parallel for collapse(3) schedule(static)\n    for (int nn = 0; nn < N; ++nn)\n        for (int ho = 0; ho < Ho; ++ho)\n            for (int wo = 0; wo < Wo; ++wo)\n                conv_pixel(c_out, c_in, r, pad, k, convention, w, x, bias, relu, H, W, nn, stride * ho + 1"),
}


def _stride_pins_hold(lib) -> bool:
    ok = True
    x = np.arange(12, dtype=np.float64)
    w = np.full(1, 2.0)
    y = np.full(4, np.nan)
    lib.circ_oracle_conv_strided(1, 1, 1, 0, 2, 1, 0, w.ctypes.data_as(_dp), x.ctypes.data_as(_dp), None, 0, 1, 3, 4, y.ctypes.data_as(_dp))
    ok &= bool(np.array_equal(y, [0.0, 4.0, 16.0, 20.0]))
    x = np.arange(16, dtype=np.float64)
    w = np.ones(4)
    y = np.full(4, np.nan)
    lib.circ_oracle_conv_strided(1, 1, 2, 0, 2, 1, 0, w.ctypes.data_as(_dp), x.ctypes.data_as(_dp), None, 0, 1, 4, 4, y.ctypes.data_as(_dp))
    ok &= bool(np.array_equal(y, [10.0, 18.0, 42.0, 50.0]))
    return bool(ok)


def test_unmutated_copy_passes_the_stride_pins(tmp_path):
    (tmp_path / "plain.c").write_text(SRC.read_text())
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(tmp_path / "plain.so"), str(tmp_path / "plain.c"), "-lm"], check=True)
    assert _stride_pins_hold(ctypes.CDLL(str(tmp_path / "plain.so")))


@pytest.mark.parametrize("name", sorted(STRIDE_MUTATIONS))
def test_planted_stride_mistake_is_caught(tmp_path, name):
    old, new = STRIDE_MUTATIONS[name]
    text = SRC.read_text()
    assert text.count(old) == 1, f"mutation anchor for {name} must be unique"
    out = tmp_path / f"{name}.c"
    out.write_text(text.replace(old, new, 1))
    lib = tmp_path / f"{name}.so"
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(lib), str(out), "-lm"], check=True)
    assert not _stride_pins_hold(ctypes.CDLL(str(lib))), f"pins did not notice mutation {name}"
