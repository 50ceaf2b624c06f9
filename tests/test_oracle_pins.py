"""Pins for the CPU oracle: everything here ties ``oracle/`` to something other than itself.

Sources of truth used: hand-computed fixtures (tests/golden), the closed-form
eigenvalues of a circulant matrix, library routines (numpy FFT, numpy matmul,
scipy.linalg.circulant, torch float64 conv2d) and algebraic invariants of the
layer definition (Eq. 1, Eq. 3, Eq. 6, Eq. 7 and the convolution theorem of
Sec. 3.1).  None of these tests touches the CUDA library.
"""
import numpy as np
import pytest
import torch
import scipy.linalg

import oracle

RNG = np.random.default_rng(1708_08917)


def _parse_fields(line):
    return [np.array(f.split(), dtype=np.float64) for f in line.split("|")]


def _hand_cases(golden_dir):
    out = []
    for line in (golden_dir / "hand_cases.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        conv, dims, w, x, y = _parse_fields(line)
        m, n, k = (int(v) for v in dims)
        out.append((int(conv[0]), m, n, k, w.reshape(m // k, n // k, k), x, y))
    return out


def test_hand_cases(golden_dir):
    cases = _hand_cases(golden_dir)
    assert len(cases) >= 15
    for conv, m, n, k, w, x, y in cases:
        got = oracle.fc(w, x, convention=conv)[0]
        assert np.array_equal(got, y), (conv, m, n, k, got, y)


def test_fig1_parameter_count():
    # Fig. 1: an 18-entry 6x3 matrix is represented by two 3x3 circulant blocks = 6 stored parameters.
    w = np.arange(1, 7, dtype=np.float64).reshape(2, 1, 3)
    dense = oracle.expand_matrix(w)
    assert dense.shape == (6, 3) and w.size == 6 and dense.size == 18
    assert len(np.unique(dense)) == 6
    for blk in (dense[:3], dense[3:]):
        for r in range(1, 3):                       # each row is the previous one rotated right (Eq. 7)
            assert np.array_equal(blk[r], np.roll(blk[r - 1], 1))


def test_eigenvalues_closed_form(golden_dir):
    for line in (golden_dir / "eigenvalues.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        kk, w, lre, lim = _parse_fields(line)
        k = int(kk[0])
        lam = lre + 1j * lim
        dre, dim = oracle.dft(w)
        np.testing.assert_allclose(dre + 1j * dim, lam, atol=1e-12)
        t = np.arange(k)
        for conv in (0, 1):
            dense = oracle.expand_block(w, conv)
            for f in range(k):
                v = np.exp(2j * np.pi * f * t / k)
                expect = lam[f] if conv == 0 else np.conj(lam[f])
                np.testing.assert_allclose(dense @ v, expect * v, atol=1e-12)


@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 8, 16, 64])
def test_eigenvalues_random(k):
    w = RNG.standard_normal(k)
    lam = np.fft.fft(w)
    t = np.arange(k)
    dense = oracle.expand_block(w, 0)
    for f in range(k):
        v = np.exp(2j * np.pi * f * t / k)
        np.testing.assert_allclose(dense @ v, lam[f] * v, atol=1e-10)
    dre, dim = oracle.dft(w)
    np.testing.assert_allclose(dre + 1j * dim, lam, atol=1e-10)


@pytest.mark.parametrize("k", [2, 3, 4, 8, 16, 128])
def test_single_block_convolution_theorem(k):
    # Sec. 3.1: W_ij x_j = IFFT(FFT(w_ij) o FFT(x_j)); numpy's FFT is the independent routine.
    w = RNG.standard_normal(k)
    x = RNG.standard_normal(k)
    via_fft = np.fft.ifft(np.fft.fft(w) * np.fft.fft(x)).real
    np.testing.assert_allclose(oracle.fc(w.reshape(1, 1, k), x)[0], via_fft, atol=1e-12)
    corr = np.fft.ifft(np.conj(np.fft.fft(w)) * np.fft.fft(x)).real      # the other convention = correlation
    np.testing.assert_allclose(oracle.fc(w.reshape(1, 1, k), x, convention=1)[0], corr, atol=1e-12)
    # the oracle's own naive DFT agrees with the library one, forward and inverse
    fr, fi = oracle.dft(x)
    np.testing.assert_allclose(fr + 1j * fi, np.fft.fft(x), atol=1e-10)
    br, bi = oracle.dft(fr, fi, sign=+1)
    np.testing.assert_allclose(br / k, x, atol=1e-10)
    np.testing.assert_allclose(bi / k, 0, atol=1e-10)


@pytest.mark.parametrize("p,q,k,batch", [(1, 1, 4, 1), (2, 3, 4, 2), (3, 2, 8, 3), (2, 2, 3, 2), (3, 1, 5, 1),
                                         (1, 3, 1, 2), (4, 5, 16, 3)])
def test_against_library_circulant_and_matmul(p, q, k, batch):
    # scipy.linalg.circulant(c)[r][s] = c[(r-s) mod k]: first COLUMN c -- exactly convention 0;
    # its transpose has first ROW c -- convention 1.
    w = RNG.standard_normal((p, q, k))
    x = RNG.standard_normal((batch, q * k))
    bias = RNG.standard_normal(p * k)
    for conv in (0, 1):
        dense = np.block([[scipy.linalg.circulant(w[i, j]) if conv == 0 else scipy.linalg.circulant(w[i, j]).T
                           for j in range(q)] for i in range(p)])
        np.testing.assert_array_equal(oracle.expand_matrix(w, conv), dense)
        np.testing.assert_allclose(oracle.fc(w, x, convention=conv), x @ dense.T, atol=1e-12)
        np.testing.assert_allclose(oracle.fc(w, x, bias=bias, relu=True, convention=conv),
                                   np.maximum(x @ dense.T + bias, 0.0), atol=1e-12)


def test_block_size_one_is_dense():
    # "no compression if the block size is 1": k=1 is an ordinary dense layer with W = [w_ij].
    p, q = 5, 7
    w = RNG.standard_normal((p, q, 1))
    x = RNG.standard_normal((3, q))
    np.testing.assert_allclose(oracle.fc(w, x), x @ w[:, :, 0].T, atol=1e-13)
    np.testing.assert_allclose(oracle.fc(w, x, convention=1), x @ w[:, :, 0].T, atol=1e-13)


def test_invariants():
    p, q, k, batch = 3, 4, 8, 2
    w = RNG.standard_normal((p, q, k))
    w2 = RNG.standard_normal((p, q, k))
    x = RNG.standard_normal((batch, q * k))
    x2 = RNG.standard_normal((batch, q * k))
    for conv in (0, 1):
        y = oracle.fc(w, x, convention=conv)
        # linearity in x and in w
        np.testing.assert_allclose(oracle.fc(w, 2 * x - 3 * x2, convention=conv),
                                   2 * y - 3 * oracle.fc(w, x2, convention=conv), atol=1e-11)
        np.testing.assert_allclose(oracle.fc(w + w2, x, convention=conv), y + oracle.fc(w2, x, convention=conv),
                                   atol=1e-11)
        # rotating every input block by s rotates every output block by s
        for s in (1, 3):
            xs = np.roll(x.reshape(batch, q, k), s, axis=2).reshape(batch, q * k)
            ys = oracle.fc(w, xs, convention=conv).reshape(batch, p, k)
            np.testing.assert_allclose(ys, np.roll(y.reshape(batch, p, k), s, axis=2), atol=1e-12)
        # DC identity: sum_r a_i[r] = sum_j (sum_t w_ij[t]) (sum_c x_j[c])
        dc = np.einsum("ij,bj->bi", w.sum(axis=2), x.reshape(batch, q, k).sum(axis=2))
        np.testing.assert_allclose(y.reshape(batch, p, k).sum(axis=2), dc, atol=1e-11)
    # the two conventions differ unless the block is symmetric
    assert not np.allclose(oracle.fc(w, x, convention=0), oracle.fc(w, x, convention=1))
    # convention 1 with w equals convention 0 with the index-reversed vector
    wr = np.roll(w[:, :, ::-1], 1, axis=2)
    np.testing.assert_allclose(oracle.fc(w, x, convention=1), oracle.fc(wr, x, convention=0), atol=1e-12)


def _dense_filters(w, k, conv):
    r, _, p, q, _ = w.shape
    F = np.empty((p * k, q * k, r, r))
    for ti in range(r):
        for tj in range(r):
            F[:, :, ti, tj] = np.block([[scipy.linalg.circulant(w[ti, tj, i, j]) if conv == 0
                                         else scipy.linalg.circulant(w[ti, tj, i, j]).T
                                         for j in range(q)] for i in range(p)])
    return F


@pytest.mark.parametrize("r,pad,p,q,k,N,H,W", [(3, 1, 2, 2, 4, 2, 5, 6), (3, 0, 1, 2, 4, 1, 4, 4), (1, 0, 2, 3, 2, 2, 3, 3),
                                               (5, 2, 2, 1, 3, 1, 6, 5), (2, 0, 1, 1, 8, 1, 4, 3)])
def test_conv_against_torch_float64(r, pad, p, q, k, N, H, W):
    # Eq. 6 is a cross-correlation (no flip) over space, summed over input channels: that is what
    # torch.nn.functional.conv2d computes once the filters are expanded to dense form.
    import torch
    w = RNG.standard_normal((r, r, p, q, k))
    x = RNG.standard_normal((N, H, W, q * k))
    bias = RNG.standard_normal(p * k)
    for conv in (0, 1):
        F = _dense_filters(w, k, conv)
        ref = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(F),
                                         bias=torch.from_numpy(bias), padding=pad).permute(0, 2, 3, 1).numpy()
        got = oracle.conv(w, x, pad, bias=bias, convention=conv)
        assert got.shape == (N, H + 2 * pad - r + 1, W + 2 * pad - r + 1, p * k)
        np.testing.assert_allclose(got, ref, atol=1e-11)
        np.testing.assert_allclose(oracle.conv(w, x, pad, bias=bias, relu=True, convention=conv),
                                   np.maximum(ref, 0), atol=1e-11)
        pix = [(0, 0, 0), (N - 1, got.shape[1] - 1, got.shape[2] - 1), (0, got.shape[1] // 2, got.shape[2] - 1)]
        sampled = oracle.conv_pixels(w, x, pad, pix, bias=bias, convention=conv)
        for t, (a, b, c) in enumerate(pix):
            np.testing.assert_allclose(sampled[t], ref[a, b, c], atol=1e-11)


def test_conv_valid_extent_and_tap_orientation():
    # Eq. 6: output extent (W-r+1) x (H-r+1); tap (i,j) multiplies X(x+i-1, y+j-1): a single 1 at tap
    # (0,2) of a 3x3 filter (k=1, one channel) copies the input shifted by (0, +2).
    w = np.zeros((3, 3, 1, 1, 1))
    w[0, 2] = 1.0
    x = RNG.standard_normal((1, 5, 6, 1))
    y = oracle.conv(w, x, pad=0)
    assert y.shape == (1, 3, 4, 1)
    np.testing.assert_array_equal(y[0, :, :, 0], x[0, 0:3, 2:6, 0])


def test_conv_1x1_equals_fc():
    p, q, k = 2, 3, 4
    w = RNG.standard_normal((p, q, k))
    x = RNG.standard_normal((2, 3, 3, q * k))
    y = oracle.conv(w.reshape(1, 1, p, q, k), x, pad=0)
    np.testing.assert_allclose(y.reshape(-1, p * k), oracle.fc(w, x.reshape(-1, q * k)), atol=1e-13)


def test_threads_reported():
    assert oracle.threads() >= 1


# ---- backward pass (Algorithm 2) -------------------------------------------------------------------

@pytest.mark.parametrize("p,q,k,batch", [(1, 1, 4, 1), (2, 3, 4, 2), (3, 2, 8, 3), (2, 2, 3, 2), (1, 3, 1, 2), (4, 5, 16, 3)])
def test_backward_against_dense_transposes(p, q, k, batch):
    # dL/dx = g W (dense expansion from the library circulant) and dL/dw = the sum of g^T x over each diagonal
    w = RNG.standard_normal((p, q, k))
    x = RNG.standard_normal((batch, q * k))
    g = RNG.standard_normal((batch, p * k))
    for conv in (0, 1):
        dense = np.block([[scipy.linalg.circulant(w[i, j]) if conv == 0 else scipy.linalg.circulant(w[i, j]).T
                           for j in range(q)] for i in range(p)])
        gx, gw = oracle.fc_backward(w, x, g, convention=conv)
        np.testing.assert_allclose(gx, g @ dense, atol=1e-12)
        full = g.T @ x                                       # dL/dW of an unstructured layer, m x n
        for i in range(p):
            for j in range(q):
                blk = full[i * k:(i + 1) * k, j * k:(j + 1) * k]
                for d in range(k):
                    # entries (r, c) with (r - c) mod k == d (convention 0) or (c - r) mod k == d (convention 1)
                    r = np.arange(k)
                    c = (r - d) % k if conv == 0 else (r + d) % k
                    assert abs(gw[i, j, d] - blk[r, c].sum()) < 1e-11


def test_backward_is_the_gradient_of_the_forward_oracle():
    # L = sum(g * a) is linear in x and in w, so central differences of the FORWARD oracle are exact up to rounding
    p, q, k, batch = 2, 3, 4, 2
    w = RNG.standard_normal((p, q, k))
    x = RNG.standard_normal((batch, q * k))
    g = RNG.standard_normal((batch, p * k))
    for conv in (0, 1):
        gx, gw = oracle.fc_backward(w, x, g, convention=conv)
        loss = lambda ww, xx: float((g * oracle.fc(ww, xx, convention=conv)).sum())
        h = 1e-3
        for idx in [(0, 0), (1, 5), (0, 11), (1, 7)]:
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            assert abs((loss(w, xp) - loss(w, xm)) / (2 * h) - gx[idx]) < 1e-9
        for idx in [(0, 0, 0), (1, 2, 3), (0, 1, 2), (1, 0, 1)]:
            wp, wm = w.copy(), w.copy()
            wp[idx] += h
            wm[idx] -= h
            assert abs((loss(wp, x) - loss(wm, x)) / (2 * h) - gw[idx]) < 1e-9


@pytest.mark.parametrize("k", [4, 8, 32])
def test_backward_matches_algorithm_2_fft_form(k):
    # Algorithm 2 with numpy's FFT: dL/dw_ij = IFFT(FFT(g_i) o FFT(x'_j)), x' the index-reversed x (FFT(x') = conj FFT(x));
    # dL/dx_j += IFFT(FFT(g_i) o conj(FFT(w_ij)))  -- for the default convention
    p, q, batch = 2, 2, 3
    w = RNG.standard_normal((p, q, k))
    x = RNG.standard_normal((batch, q * k))
    g = RNG.standard_normal((batch, p * k))
    gx, gw = oracle.fc_backward(w, x, g)
    X = np.fft.fft(x.reshape(batch, q, k), axis=2)
    G = np.fft.fft(g.reshape(batch, p, k), axis=2)
    W = np.fft.fft(w, axis=2)
    gw_fft = np.fft.ifft(np.einsum("bif,bjf->ijf", G, np.conj(X)), axis=2).real
    gx_fft = np.fft.ifft(np.einsum("bif,ijf->bjf", G, np.conj(W)), axis=2).real.reshape(batch, q * k)
    np.testing.assert_allclose(gw, gw_fft, atol=1e-10)
    np.testing.assert_allclose(gx, gx_fft, atol=1e-10)


@pytest.mark.parametrize("r,pad,p,q,k,N,H,W", [(3, 1, 2, 2, 4, 2, 5, 6), (3, 0, 1, 2, 4, 1, 4, 5), (1, 0, 2, 3, 2, 2, 3, 3),
                                               (5, 2, 2, 1, 3, 1, 6, 5), (2, 1, 1, 2, 8, 1, 4, 3), (3, 2, 2, 2, 4, 1, 3, 3)])
def test_conv_backward_input_against_torch_autograd(r, pad, p, q, k, N, H, W):
    # gradient of sum(g * conv2d(x, F)) with respect to x, computed by torch's float64 autograd on the dense filters
    import torch
    w = RNG.standard_normal((r, r, p, q, k))
    Ho, Wo = H + 2 * pad - r + 1, W + 2 * pad - r + 1
    g = RNG.standard_normal((N, Ho, Wo, p * k))
    for conv in (0, 1):
        F = torch.from_numpy(_dense_filters(w, k, conv))
        x = torch.zeros(N, q * k, H, W, dtype=torch.float64, requires_grad=True)
        y = torch.nn.functional.conv2d(x, F, padding=pad)
        (y * torch.from_numpy(g).permute(0, 3, 1, 2)).sum().backward()
        ref = x.grad.permute(0, 2, 3, 1).numpy()
        np.testing.assert_allclose(oracle.conv_backward_input(w, g, pad, H, W, convention=conv), ref, atol=1e-11)


def test_conv_backward_input_is_the_gradient_of_the_forward_oracle():
    r, pad, p, q, k, N, H, W = 3, 1, 1, 2, 4, 1, 4, 3
    w = RNG.standard_normal((r, r, p, q, k))
    x = RNG.standard_normal((N, H, W, q * k))
    g = RNG.standard_normal((N, H, W, p * k))
    gx = oracle.conv_backward_input(w, g, pad, H, W)
    h = 1e-3
    for idx in [(0, 0, 0, 0), (0, 3, 2, 7), (0, 1, 1, 4), (0, 2, 0, 5)]:
        xp, xm = x.copy(), x.copy()
        xp[idx] += h
        xm[idx] -= h
        fd = ((g * oracle.conv(w, xp, pad)).sum() - (g * oracle.conv(w, xm, pad)).sum()) / (2 * h)
        assert abs(fd - gx[idx]) < 1e-9


def test_conv_backward_input_is_the_adjoint_of_the_forward_oracle():
    # <conv(x), g> = <x, conv_backward_input(g)> for any x, g: the two maps are transposes of each other
    r, pad, p, q, k, N, H, W = 3, 1, 2, 3, 4, 2, 5, 4
    w = RNG.standard_normal((r, r, p, q, k))
    x = RNG.standard_normal((N, H, W, q * k))
    g = RNG.standard_normal((N, H, W, p * k))
    for conv in (0, 1):
        lhs = (oracle.conv(w, x, pad, convention=conv) * g).sum()
        rhs = (x * oracle.conv_backward_input(w, g, pad, H, W, convention=conv)).sum()
        assert abs(lhs - rhs) < 1e-10 * max(1.0, abs(lhs))


@pytest.mark.parametrize("r,pad,p,q,k,N,H,W", [(3, 1, 2, 2, 4, 2, 5, 6), (3, 0, 1, 2, 4, 1, 4, 5), (1, 0, 2, 3, 2, 2, 3, 3),
                                               (5, 2, 2, 1, 3, 1, 6, 5), (2, 1, 1, 2, 8, 1, 4, 3)])
def test_conv_backward_weight_against_torch_autograd(r, pad, p, q, k, N, H, W):
    # torch's float64 autograd gives dL/dF for the dense filters; the gradient of a defining-vector element is the sum
    # of dL/dF over the entries of the circulant block that hold it (numpy diagonals here, index arithmetic in the oracle)
    import torch
    x = RNG.standard_normal((N, H, W, q * k))
    Ho, Wo = H + 2 * pad - r + 1, W + 2 * pad - r + 1
    g = RNG.standard_normal((N, Ho, Wo, p * k))
    w = RNG.standard_normal((r, r, p, q, k))
    for conv in (0, 1):
        F = torch.from_numpy(_dense_filters(w, k, conv)).requires_grad_(True)
        y = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), F, padding=pad)
        (y * torch.from_numpy(g).permute(0, 3, 1, 2)).sum().backward()
        dF = F.grad.numpy()  # [p*k][q*k][r][r]
        ref = np.zeros((r, r, p, q, k))
        for ti in range(r):
            for tj in range(r):
                for i in range(p):
                    for j in range(q):
                        blk = dF[i * k:(i + 1) * k, j * k:(j + 1) * k, ti, tj]
                        if conv == 1:
                            blk = blk.T
                        # scipy.linalg.circulant(c)[a][b] = c[(a - b) mod k]: element d lies on the wrapped diagonal a - b = d
                        for d in range(k):
                            ref[ti, tj, i, j, d] = np.trace(blk, offset=-d) + (np.trace(blk, offset=k - d) if d else 0.0)
        np.testing.assert_allclose(oracle.conv_backward_weight(x, g, r, pad, k, convention=conv), ref, atol=1e-10)


def test_conv_backward_weight_is_the_gradient_of_the_forward_oracle():
    # L = sum(g * conv(w, x)) is linear in w, so a central difference is exact up to rounding
    r, pad, p, q, k, N, H, W = 3, 1, 2, 2, 4, 2, 4, 3
    w = RNG.standard_normal((r, r, p, q, k))
    x = RNG.standard_normal((N, H, W, q * k))
    g = RNG.standard_normal((N, H, W, p * k))
    gw = oracle.conv_backward_weight(x, g, r, pad, k)
    h = 1e-3
    for idx in [(0, 0, 0, 0, 0), (2, 2, 1, 1, 3), (0, 2, 1, 0, 1), (1, 1, 0, 1, 2), (2, 0, 0, 0, 3)]:
        wp, wm = w.copy(), w.copy()
        wp[idx] += h
        wm[idx] -= h
        fd = ((g * oracle.conv(wp, x, pad)).sum() - (g * oracle.conv(wm, x, pad)).sum()) / (2 * h)
        assert abs(fd - gw[idx]) < 1e-9


def test_conv_backward_weight_one_tap_reduces_to_fc_backward():
    # r = 1: every pixel is a sample of a fully-connected layer
    p, q, k, N, H, W = 2, 3, 4, 2, 3, 2
    x = RNG.standard_normal((N, H, W, q * k))
    g = RNG.standard_normal((N, H, W, p * k))
    w = RNG.standard_normal((p, q, k))
    for conv in (0, 1):
        _, gw_fc = oracle.fc_backward(w, x.reshape(-1, q * k), g.reshape(-1, p * k), convention=conv)
        np.testing.assert_allclose(oracle.conv_backward_weight(x, g, 1, 0, k, convention=conv)[0, 0], gw_fc, atol=1e-11)


# ---- pooling layer (Sec. 2.1, Sec. 4.2) -------------------------------------------------------------------------------
def _pool_cases(golden_dir):
    cases = []
    for line in (golden_dir / "pool_cases.txt").read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, shape, xs, ys = [part.split() for part in line.split("|")]
        mode, window, stride = (int(v) for v in head)
        H, W, C = (int(v) for v in shape)
        cases.append((mode, window, stride, np.array(xs, dtype=np.float64).reshape(1, H, W, C), np.array(ys, dtype=np.float64)))
    return cases


def test_pool_hand_cases(golden_dir):
    cases = _pool_cases(golden_dir)
    assert len(cases) >= 12
    for mode, window, stride, x, want in cases:
        got = oracle.pool(x, window, stride, mode)
        assert got.shape[1] == (x.shape[1] - window) // stride + 1 and got.shape[2] == (x.shape[2] - window) // stride + 1
        np.testing.assert_allclose(got.reshape(-1), want, rtol=0, atol=1e-12)


@pytest.mark.parametrize("N,H,W,C,window,stride", [(2, 13, 13, 5, 3, 2), (1, 28, 28, 3, 2, 2), (3, 9, 11, 4, 3, 1), (1, 7, 5, 2, 5, 3),
                                                   (2, 6, 6, 1, 1, 1), (1, 8, 8, 2, 2, 3)])
def test_pool_against_torch_float64(N, H, W, C, window, stride):
    rng = np.random.default_rng(N * 1000 + H * 10 + window)
    x = rng.standard_normal((N, H, W, C))
    t = torch.from_numpy(x).permute(0, 3, 1, 2)                      # the library routine takes [N][C][H][W]
    want_max = torch.nn.functional.max_pool2d(t, window, stride).permute(0, 2, 3, 1).numpy()
    want_avg = torch.nn.functional.avg_pool2d(t, window, stride).permute(0, 2, 3, 1).numpy()
    want_l2 = torch.nn.functional.lp_pool2d(t, 2.0, window, stride).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(oracle.pool(x, window, stride, oracle.POOL_MAX), want_max)      # a maximum is exact
    np.testing.assert_allclose(oracle.pool(x, window, stride, oracle.POOL_AVG), want_avg, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(oracle.pool(x, window, stride, oracle.POOL_L2), want_l2, rtol=1e-12, atol=1e-13)


def test_pool_invariants():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 10, 9, 3))
    for mode in (oracle.POOL_MAX, oracle.POOL_AVG):
        assert np.array_equal(oracle.pool(x, 1, 1, mode), x)                       # a 1 x 1 window is the identity
    np.testing.assert_allclose(oracle.pool(x, 1, 1, oracle.POOL_L2), np.abs(x), rtol=1e-15)
    assert np.array_equal(oracle.pool(x, 1, 2, oracle.POOL_MAX), x[:, ::2, ::2, :])   # stride alone subsamples
    mx, av, l2 = (oracle.pool(x, 3, 2, m) for m in (oracle.POOL_MAX, oracle.POOL_AVG, oracle.POOL_L2))
    assert (mx >= av).all() and (l2 >= np.abs(av) * 3 - 1e-12).all()                  # max >= mean; ||v||_2 >= sqrt(n) |mean|, n = 9
    c = np.full((1, 6, 6, 2), -2.5)
    assert (oracle.pool(c, 2, 2, oracle.POOL_MAX) == -2.5).all() and (oracle.pool(c, 2, 2, oracle.POOL_AVG) == -2.5).all()
    assert np.allclose(oracle.pool(c, 2, 2, oracle.POOL_L2), 5.0)
    # transposing the image transposes the result (rows and columns are treated alike)
    xt = np.ascontiguousarray(x.transpose(0, 2, 1, 3))
    assert np.array_equal(oracle.pool(xt, 3, 2, oracle.POOL_MAX), oracle.pool(x, 3, 2, oracle.POOL_MAX).transpose(0, 2, 1, 3))


# ---- strided convolution: Eq. 6 kept at every stride-th output position -------------------------------------------------
@pytest.mark.parametrize("r,pad,stride,p,q,k,N,H,W", [(3, 1, 2, 2, 2, 4, 2, 9, 8), (3, 0, 2, 1, 2, 4, 1, 7, 7), (5, 2, 3, 1, 1, 3, 1, 11, 10),
                                                      (1, 0, 2, 2, 1, 2, 2, 5, 4), (3, 1, 4, 1, 1, 2, 1, 13, 6), (2, 0, 2, 1, 1, 4, 1, 5, 8)])
def test_strided_conv_against_torch_float64(r, pad, stride, p, q, k, N, H, W):
    w = RNG.standard_normal((r, r, p, q, k))
    x = RNG.standard_normal((N, H, W, q * k))
    bias = RNG.standard_normal(p * k)
    for conv in (0, 1):
        F = _dense_filters(w, k, conv)
        ref = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(F), bias=torch.from_numpy(bias),
                                         padding=pad, stride=stride).permute(0, 2, 3, 1).numpy()
        got = oracle.conv(w, x, pad, bias=bias, convention=conv, stride=stride)
        assert got.shape == ref.shape == (N, (H + 2 * pad - r) // stride + 1, (W + 2 * pad - r) // stride + 1, p * k)
        np.testing.assert_allclose(got, ref, atol=1e-11)
        # and it is the stride-1 result of Eq. 6 kept at every stride-th position, rows and columns alike
        full = oracle.conv(w, x, pad, bias=bias, convention=conv)
        assert np.array_equal(got, full[:, ::stride, ::stride, :][:, :got.shape[1], :got.shape[2], :])


def test_strided_conv_hand_case():
    # one channel (k = 1 makes the block a scalar), 1 x 1 filter of weight 2, stride 2 on a 3 x 4 image: picks and doubles
    # pixels (0,0), (0,2), (2,0), (2,2); a row index mistaken for a column index would pick others
    x = np.arange(12, dtype=np.float64).reshape(1, 3, 4, 1)
    w = np.full((1, 1, 1, 1, 1), 2.0)
    got = oracle.conv(w, x, 0, stride=2)
    assert got.shape == (1, 2, 2, 1) and np.array_equal(got.reshape(-1), [0.0, 4.0, 16.0, 20.0])
    # 2 x 2 filter of ones, stride 2, no padding: sums of the four 2 x 2 corners of a 4 x 4 image
    x = np.arange(16, dtype=np.float64).reshape(1, 4, 4, 1)
    got = oracle.conv(np.ones((2, 2, 1, 1, 1)), x, 0, stride=2)
    assert np.array_equal(got.reshape(-1), [10.0, 18.0, 42.0, 50.0])
