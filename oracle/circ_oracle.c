/*
 * CPU oracle for block-circulant layers -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.  It shares no code, header, table or constant with the CUDA path.
 *
 * What it computes is the plain definition the fast method must reproduce
 * exactly (up to rounding order):
 *
 *   FC   : y = psi(W x + theta)                         (Eq. 1)
 *          with W cut into p x q circulant k x k blocks  (Eq. 3, Sec. 3.1)
 *   CONV : Y(x,y,p) = sum_{i,j,c} F(i,j,c,p) X(x+i-1, y+j-1, c)   (Eq. 6)
 *          with the channel pair (c,p) of F block-circulant at every tap (Sec. 3.2, Eq. 7)
 *   POOL : max / mean / L2 norm over window x window pixels, per channel   (Sec. 2.1)
 *
 * Every circulant block is expanded element by element from its defining
 * vector; all arithmetic is float64; there is no FFT anywhere in the layer
 * functions.  The naive O(k^2) DFT at the bottom exists only so that tests can
 * check the closed-form eigenvalue property of the expanded blocks.
 *
 * Circulant convention (the paper states "first row vector" and the
 * convolution-theorem product together; they agree in the Y = XF orientation
 * of Sec. 3.2):
 *   convention 0 : W_ij[r][c] = w_ij[(r - c) mod k]   (a_i = sum_j w_ij (*) x_j, circular convolution;
 *                                                       this is what Algorithm 1 computes)
 *   convention 1 : W_ij[r][c] = w_ij[(c - r) mod k]   (w_ij literally the first row with column-vector x)
 *
 * All pins that tie this file to something other than itself live in
 * tests/test_oracle_pins.py; no function here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_API __attribute__((visibility("default")))

/* Entry (r, c), 0 <= r, c < k, of the dense k x k expansion of one circulant block. */
static inline double block_entry(const double* wij, int k, int convention, int r, int c) {
    int d = convention == 0 ? r - c : c - r; /* in (-k, k) */
    if (d < 0) d += k;                       /* d mod k */
    return wij[d];
}

ORACLE_API int circ_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Dense expansion of a single block into dense[k][k] (row-major).  Eq. 3's W_ij. */
ORACLE_API void circ_oracle_expand_block(int k, int convention, const double* wij, double* dense) {
    for (int r = 0; r < k; ++r)
        for (int c = 0; c < k; ++c)
            dense[(size_t)r * k + c] = block_entry(wij, k, convention, r, c);
}

/* Dense expansion of the whole m x n weight matrix (row-major).  Small cases only. */
ORACLE_API void circ_oracle_expand_matrix(int m, int n, int k, int convention, const double* w, double* dense) {
    int p = m / k, q = n / k;
    for (int i = 0; i < p; ++i)
        for (int j = 0; j < q; ++j)
            for (int r = 0; r < k; ++r)
                for (int c = 0; c < k; ++c)
                    dense[((size_t)i * k + r) * n + (size_t)j * k + c] =
                        block_entry(w + ((size_t)i * q + j) * k, k, convention, r, c);
}

/*
 * FC layer, Eq. 1 with the block structure of Eq. 3.
 *   w    [p][q][k]   defining vectors
 *   x    [batch][n]
 *   bias [m] or NULL
 *   y    [batch][m]
 * relu != 0 applies psi(v) = max(0, v).
 */
ORACLE_API void circ_oracle_fc(int m, int n, int k, int convention, const double* w, const double* x,
                               const double* bias, int relu, long batch, double* y) {
    const int p = m / k, q = n / k;
#pragma omp parallel for collapse(2) schedule(static)
    for (long b = 0; b < batch; ++b) {
        for (int i = 0; i < p; ++i) {
            const double* xb = x + (size_t)b * n;
            for (int r = 0; r < k; ++r) {
                double acc = 0.0;
                for (int j = 0; j < q; ++j) {
                    const double* wij = w + ((size_t)i * q + j) * k;
                    const double* xj = xb + (size_t)j * k;
                    for (int c = 0; c < k; ++c) acc += block_entry(wij, k, convention, r, c) * xj[c];
                }
                if (bias) acc += bias[(size_t)i * k + r];
                if (relu && acc < 0.0) acc = 0.0;
                y[(size_t)b * m + (size_t)i * k + r] = acc;
            }
        }
    }
}

/*
 * CONV layer, Eq. 6 (no filter flip, stride 1) with zero padding `pad` on each
 * side, channel-last tensors, and the channel pair block-circulant per tap:
 *   w    [r][r][p][q][k]       p = c_out / k, q = c_in / k
 *   x    [N][H][W][c_in]
 *   y    [N][Ho][Wo][c_out]    Ho = H + 2 pad - r + 1, Wo likewise
 * Tap (i, j) reads input pixel (h + i - pad, w + j - pad); outside the image it reads 0.
 */
/* All c_out outputs of one output pixel (nn, ho, wo); `out` has c_out entries. */
static void conv_pixel(int c_out, int c_in, int r, int pad, int k, int convention, const double* w, const double* x,
                       const double* bias, int relu, int H, int W, int nn, int ho, int wo, double* out) {
    const int p = c_out / k, q = c_in / k;
    for (int ib = 0; ib < p; ++ib) {
        for (int rr = 0; rr < k; ++rr) {
            double acc = 0.0;
            for (int ti = 0; ti < r; ++ti) {
                int hi = ho + ti - pad;
                if (hi < 0 || hi >= H) continue;
                for (int tj = 0; tj < r; ++tj) {
                    int wi = wo + tj - pad;
                    if (wi < 0 || wi >= W) continue;
                    const double* xp = x + (((size_t)nn * H + hi) * W + wi) * c_in;
                    for (int jb = 0; jb < q; ++jb) {
                        const double* wv = w + ((((size_t)ti * r + tj) * p + ib) * q + jb) * k;
                        for (int c = 0; c < k; ++c)
                            acc += block_entry(wv, k, convention, rr, c) * xp[(size_t)jb * k + c];
                    }
                }
            }
            if (bias) acc += bias[(size_t)ib * k + rr];
            if (relu && acc < 0.0) acc = 0.0;
            out[(size_t)ib * k + rr] = acc;
        }
    }
}

ORACLE_API void circ_oracle_conv(int c_out, int c_in, int r, int pad, int k, int convention, const double* w,
                                 const double* x, const double* bias, int relu, int N, int H, int W, double* y) {
    const int Ho = H + 2 * pad - r + 1, Wo = W + 2 * pad - r + 1;
#pragma omp parallel for collapse(3) schedule(static)
    for (int nn = 0; nn < N; ++nn)
        for (int ho = 0; ho < Ho; ++ho)
            for (int wo = 0; wo < Wo; ++wo)
                conv_pixel(c_out, c_in, r, pad, k, convention, w, x, bias, relu, H, W, nn, ho, wo,
                           y + (((size_t)nn * Ho + ho) * Wo + wo) * c_out);
}

/*
 * Strided CONV layer: Eq. 6 evaluated at every `stride`-th output position in both directions (the subsampling
 * convolution of the networks the paper evaluates; Eq. 6 itself is the stride-1 case):
 *   y(n, i, j, :) = [Eq. 6 output](n, stride i, stride j, :),   Ho = (H + 2 pad - r) / stride + 1, Wo likewise.
 */
ORACLE_API void circ_oracle_conv_strided(int c_out, int c_in, int r, int pad, int stride, int k, int convention, const double* w,
                                         const double* x, const double* bias, int relu, int N, int H, int W, double* y) {
    const int Ho = (H + 2 * pad - r) / stride + 1, Wo = (W + 2 * pad - r) / stride + 1;
#pragma omp parallel for collapse(3) schedule(static)
    for (int nn = 0; nn < N; ++nn)
        for (int ho = 0; ho < Ho; ++ho)
            for (int wo = 0; wo < Wo; ++wo)
                conv_pixel(c_out, c_in, r, pad, k, convention, w, x, bias, relu, H, W, nn, stride * ho, stride * wo,
                           y + (((size_t)nn * Ho + ho) * Wo + wo) * c_out);
}

/*
 * The same definition evaluated only at the listed output pixels (for checks at
 * sizes where the whole tensor would take too long): pix[3*t..3*t+2] = (n, ho, wo),
 * y_out[t][c_out].
 */
ORACLE_API void circ_oracle_conv_pixels(int c_out, int c_in, int r, int pad, int k, int convention, const double* w,
                                        const double* x, const double* bias, int relu, int N, int H, int W,
                                        long n_pix, const int* pix, double* y_out) {
    (void)N;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < n_pix; ++t)
        conv_pixel(c_out, c_in, r, pad, k, convention, w, x, bias, relu, H, W, pix[3 * t], pix[3 * t + 1],
                   pix[3 * t + 2], y_out + (size_t)t * c_out);
}

/*
 * FC backward pass (what Algorithm 2 computes with FFTs), written out from the chain rule on
 * a = W x with the block-circulant W of Eq. 3:
 *   dL/dx_j[c]  = sum_i sum_r  g_i[r] * W_ij[r][c]                     (= W^T g)
 *   dL/dw_ij[t] = sum_b sum_{(r,c): W_ij[r][c] is w_ij[t]} g_i^b[r] * x_j^b[c]
 * with g = dL/da ([batch][m]).  Every entry (r, c) of a block holds w_ij[d], d = (r - c) mod k
 * (convention 0) or (c - r) mod k (convention 1), so dL/dw_ij[d] collects g[r] x[c] over that diagonal.
 *   gx [batch][n] and gw [p][q][k] are outputs; either may be NULL to skip it.
 */
ORACLE_API void circ_oracle_fc_backward(int m, int n, int k, int convention, const double* w, const double* x,
                                        const double* g, long batch, double* gx, double* gw) {
    const int p = m / k, q = n / k;
    if (gx) {
#pragma omp parallel for collapse(2) schedule(static)
        for (long b = 0; b < batch; ++b) {
            for (int j = 0; j < q; ++j) {
                for (int c = 0; c < k; ++c) {
                    double acc = 0.0;
                    for (int i = 0; i < p; ++i) {
                        const double* wij = w + ((size_t)i * q + j) * k;
                        const double* gi = g + (size_t)b * m + (size_t)i * k;
                        for (int r = 0; r < k; ++r) acc += gi[r] * block_entry(wij, k, convention, r, c);
                    }
                    gx[(size_t)b * n + (size_t)j * k + c] = acc;
                }
            }
        }
    }
    if (gw) {
#pragma omp parallel for collapse(2) schedule(static)
        for (int i = 0; i < p; ++i) {
            for (int j = 0; j < q; ++j) {
                double* out = gw + ((size_t)i * q + j) * k;
                for (int d = 0; d < k; ++d) out[d] = 0.0;
                for (long b = 0; b < batch; ++b) {
                    const double* gi = g + (size_t)b * m + (size_t)i * k;
                    const double* xj = x + (size_t)b * n + (size_t)j * k;
                    for (int r = 0; r < k; ++r) {
                        for (int c = 0; c < k; ++c) {
                            int d = convention == 0 ? r - c : c - r;
                            if (d < 0) d += k;
                            out[d] += gi[r] * xj[c];
                        }
                    }
                }
            }
        }
    }
}

/*
 * CONV backward pass with respect to the input (the CONV analogue of Algorithm 2's dL/dx line; Sec. 3.2 says the
 * training process "can be formulated in a similar way").  From Eq. 6 with zero padding,
 *   y[n][ho][wo][P] = sum_{ti,tj,c} F(ti,tj,c,P) x[n][ho+ti-pad][wo+tj-pad][c],
 * the chain rule gives
 *   dL/dx[n][h][w][c] = sum_{ti,tj,P} F(ti,tj,c,P) g[n][h-ti+pad][w-tj+pad][P]      (terms outside the output image are 0)
 * with g = dL/dy ([N][Ho][Wo][c_out]) and F(ti,tj,c,P) the dense expansion of the block-circulant channel pair.
 */
ORACLE_API void circ_oracle_conv_backward_input(int c_out, int c_in, int r, int pad, int k, int convention, const double* w,
                                                const double* g, int N, int H, int W, double* gx) {
    const int p = c_out / k, q = c_in / k;
    const int Ho = H + 2 * pad - r + 1, Wo = W + 2 * pad - r + 1;
#pragma omp parallel for collapse(3) schedule(static)
    for (int nn = 0; nn < N; ++nn)
        for (int h = 0; h < H; ++h)
            for (int ww = 0; ww < W; ++ww) {
                double* out = gx + (((size_t)nn * H + h) * W + ww) * c_in;
                for (int jb = 0; jb < q; ++jb)
                    for (int c = 0; c < k; ++c) {
                        double acc = 0.0;
                        for (int ti = 0; ti < r; ++ti) {
                            const int ho = h - ti + pad;
                            if (ho < 0 || ho >= Ho) continue;
                            for (int tj = 0; tj < r; ++tj) {
                                const int wo = ww - tj + pad;
                                if (wo < 0 || wo >= Wo) continue;
                                const double* gp = g + (((size_t)nn * Ho + ho) * Wo + wo) * c_out;
                                for (int ib = 0; ib < p; ++ib) {
                                    const double* wv = w + ((((size_t)ti * r + tj) * p + ib) * q + jb) * k;
                                    for (int rr = 0; rr < k; ++rr)
                                        acc += block_entry(wv, k, convention, rr, c) * gp[(size_t)ib * k + rr];
                                }
                            }
                        }
                        out[(size_t)jb * k + c] = acc;
                    }
            }
}

/*
 * CONV backward pass with respect to the defining vectors (the CONV analogue of Algorithm 2's dL/dw line).
 * Entry (rr, cc) of the dense channel block (i, j) of tap (ti, tj) multiplies x[..][j*k + cc] into y[..][i*k + rr], so
 *   dL/dF(ti,tj)[i*k+rr][j*k+cc] = sum_{n,ho,wo} g[n][ho][wo][i*k+rr] x[n][ho+ti-pad][wo+tj-pad][j*k+cc]
 * (terms whose input pixel lies in the zero padding vanish), and every entry of a circulant block is one element of
 * its defining vector, entry (rr, cc) being w[(rr - cc) mod k] (convention 0) or w[(cc - rr) mod k] (convention 1):
 * dL/dw[ti][tj][i][j][d] is the sum of dL/dF over the entries that hold element d.
 */
ORACLE_API void circ_oracle_conv_backward_weight(int c_out, int c_in, int r, int pad, int k, int convention, const double* x,
                                                 const double* g, int N, int H, int W, double* gw) {
    const int p = c_out / k, q = c_in / k;
    const int Ho = H + 2 * pad - r + 1, Wo = W + 2 * pad - r + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int tap = 0; tap < r * r; ++tap)
        for (int ib = 0; ib < p; ++ib) {
            const int ti = tap / r, tj = tap % r;
            for (int jb = 0; jb < q; ++jb) {
                double* out = gw + (((size_t)tap * p + ib) * q + jb) * k;
                for (int d = 0; d < k; ++d) out[d] = 0.0;
                for (int nn = 0; nn < N; ++nn)
                    for (int ho = 0; ho < Ho; ++ho) {
                        const int h = ho + ti - pad;
                        if (h < 0 || h >= H) continue;
                        for (int wo = 0; wo < Wo; ++wo) {
                            const int ww = wo + tj - pad;
                            if (ww < 0 || ww >= W) continue;
                            const double* gp = g + (((size_t)nn * Ho + ho) * Wo + wo) * c_out + (size_t)ib * k;
                            const double* xp = x + (((size_t)nn * H + h) * W + ww) * c_in + (size_t)jb * k;
                            for (int rr = 0; rr < k; ++rr)
                                for (int cc = 0; cc < k; ++cc) {
                                    int d = convention == 0 ? rr - cc : cc - rr;
                                    if (d < 0) d += k;
                                    out[d] += gp[rr] * xp[cc];
                                }
                        }
                    }
            }
        }
}

/*
 * Pooling layer (Sec. 2.1: subsampling of the extracted features by a max, average or L2-norm over a window; Sec. 4.2:
 * the peripheral computing block): x[N][H][W][C] -> y[N][Ho][Wo][C], Ho = (H - window) / stride + 1 (whole windows
 * only, no padding), y(n, i, j, c) = op over a, b in [0, window) of x(n, stride i + a, stride j + b, c).
 * mode 0: maximum, 1: arithmetic mean, 2: L2 norm (square root of the sum of squares).
 */
ORACLE_API void circ_oracle_pool(int mode, int window, int stride, int N, int H, int W, int C, const double* x, double* y) {
    const int Ho = (H - window) / stride + 1, Wo = (W - window) / stride + 1;
#ifdef _OPENMP
#pragma omp parallel for collapse(2) schedule(static)
#endif
    for (int n = 0; n < N; ++n)
        for (int i = 0; i < Ho; ++i)
            for (int j = 0; j < Wo; ++j)
                for (int c = 0; c < C; ++c) {
                    double acc = mode == 0 ? -INFINITY : 0.0;
                    for (int a = 0; a < window; ++a)
                        for (int b = 0; b < window; ++b) {
                            const double v = x[(((size_t)n * H + (size_t)(stride * i + a)) * W + (size_t)(stride * j + b)) * C + c];
                            if (mode == 0)
                                acc = v > acc ? v : acc;
                            else if (mode == 1)
                                acc += v;
                            else
                                acc += v * v;
                        }
                    if (mode == 1) acc /= (double)(window * window);
                    if (mode == 2) acc = sqrt(acc);
                    y[(((size_t)n * Ho + i) * Wo + j) * C + c] = acc;
                }
}

/*
 * Naive discrete Fourier transform, forward kernel exp(-2 pi i f t / k), unnormalised.
 * Used by tests only, for the eigenvalue closed form (the eigenvalues of a
 * circulant block are the DFT of its defining vector) and for the single-block
 * convolution-theorem identity of Sec. 3.1.  sign = -1 forward, +1 inverse
 * (inverse is also unnormalised; the caller divides by k).
 */
ORACLE_API void circ_oracle_dft(int k, int sign, const double* in_re, const double* in_im, double* out_re,
                                double* out_im) {
    const double two_pi = 6.283185307179586476925286766559;
    for (int f = 0; f < k; ++f) {
        double sr = 0.0, si = 0.0;
        for (int t = 0; t < k; ++t) {
            double ang = sign * two_pi * (double)(((long)f * t) % k) / (double)k;
            double c = cos(ang), s = sin(ang);
            double a = in_re[t], b = in_im ? in_im[t] : 0.0;
            sr += a * c - b * s;
            si += a * s + b * c;
        }
        out_re[f] = sr;
        out_im[f] = si;
    }
}
