// Backward pass (Algorithm 2): gradients of the fully-connected layer with respect to the input and to
// the defining vectors, from g = dL/da; and the input gradient of the convolution layer, which Sec. 3.2
// says "can be formulated in a similar way": it is the convolution of dL/dy with the flipped taps of the
// transposed (again block-circulant) channel blocks; and its weight gradient, the batch sum below taken
// over pixels with the input moved by each filter tap.
//
//   dL/dx   = W^T g.  W^T is itself block-circulant: its block (j, i) is defined by the index-reversed
//             vector of w_ij, so dL/dx is an ordinary forward pass of the q x p "transposed" layer
//             (kept inside the handle, built on first use), on whichever kernels the planner picks.
//   dL/dw_ij = IFFT( sum_b FFT(g_i^b) o conj(FFT(x_j^b)) )     (the paper's FFT(x'_j) is conj(FFT(x_j)):
//             x' is x with its indices reversed).  Three kernels: forward transforms of x and of g
//             (the same kernel as the forward pass), a per-frequency product summed over the batch,
//             and the inverse-transform kernel of the forward pass run over (i, j) blocks.
//
// Pairing in the batch sum.  The transform kernels carry two samples in one complex transform:
// Z = X_a + i X_b and H = G_a + i G_b.  What the gradient needs is G_a conj(X_a) + G_b conj(X_b),
// which equals ( H conj(Z) + H' conj(Z') ) / 2 with Z' = conj(Z[k - f]), H' = conj(H[k - f]): exactly
// the "mirror" columns the operands already hold.  So for every frequency problem the gradient
// spectrum is a plain sum over ALL columns of the stored operands, G[col][.] * conj(X[col][.]).
#include "circ_common.cuh"

namespace circ {

// w_t[j][i][t] = w[i][j][(-t) mod k]
__global__ void transpose_reverse_kernel(const float* __restrict__ w, float* __restrict__ wt, int p, int q, int k) {
    const long total = (long)p * q * k;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int t = (int)(idx % k);
        const long blk = idx / k;  // j * p + i
        const int i = (int)(blk % p), j = (int)(blk / p);
        wt[idx] = w[((size_t)i * q + j) * k + (t ? k - t : 0)];
    }
}

// CONV: w_t[r-1-ti][r-1-tj][j][i][t] = w[ti][tj][i][j][(-t) mod k]  (taps flipped, channel blocks transposed, vectors reversed)
__global__ void transpose_reverse_conv_kernel(const float* __restrict__ w, float* __restrict__ wt, int r, int p, int q, int k) {
    const long total = (long)r * r * p * q * k;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int t = (int)(idx % k);
        long rest = idx / k;
        const int i = (int)(rest % p);
        rest /= p;
        const int j = (int)(rest % q);
        rest /= q;
        const int tj = (int)(rest % r), ti = (int)(rest / r);     // destination tap
        const int si = r - 1 - ti, sj = r - 1 - tj;               // source tap
        wt[idx] = w[((((size_t)si * r + sj) * p + i) * q + j) * k + (t ? k - t : 0)];
    }
}

// Gradient spectra, written in the layout the inverse-transform kernel reads (circ_common.cuh) with
// the roles "sample" := row block i and "row block" := column block j, so that its output y[i][j*k + t]
// is dL/dw[i][j][t].  Pair c holds row blocks c (real part) and c + Ph (imaginary part), Ph = ceil(p/2):
//   complex problem, column c      : U + i V      U = dWhat_{c,j}[f], V = dWhat_{c+Ph,j}[f]
//                    column Ph + c : U - i V      (the conjugate of bin k - f, as the kernel expects)
//   real problem,    column c : U,  column Ph + c : V.
// One CTA: 16 pairs x 16 column blocks of one problem; the batch columns are walked 16 at a time.
struct GradWArgs {
    const float* gop;  // G operand [problem][col][p | 2p]
    const float* xop;  // X operand [problem][col][q | 2q]
    float* yop;        // output spectra [problem][2*Ph][q | 2q]
    int p, q, k, cols, Ph, convention;
    float scale;       // 1/k (inverse transform) and 1/2 (pairing) for the complex problems are applied here
};

__global__ void __launch_bounds__(256) grad_w_spectrum_kernel(GradWArgs a) {
    const int prob = blockIdx.z;
    const bool real = problem_is_real(prob);
    const int c0 = blockIdx.y * 16, j0 = blockIdx.x * 16;
    const int tc = threadIdx.x / 16, tj = threadIdx.x % 16;
    const int gw_ = real ? a.p : 2 * a.p, xw = real ? a.q : 2 * a.q;
    const float* G = a.gop + problem_offset(prob, (size_t)a.cols * a.p, (size_t)a.cols * 2 * a.p);
    const float* X = a.xop + problem_offset(prob, (size_t)a.cols * a.q, (size_t)a.cols * 2 * a.q);
    const size_t y_real = (size_t)2 * a.Ph * a.q;
    float* Y = a.yop + problem_offset(prob, y_real, 2 * y_real);

    // shared slices: for 16 batch columns, the G entries of the 16 + 16 row blocks and the X entries of the 16 column blocks
    __shared__ float gs[16][2][32];  // [col][half: c | c + Ph][(Re, Im) x 16 row blocks]  (real problems use the first 16)
    __shared__ float xs[16][32];     // [col][(Re, Im) x 16 column blocks]
    const int e = real ? 1 : 2;      // floats per block entry

    float ur = 0.f, ui = 0.f, vr = 0.f, vi = 0.f;
    for (int col0 = 0; col0 < a.cols; col0 += 16) {
        // cooperative loads (zero outside the operands)
        for (int idx = threadIdx.x; idx < 16 * 2 * 16 * e; idx += 256) {
            const int w_in = idx % (16 * e), half = (idx / (16 * e)) % 2, cc = idx / (2 * 16 * e);
            const int col = col0 + cc, blk = c0 + w_in / e + half * a.Ph;
            const bool ok = col < a.cols && (c0 + w_in / e) < a.Ph && blk < a.p;
            gs[cc][half][w_in] = ok ? __ldg(G + (size_t)col * gw_ + (size_t)blk * e + w_in % e) : 0.f;
        }
        for (int idx = threadIdx.x; idx < 16 * 16 * e; idx += 256) {
            const int w_in = idx % (16 * e), cc = idx / (16 * e);
            const int col = col0 + cc, blk = j0 + w_in / e;
            xs[cc][w_in] = (col < a.cols && blk < a.q) ? __ldg(X + (size_t)col * xw + (size_t)blk * e + w_in % e) : 0.f;
        }
        __syncthreads();
        if (real) {
#pragma unroll
            for (int cc = 0; cc < 16; ++cc) {
                const float x = xs[cc][tj];
                ur = fmaf(gs[cc][0][tc], x, ur);
                vr = fmaf(gs[cc][1][tc], x, vr);
            }
        } else {
#pragma unroll
            for (int cc = 0; cc < 16; ++cc) {
                const float xr = xs[cc][2 * tj], xi = xs[cc][2 * tj + 1];
                const float hr = gs[cc][0][2 * tc], hi = gs[cc][0][2 * tc + 1];
                const float kr = gs[cc][1][2 * tc], ki = gs[cc][1][2 * tc + 1];
                // (hr + i hi) * (xr - i xi)
                ur = fmaf(hr, xr, fmaf(hi, xi, ur));
                ui = fmaf(hi, xr, fmaf(-hr, xi, ui));
                vr = fmaf(kr, xr, fmaf(ki, xi, vr));
                vi = fmaf(ki, xr, fmaf(-kr, xi, vi));
            }
        }
        __syncthreads();
    }
    const int c = c0 + tc, j = j0 + tj;
    if (c >= a.Ph || j >= a.q) return;
    if (real) {
        Y[(size_t)c * a.q + j] = a.scale * ur;
        Y[((size_t)a.Ph + c) * a.q + j] = a.scale * vr;
    } else {
        const float s = 0.5f * a.scale;
        if (a.convention == 1) {  // correlation layer: the gradient spectrum is conj(G) * X, the conjugate of the above
            ui = -ui;
            vi = -vi;
        }
        float* y0 = Y + (size_t)c * 2 * a.q + 2 * j;
        float* y1 = Y + ((size_t)a.Ph + c) * 2 * a.q + 2 * j;
        *reinterpret_cast<float2*>(y0) = make_float2(s * (ur - vi), s * (ui + vr));   // U + i V
        *reinterpret_cast<float2*>(y1) = make_float2(s * (ur + vi), s * (ui - vr));   // U - i V
    }
}

// ---- tensor-core route for the batch sum ----------------------------------------------------------
// The product sums over batch columns, so the operands must be contiguous along the columns to be
// "K-major" for the MMA.  This kernel transposes one float32 operand [problem][col][width] into split
// bfloat16 [problem][row][hi | lo][cols_padded] (width = w1 for the two real problems, 2 * w1 for the rest).
__global__ void __launch_bounds__(256) transpose_split_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                              int cols, int cols_padded, int w1) {
    __shared__ float tile[32][33];
    const int prob = blockIdx.z;
    const int width = problem_is_real(prob) ? w1 : 2 * w1;
    const int col0 = blockIdx.x * 32, row0 = blockIdx.y * 32;
    if (row0 >= width) return;
    const float* S = src + problem_offset(prob, (size_t)cols * w1, (size_t)cols * 2 * w1);
    __nv_bfloat16* D = dst + problem_offset(prob, (size_t)w1 * 2 * cols_padded, (size_t)2 * w1 * 2 * cols_padded);
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
    for (int r = ty; r < 32; r += 8) {
        const int col = col0 + r, row = row0 + tx;
        tile[r][tx] = (col < cols && row < width) ? __ldg(S + (size_t)col * width + row) : 0.f;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int row = row0 + r, col = col0 + tx;
        if (row < width && col < cols) {
            const float v = tile[tx][r];
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            __nv_bfloat16* d = D + (size_t)row * 2 * cols_padded + col;
            d[0] = hi;
            d[cols_padded] = __float2bfloat16_rn(v - __bfloat162float(hi));
        }
    }
}

// Turns the products P[a][b] = sum_col G[col][a] X[col][b] (stored transposed, Pt[b][a]) into the gradient
// spectra in the inverse-transform kernel's input layout (see grad_w_spectrum_kernel for the layout).
struct CombineArgs {
    const float* pt_real;  // [2][q][p]
    const float* pt_cplx;  // [k/2-1][2q][2p]
    float* yop;
    int p, q, k, Ph, convention;
    float scale;
};
__global__ void __launch_bounds__(256) grad_w_combine_kernel(CombineArgs a) {
    const int prob = blockIdx.z;
    const int j = blockIdx.x * 32 + threadIdx.x % 32, c = blockIdx.y * 8 + threadIdx.x / 32;
    if (j >= a.q || c >= a.Ph) return;
    const size_t y_real = (size_t)2 * a.Ph * a.q;
    float* Y = a.yop + problem_offset(prob, y_real, 2 * y_real);
    const int i1 = c + a.Ph;
    if (problem_is_real(prob)) {
        const float* P = a.pt_real + (size_t)prob * a.q * a.p + (size_t)j * a.p;
        Y[(size_t)c * a.q + j] = a.scale * P[c];
        Y[((size_t)a.Ph + c) * a.q + j] = i1 < a.p ? a.scale * P[i1] : 0.f;
    } else {
        const float* P = a.pt_cplx + (size_t)(prob - 2) * 4 * a.p * a.q;
        const float* r0 = P + (size_t)(2 * j) * 2 * a.p;      // b = 2j   : P[.][2j]
        const float* r1 = P + (size_t)(2 * j + 1) * 2 * a.p;  // b = 2j+1 : P[.][2j+1]
        const float s = 0.5f * a.scale;
        // U = dWhat of row block c:  Ur = P[2i][2j] + P[2i+1][2j+1],  Ui = P[2i+1][2j] - P[2i][2j+1]
        float ur = r0[2 * c] + r1[2 * c + 1], ui = r0[2 * c + 1] - r1[2 * c];
        float vr = 0.f, vi = 0.f;
        if (i1 < a.p) {
            vr = r0[2 * i1] + r1[2 * i1 + 1];
            vi = r0[2 * i1 + 1] - r1[2 * i1];
        }
        if (a.convention == 1) {
            ui = -ui;
            vi = -vi;
        }
        *reinterpret_cast<float2*>(Y + (size_t)c * 2 * a.q + 2 * j) = make_float2(s * (ur - vi), s * (ui + vr));
        *reinterpret_cast<float2*>(Y + ((size_t)a.Ph + c) * 2 * a.q + 2 * j) = make_float2(s * (ur + vi), s * (ui - vr));
    }
}

// ---- CONV: gradient with respect to the defining vectors -------------------------------------------
// dWhat(tap)_{ij}[f] = sum over output pixels of G[f][pixel][i] * conj(X[f][pixel shifted by the tap][j]): the batch sum of
// the fully-connected case with the pixels as the batch and the X column moved by the tap (input pixels in the
// zero padding contribute nothing).  Channel counts per block grid are small for convolutions (p, q of 4..32), so
// each frequency problem is a skinny product with a very long sum: float32 FMA with the sum split over CTAs.
//
// One CTA (64 threads): one problem, 16 x 16 (i, j) blocks, one filter row a (its R taps b = 0..R-1), a strided
// set ("slice") of output image rows.  Per output row the CTA stages G of that row and the one input row
// ho + a - pad with its R - 1 halo pixels; each thread owns 2 x 2 (i, j) blocks and slides along the row with a
// register window of R input pixels, keeping 4 R complex accumulators.  Partial sums go to
// part[slice][problem][tap][i][j] (float2; real problems use .x), which a second kernel adds up in a fixed order.
struct ConvGradWArgs {
    const float* gop;  // G operand [problem][2 * Bhg][p | 2p], Bhg = Nh * Ho * Wo
    const float* xop;  // X operand [problem][2 * Bhx][q | 2q], Bhx = Nh * H * W
    float2* part;      // [slices][problems][taps][p][q]
    float* yop;        // [problem][2 * St][q | 2q]: the inverse-transform kernel's input
    int p, q, k, r, pad, H, W, Ho, Wo, Nh, St, convention;
    int slices, slices_real;   // row slices of a complex / of a real problem
    int rows;          // 2 * Nh * Ho output rows in all (both column halves)
    float scale;
};

constexpr int kGwRow = 32;   // output pixels staged per step

// One staged row segment: thread (ti, tj) adds G[px][2 ti + u] * conj(X[px + b][2 tj + v]) for all px < cw, b < R.
template <int R>
__device__ __forceinline__ void grad_w_accumulate(bool real, int cw, const float (*gs)[32], const float (*xs)[32], int ti, int tj,
                                                  float (&ar)[R][2][2], float (&ai)[R][2][2]) {
    if (real) {
        float2 win[R];   // win[(px + b) % R] = xs[px + b]
#pragma unroll
        for (int b = 0; b + 1 < R; ++b) win[b] = *reinterpret_cast<const float2*>(&xs[b][2 * tj]);
        for (int px0 = 0; px0 < cw; px0 += R) {
#pragma unroll
            for (int u = 0; u < R; ++u) {
                const int px = px0 + u;
                if (px < cw) {
                    win[(u + R - 1) % R] = *reinterpret_cast<const float2*>(&xs[px + R - 1][2 * tj]);
                    const float2 g = *reinterpret_cast<const float2*>(&gs[px][2 * ti]);
#pragma unroll
                    for (int b = 0; b < R; ++b) {
                        const float2 x = win[(u + b) % R];
                        ar[b][0][0] = fmaf(g.x, x.x, ar[b][0][0]);
                        ar[b][0][1] = fmaf(g.x, x.y, ar[b][0][1]);
                        ar[b][1][0] = fmaf(g.y, x.x, ar[b][1][0]);
                        ar[b][1][1] = fmaf(g.y, x.y, ar[b][1][1]);
                    }
                }
            }
        }
    } else {
        float4 win[R];
#pragma unroll
        for (int b = 0; b + 1 < R; ++b) win[b] = *reinterpret_cast<const float4*>(&xs[b][4 * tj]);
        for (int px0 = 0; px0 < cw; px0 += R) {
#pragma unroll
            for (int u = 0; u < R; ++u) {
                const int px = px0 + u;
                if (px < cw) {
                    win[(u + R - 1) % R] = *reinterpret_cast<const float4*>(&xs[px + R - 1][4 * tj]);
                    const float4 g = *reinterpret_cast<const float4*>(&gs[px][4 * ti]);   // (Re, Im) of two row blocks
#pragma unroll
                    for (int b = 0; b < R; ++b) {
                        const float4 x = win[(u + b) % R];                                 // (Re, Im) of two column blocks
                        // (gr + i gi) * (xr - i xi)
                        ar[b][0][0] = fmaf(g.x, x.x, fmaf(g.y, x.y, ar[b][0][0]));
                        ai[b][0][0] = fmaf(g.y, x.x, fmaf(-g.x, x.y, ai[b][0][0]));
                        ar[b][0][1] = fmaf(g.x, x.z, fmaf(g.y, x.w, ar[b][0][1]));
                        ai[b][0][1] = fmaf(g.y, x.z, fmaf(-g.x, x.w, ai[b][0][1]));
                        ar[b][1][0] = fmaf(g.z, x.x, fmaf(g.w, x.y, ar[b][1][0]));
                        ai[b][1][0] = fmaf(g.w, x.x, fmaf(-g.z, x.y, ai[b][1][0]));
                        ar[b][1][1] = fmaf(g.z, x.z, fmaf(g.w, x.w, ar[b][1][1]));
                        ai[b][1][1] = fmaf(g.w, x.z, fmaf(-g.z, x.w, ai[b][1][1]));
                    }
                }
            }
        }
    }
}

// VEC: p and q are multiples of 4, so every 16-byte piece of an operand row is wholly inside or outside the
// operand; the row segments are then fetched with 128-bit loads into registers one step ahead of the arithmetic.
template <int R, bool VEC>
__global__ void __launch_bounds__(64, R <= 3 ? 8 : 4) conv_grad_w_kernel(ConvGradWArgs a) {
    const int prob = blockIdx.z;
    const bool real = problem_is_real(prob);
    const int e = real ? 1 : 2;
    const int jt = (a.q + 15) / 16;
    const int j0 = (blockIdx.x % jt) * 16, i0 = (blockIdx.x / jt) * 16;
    const int fa = blockIdx.y % a.r;                       // filter row
    const int slice = blockIdx.y / a.r;
    const int nslice = real ? a.slices_real : a.slices;
    if (slice >= nslice) return;                           // the grid is sized for the complex problems
    const int ti = threadIdx.x / 8, tj = threadIdx.x % 8;  // row blocks i0 + 2 ti + {0, 1}, column blocks j0 + 2 tj + {0, 1}
    const int gw_ = e * a.p, xw = e * a.q;
    const size_t Bhg = (size_t)a.Nh * a.Ho * a.Wo, Bhx = (size_t)a.Nh * a.H * a.W;
    const float* G = a.gop + problem_offset(prob, 2 * Bhg * a.p, 2 * Bhg * 2 * a.p);
    const float* X = a.xop + problem_offset(prob, 2 * Bhx * a.q, 2 * Bhx * 2 * a.q);

    __shared__ __align__(16) float gs[kGwRow][32];            // [pixel][(Re, Im) x 16 row blocks]
    __shared__ __align__(16) float xs[kGwRow + R - 1][32];    // [pixel + b][(Re, Im) x 16 column blocks]

    // acc[b][u][v]: tap b, row block 2 ti + u, column block 2 tj + v
    float ar[R][2][2], ai[R][2][2];
#pragma unroll
    for (int b = 0; b < R; ++b)
#pragma unroll
        for (int u = 0; u < 2; ++u) ar[b][u][0] = ar[b][u][1] = ai[b][u][0] = ai[b][u][1] = 0.f;

    // the steps of this CTA: its rows (slice, slice + slices, ...) times the segments of kGwRow output pixels per row
    const int nseg = (a.Wo + kGwRow - 1) / kGwRow;
    const int nstep = ((a.rows - slice + nslice - 1) / nslice) * nseg;
    const float *grow = nullptr, *xrow = nullptr;
    int wo0 = 0, cw = 0;
    // sets grow / xrow / wo0 / cw for step t; false if the step's input row lies in the zero padding (uniform per CTA)
    auto locate = [&](int t) -> bool {
        const int row = slice + (t / nseg) * nslice;
        const int ho = row % a.Ho, img = row / a.Ho;          // img = half * Nh + pair
        const int hi = ho + fa - a.pad;
        if (hi < 0 || hi >= a.H) return false;
        const int half = img / a.Nh, pair = img % a.Nh;
        grow = G + ((size_t)half * Bhg + ((size_t)pair * a.Ho + ho) * a.Wo) * gw_;
        xrow = X + ((size_t)half * Bhx + ((size_t)pair * a.H + hi) * a.W) * xw;
        wo0 = (t % nseg) * kGwRow;
        cw = a.Wo - wo0 < kGwRow ? a.Wo - wo0 : kGwRow;
        return true;
    };

    if constexpr (VEC) {
        constexpr int NV = ((2 * kGwRow + R - 1) * 8 + 63) / 64;   // 16-byte pieces per thread and step, at most
        const int vs = real ? 2 : 3;                                // pieces per pixel: 4 (real) or 8 (complex), as a shift
        float4 v[NV];
        auto fetch = [&](int t) -> bool {
            if (!locate(t)) return false;
            const int ng = cw << vs, nx = (cw + R - 1) << vs;
#pragma unroll
            for (int tt = 0; tt < NV; ++tt) {
                const int idx = threadIdx.x + tt * 64;
                const float* src = nullptr;
                if (idx < ng) {
                    const int px = idx >> vs, off = (idx & ((1 << vs) - 1)) * 4;
                    if (i0 * e + off < gw_) src = grow + (size_t)(wo0 + px) * gw_ + i0 * e + off;
                } else if (idx < ng + nx) {
                    const int id2 = idx - ng, px = id2 >> vs, off = (id2 & ((1 << vs) - 1)) * 4;
                    const int wi = wo0 + px - a.pad;
                    if (wi >= 0 && wi < a.W && j0 * e + off < xw) src = xrow + (size_t)wi * xw + j0 * e + off;
                }
                v[tt] = src ? __ldg(reinterpret_cast<const float4*>(src)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            return true;
        };
        bool cur = nstep > 0 && fetch(0);
        int cur_cw = cw;
        for (int t = 0; t < nstep; ++t) {
            if (cur) {
                const int ng = cur_cw << vs, nx = (cur_cw + R - 1) << vs;
#pragma unroll
                for (int tt = 0; tt < NV; ++tt) {
                    const int idx = threadIdx.x + tt * 64;
                    if (idx < ng)
                        *reinterpret_cast<float4*>(&gs[idx >> vs][(idx & ((1 << vs) - 1)) * 4]) = v[tt];
                    else if (idx < ng + nx)
                        *reinterpret_cast<float4*>(&xs[(idx - ng) >> vs][((idx - ng) & ((1 << vs) - 1)) * 4]) = v[tt];
                }
            }
            __syncthreads();
            const int this_cw = cur_cw;
            const bool was = cur;
            cur = t + 1 < nstep && fetch(t + 1);   // next step's loads fly during the arithmetic
            cur_cw = cw;
            if (was) grad_w_accumulate<R>(real, this_cw, gs, xs, ti, tj, ar, ai);
            __syncthreads();
        }
    } else {
        for (int t = 0; t < nstep; ++t) {
            if (!locate(t)) continue;
            for (int idx = threadIdx.x; idx < cw * 16 * e; idx += 64) {
                const int w_in = idx % (16 * e), px = idx / (16 * e);
                const int blk = i0 + w_in / e;
                gs[px][w_in] = blk < a.p ? __ldg(grow + (size_t)(wo0 + px) * gw_ + (size_t)blk * e + w_in % e) : 0.f;
            }
            for (int idx = threadIdx.x; idx < (cw + R - 1) * 16 * e; idx += 64) {
                const int w_in = idx % (16 * e), px = idx / (16 * e);
                const int wi = wo0 + px - a.pad, blk = j0 + w_in / e;
                xs[px][w_in] = (wi >= 0 && wi < a.W && blk < a.q) ? __ldg(xrow + (size_t)wi * xw + (size_t)blk * e + w_in % e) : 0.f;
            }
            __syncthreads();
            grad_w_accumulate<R>(real, cw, gs, xs, ti, tj, ar, ai);
            __syncthreads();
        }
    }

    const int taps = a.r * a.r;
    float2* P = a.part + ((size_t)slice * gridDim.z + prob) * taps * a.p * a.q;
#pragma unroll
    for (int b = 0; b < R; ++b)
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int i = i0 + 2 * ti + u, j = j0 + 2 * tj;
            if (i >= a.p || j >= a.q) continue;
            float2* dst = P + ((size_t)(fa * R + b) * a.p + i) * a.q + j;
            dst[0] = make_float2(ar[b][u][0], ai[b][u][0]);
            if (j + 1 < a.q) dst[1] = make_float2(ar[b][u][1], ai[b][u][1]);
        }
}

// Adds the slices up (fixed order) and writes the gradient spectra in the input layout of the inverse-transform
// kernel with "sample" s = tap * p + i: samples s < St (St = ceil(taps / 2) * p) are the real parts U of column s,
// samples s + St the imaginary parts V; the kernel wants U + iV in column c and U - iV in the mirror column St + c.
__global__ void __launch_bounds__(256) conv_grad_w_reduce_kernel(ConvGradWArgs a) {
    // block = 32 columns j x 8 slice groups; one sample pair c per block
    const int prob = blockIdx.z, nprob = gridDim.z;
    const int lane = threadIdx.x % 32, grp = threadIdx.x / 32;
    const int j = blockIdx.x * 32 + lane, c = blockIdx.y;
    const int taps = a.r * a.r;
    const size_t per_prob = (size_t)taps * a.p * a.q;
    const bool has_v = c + a.St < taps * a.p;
    __shared__ float4 red[8][32];
    float ur = 0.f, ui = 0.f, vr = 0.f, vi = 0.f;
    if (j < a.q) {
        const float2* pu = a.part + (size_t)prob * per_prob + (size_t)c * a.q + j;            // sample c = (tap, i) in order
        const float2* pv = a.part + (size_t)prob * per_prob + (size_t)(c + a.St) * a.q + j;
        const int nslice = problem_is_real(prob) ? a.slices_real : a.slices;
        for (int sl = grp; sl < nslice; sl += 8) {
            const float2 u = __ldg(pu + (size_t)sl * nprob * per_prob);
            ur += u.x; ui += u.y;
            if (has_v) {
                const float2 v = __ldg(pv + (size_t)sl * nprob * per_prob);
                vr += v.x; vi += v.y;
            }
        }
    }
    red[grp][lane] = make_float4(ur, ui, vr, vi);
    __syncthreads();
    if (grp != 0 || j >= a.q) return;
    for (int g = 1; g < 8; ++g) {
        const float4 t = red[g][lane];
        ur += t.x; ui += t.y; vr += t.z; vi += t.w;
    }
    if (problem_is_real(prob)) {
        float* Y = a.yop + (size_t)prob * 2 * a.St * a.q;
        Y[(size_t)c * a.q + j] = a.scale * ur;
        Y[((size_t)a.St + c) * a.q + j] = a.scale * vr;
    } else {
        float* Y = a.yop + problem_offset(prob, (size_t)2 * a.St * a.q, (size_t)2 * a.St * 2 * a.q);
        const float s = 0.5f * a.scale;
        if (a.convention == 1) {  // correlation layer: the conjugate spectrum
            ui = -ui;
            vi = -vi;
        }
        *reinterpret_cast<float2*>(Y + (size_t)c * 2 * a.q + 2 * j) = make_float2(s * (ur - vi), s * (ui + vr));
        *reinterpret_cast<float2*>(Y + ((size_t)a.St + c) * 2 * a.q + 2 * j) = make_float2(s * (ur + vi), s * (ui - vr));
    }
}

template <int R>
static void launch_conv_grad_w(const ConvGradWArgs& a, dim3 grid, cudaStream_t s) {
    if (a.p % 4 == 0 && a.q % 4 == 0)
        conv_grad_w_kernel<R, true><<<grid, 64, 0, s>>>(a);
    else
        conv_grad_w_kernel<R, false><<<grid, 64, 0, s>>>(a);
}

// CTAs of conv_grad_w_kernel<R, .> that fit on the device at once (one wave); the slower variant's count is used for both
template <int R>
static int conv_grad_w_wave() {
    static int wave = 0;
    if (wave == 0) {
        int dev = 0, sms = 148, b1 = 1, b2 = 1;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b1, conv_grad_w_kernel<R, true>, 64, 0) != cudaSuccess) b1 = 1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2, conv_grad_w_kernel<R, false>, 64, 0) != cudaSuccess) b2 = 1;
        cudaGetLastError();
        const int b = b1 < b2 ? b1 : b2;
        wave = sms * (b > 0 ? b : 1);
    }
    return wave;
}

static int build_transposed(Layer* L) {
    if (L->transposed) return CIRC_OK;
    const int p = L->geo.p, q = L->geo.q, k = L->geo.ku, r = L->geo.r, taps = L->geo.taps;   // the caller's block size: W^T is
    float* wt = nullptr;                                                                       // built from the defining vectors
    const size_t count = (size_t)taps * p * q * k;
    if (dev_alloc(&wt, count * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        set_error(CIRC_ERR_ALLOC, "allocation of the transposed weights (%zu bytes) failed", count * sizeof(float));
        return CIRC_ERR_ALLOC;
    }
    long blocks = (long)((count + 255) / 256);
    if (blocks > 148L * 32) blocks = 148L * 32;
    // the defining vectors: the retained copy (embedded block sizes), else recovered from the stored spectra
    float* w_src = L->w_dev;
    float* w_tmp = nullptr;
    if (!w_src) {
        if (dev_alloc(&w_tmp, count * sizeof(float)) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(wt);
            set_error(CIRC_ERR_ALLOC, "allocation of the defining vectors (%zu bytes) failed", count * sizeof(float));
            return CIRC_ERR_ALLOC;
        }
        // the spectra hold the layer's current convention; the vectors are wanted in the caller's (convention 0) form
        if (launch_defining_vectors(L, w_tmp, 0) != CIRC_OK) {
            cudaFree(wt);
            cudaFree(w_tmp);
            return CIRC_ERR_CUDA;
        }
        w_src = w_tmp;
    }
    if (L->kind == 1)
        transpose_reverse_conv_kernel<<<(unsigned)blocks, 256>>>(w_src, wt, r, p, q, k);
    else
        transpose_reverse_kernel<<<(unsigned)blocks, 256>>>(w_src, wt, p, q, k);
    count_launches(1);
    Layer* T = nullptr;
    // the transposed layer maps c_out -> c_in; a convolution's gradient is a convolution with padding r - 1 - pad
    if (cudaDeviceSynchronize() == cudaSuccess)
        T = make_layer(L->kind, L->n, L->m, k, taps, r, L->kind == 1 ? r - 1 - L->geo.pad : 0, wt);  // copies wt, computes spectra
    cudaFree(wt);
    cudaFree(w_tmp);
    if (!T) return circ_last_code() != CIRC_OK ? circ_last_code() : CIRC_ERR_CUDA;
    T->x_dtype = L->y_dtype;   // the gradient flows from the output side to the input side
    T->y_dtype = L->x_dtype;
    if (L->convention != 0) {
        int rc = circ_set_convention(reinterpret_cast<circ_handle>(T), L->convention);
        if (rc != CIRC_OK || cudaDeviceSynchronize() != cudaSuccess) {
            free_layer(T);
            set_error(CIRC_ERR_CUDA, "spectrum precompute of the transposed layer failed");
            return CIRC_ERR_CUDA;
        }
    }
    L->transposed = T;
    return CIRC_OK;
}

}  // namespace circ

using namespace circ;

extern "C" {

int circ_fc_backward(circ_handle h, const void* x, const void* grad_a, void* grad_x, float* grad_w, int batch, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || L->kind != 0) {
        set_error(CIRC_ERR_ARG, "circ_fc_backward needs a fully-connected handle");
        return CIRC_ERR_ARG;
    }
    if (!grad_a || (!grad_x && !grad_w) || (grad_w && !x) || (reinterpret_cast<uintptr_t>(grad_a) & 15u) ||
        (reinterpret_cast<uintptr_t>(grad_x) & 15u) || (reinterpret_cast<uintptr_t>(grad_w) & 15u) ||
        (reinterpret_cast<uintptr_t>(x) & 15u)) {
        set_error(CIRC_ERR_ARG, "grad_a (and x when grad_w is wanted) must be non-NULL; all pointers 16-byte aligned");
        return CIRC_ERR_ARG;
    }
    if (batch < 1) {
        set_error(CIRC_ERR_SHAPE, "batch=%d must be >= 1", batch);
        return CIRC_ERR_SHAPE;
    }
    if (L->x_dtype != CIRC_F32 || L->y_dtype != CIRC_F32) {
        set_error(CIRC_ERR_UNSUPPORTED, "the backward pass takes float32 tensors only");
        return CIRC_ERR_UNSUPPORTED;
    }
    int rc = build_transposed(L);  // first call: allocates and synchronises
    if (rc != CIRC_OK) return rc;
    Layer* T = L->transposed;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if (grad_x) {  // dL/dx = W^T g: a forward pass of the transposed layer
        if ((rc = circ_fc_forward(reinterpret_cast<circ_handle>(T), grad_a, grad_x, batch, stream)) != CIRC_OK) return rc;
    }
    if (grad_w) {
        const int p = L->geo.p, q = L->geo.q, k = L->geo.k;
        Extent e;
        e.B = e.Bo = batch;
        e.Bh = e.Bho = (batch + 1) / 2;
        e.H = e.Ho = 1;
        e.W = e.Wo = batch;
        e.Nh = e.Bh;
        const int Ph = (p + 1) / 2;
        const int cols = 2 * e.Bh, cols_padded = (cols + 7) & ~7;
        const bool tensor = batch >= 32 && tensor_batch_product_supported(cols);
        const size_t nk = (size_t)q * k, mk = (size_t)p * k;   // widths at the transform size (= n, m unless embedded)
        const size_t x_floats = ((size_t)cols * nk + 63) & ~(size_t)63;
        const size_t g_floats = ((size_t)cols * mk + 63) & ~(size_t)63;
        const size_t y_floats = ((size_t)2 * Ph * nk + 63) & ~(size_t)63;
        // tensor route only: transposed split operands (bfloat16) and the raw products (float32)
        const size_t xt_halves = tensor ? ((nk * 2 * cols_padded + 127) & ~(size_t)127) : 0;
        const size_t gt_halves = tensor ? ((mk * 2 * cols_padded + 127) & ~(size_t)127) : 0;
        const size_t pt_floats = tensor ? (size_t)2 * p * q + (size_t)(k / 2 - 1) * 4 * p * q : 0;
        const size_t need = (x_floats + g_floats + y_floats + pt_floats) * sizeof(float) + (xt_halves + gt_halves) * 2 + 1024;
        if ((rc = ensure_workspace(L, need)) != CIRC_OK) return rc;
        float* xop = static_cast<float*>(L->ws);
        float* gop = xop + x_floats;
        float* yop = gop + g_floats;
        float* pt = yop + y_floats;
        __nv_bfloat16* xt = reinterpret_cast<__nv_bfloat16*>(pt + ((pt_floats + 63) & ~(size_t)63));
        __nv_bfloat16* gt = xt + xt_halves;
        // transforms: x with this layer's geometry (n, q); g with the transposed layer's (its n is m, its q is p)
        if ((rc = launch_input_fft(L, x, xop, 0, e, s)) != CIRC_OK) return rc;
        if ((rc = launch_input_fft(T, grad_a, gop, 0, e, s)) != CIRC_OK) return rc;
        if (tensor) {
            const int nprob = num_problems(k);
            transpose_split_kernel<<<dim3((cols + 31) / 32, (2 * q + 31) / 32, nprob), 256, 0, s>>>(xop, xt, cols, cols_padded, q);
            transpose_split_kernel<<<dim3((cols + 31) / 32, (2 * p + 31) / 32, nprob), 256, 0, s>>>(gop, gt, cols, cols_padded, p);
            count_launches(2);
            CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
            float* pt_real = pt;
            float* pt_cplx = pt + (size_t)2 * p * q;
            if ((rc = launch_tc_batch_product(xt, q, gt, p, k, cols, cols_padded, pt_real, pt_cplx, L->dev_status, s)) != CIRC_OK)
                return rc;
            CombineArgs ca;
            ca.pt_real = pt_real; ca.pt_cplx = pt_cplx; ca.yop = yop;
            ca.p = p; ca.q = q; ca.k = k; ca.Ph = Ph; ca.convention = L->convention;
            ca.scale = 1.0f / (float)k;
            grad_w_combine_kernel<<<dim3((q + 31) / 32, (Ph + 7) / 8, nprob), 256, 0, s>>>(ca);
            count_launches(1);
            CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
        } else {
            GradWArgs a;
            a.gop = gop; a.xop = xop; a.yop = yop;
            a.p = p; a.q = q; a.k = k; a.cols = cols; a.Ph = Ph; a.convention = L->convention;
            a.scale = 1.0f / (float)k;
            dim3 grid((q + 15) / 16, (Ph + 15) / 16, num_problems(k));
            grad_w_spectrum_kernel<<<grid, 256, 0, s>>>(a);
            count_launches(1);
            CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
        }
        // inverse transforms over (i, j): "samples" are the p row blocks, "row blocks" the q column blocks,
        // which is the transposed layer's geometry (its m is n, its p is q); no bias, no activation
        Extent ew;
        ew.B = ew.Bo = p;
        ew.Bh = ew.Bho = Ph;
        ew.H = ew.Ho = 1;
        ew.W = ew.Wo = p;
        ew.Nh = Ph;
        if ((rc = launch_output_ifft(T, yop, grad_w, ew, s, true)) != CIRC_OK) return rc;
    }
    return CIRC_OK;
}

int circ_conv_backward_input(circ_handle h, const void* grad_y, void* grad_x, int N, int H, int W, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || L->kind != 1) {
        set_error(CIRC_ERR_ARG, "circ_conv_backward_input needs a convolution handle");
        return CIRC_ERR_ARG;
    }
    if (reinterpret_cast<Layer*>(h)->geo.stride != 1) {
        set_error(CIRC_ERR_UNSUPPORTED, "the backward passes serve stride 1 only");
        return CIRC_ERR_UNSUPPORTED;
    }
    const int Ho = H + 2 * L->geo.pad - L->geo.r + 1, Wo = W + 2 * L->geo.pad - L->geo.r + 1;
    if (N < 1 || H < 1 || W < 1 || Ho < 1 || Wo < 1) {
        set_error(CIRC_ERR_SHAPE, "bad image extent N=%d H=%d W=%d for r=%d pad=%d", N, H, W, L->geo.r, L->geo.pad);
        return CIRC_ERR_SHAPE;
    }
    int rc = build_transposed(L);  // first call: allocates and synchronises
    if (rc != CIRC_OK) return rc;
    // dL/dx = the transposed layer applied to dL/dy, whose image is Ho x Wo; its padding r - 1 - pad restores H x W
    L->transposed->x_dtype = L->y_dtype;
    L->transposed->y_dtype = L->x_dtype;
    return circ_conv_forward(reinterpret_cast<circ_handle>(L->transposed), grad_y, grad_x, N, Ho, Wo, stream);
}

int circ_conv_backward_weight(circ_handle h, const void* x, const void* grad_y, float* grad_w, int N, int H, int W, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || L->kind != 1) {
        set_error(CIRC_ERR_ARG, "circ_conv_backward_weight needs a convolution handle");
        return CIRC_ERR_ARG;
    }
    if (reinterpret_cast<Layer*>(h)->geo.stride != 1) {
        set_error(CIRC_ERR_UNSUPPORTED, "the backward passes serve stride 1 only");
        return CIRC_ERR_UNSUPPORTED;
    }
    if (!x || !grad_y || !grad_w || (reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(grad_y) & 15u) ||
        (reinterpret_cast<uintptr_t>(grad_w) & 15u)) {
        set_error(CIRC_ERR_ARG, "x, grad_y and grad_w must be non-NULL and 16-byte aligned");
        return CIRC_ERR_ARG;
    }
    const int p = L->geo.p, q = L->geo.q, k = L->geo.k, r = L->geo.r, pad = L->geo.pad, taps = L->geo.taps;
    const int Ho = H + 2 * pad - r + 1, Wo = W + 2 * pad - r + 1;
    if (N < 1 || H < 1 || W < 1 || Ho < 1 || Wo < 1 || (long)N * H * W > (1L << 30) || (long)N * Ho * Wo > (1L << 30)) {
        set_error(CIRC_ERR_SHAPE, "bad image extent N=%d H=%d W=%d for r=%d pad=%d", N, H, W, r, pad);
        return CIRC_ERR_SHAPE;
    }
    if (r > 7) {
        set_error(CIRC_ERR_UNSUPPORTED, "weight gradients are built for filters up to 7 x 7 (r=%d)", r);
        return CIRC_ERR_UNSUPPORTED;
    }
    int rc = build_transposed(L);  // first call: allocates and synchronises
    if (rc != CIRC_OK) return rc;
    Layer* T = L->transposed;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    Extent ex, eg;   // input-side descriptions of x and of grad_y for the transform kernel
    ex.H = ex.Ho = H; ex.W = ex.Wo = W;
    ex.Nh = (N + 1) / 2;
    ex.B = ex.Bo = N * H * W;
    ex.Bh = ex.Bho = ex.Nh * H * W;
    eg = ex;
    eg.H = eg.Ho = Ho; eg.W = eg.Wo = Wo;
    eg.B = eg.Bo = N * Ho * Wo;
    eg.Bh = eg.Bho = eg.Nh * Ho * Wo;
    const int NhT = (taps + 1) / 2, St = NhT * p;
    const size_t nk = (size_t)q * k, mk = (size_t)p * k;   // channel counts at the transform size (= c_in, c_out unless embedded)
    const size_t x_floats = ((size_t)2 * ex.Bh * nk + 63) & ~(size_t)63;
    const size_t g_floats = ((size_t)2 * eg.Bh * mk + 63) & ~(size_t)63;
    const size_t y_floats = ((size_t)2 * St * nk + 63) & ~(size_t)63;
    const int tiles = ((p + 15) / 16) * ((q + 15) / 16), nprob = num_problems(k);
    const int rows = 2 * ex.Nh * Ho;
    // split the pixel sum so that the grid is one full wave of CTAs (a few CTAs more would cost a second wave)
    int wave;
    switch (r) {
        case 1: wave = conv_grad_w_wave<1>(); break;
        case 2: wave = conv_grad_w_wave<2>(); break;
        case 3: wave = conv_grad_w_wave<3>(); break;
        case 4: wave = conv_grad_w_wave<4>(); break;
        case 5: wave = conv_grad_w_wave<5>(); break;
        case 6: wave = conv_grad_w_wave<6>(); break;
        default: wave = conv_grad_w_wave<7>(); break;
    }
    // (giving the cheaper real problems fewer slices, to even out CTA run times, measured slower: their CTAs come
    // first in launch order and the early finishers make room for nothing in a one-wave grid either way)
    const long unit = (long)tiles * r;
    long slices = wave / (unit * nprob);
    if (slices > rows) slices = rows;
    if (slices * r > 65535) slices = 65535 / r;
    if (slices < 1) slices = 1;
    const long slices_real = slices;
    const size_t part_floats = ((size_t)slices * nprob * taps * p * q * 2 + 63) & ~(size_t)63;
    if ((rc = ensure_workspace(L, (x_floats + g_floats + y_floats + part_floats) * sizeof(float) + 1024)) != CIRC_OK) return rc;
    float* xop = static_cast<float*>(L->ws);
    float* gop = xop + x_floats;
    float* yop = gop + g_floats;
    float* part = yop + y_floats;
    T->x_dtype = L->y_dtype;
    if ((rc = launch_input_fft(L, x, xop, 0, ex, s)) != CIRC_OK) return rc;
    if ((rc = launch_input_fft(T, grad_y, gop, 0, eg, s)) != CIRC_OK) return rc;

    ConvGradWArgs a;
    a.gop = gop; a.xop = xop; a.yop = yop;
    a.part = reinterpret_cast<float2*>(part);
    a.p = p; a.q = q; a.k = k; a.r = r; a.pad = pad; a.H = H; a.W = W; a.Ho = Ho; a.Wo = Wo;
    a.Nh = ex.Nh; a.St = St; a.convention = L->convention; a.slices = (int)slices; a.slices_real = (int)slices_real;
    a.rows = rows;
    a.scale = 1.0f / (float)k;
    const dim3 grid((unsigned)tiles, (unsigned)(slices * r), (unsigned)nprob);
    switch (r) {
        case 1: launch_conv_grad_w<1>(a, grid, s); break;
        case 2: launch_conv_grad_w<2>(a, grid, s); break;
        case 3: launch_conv_grad_w<3>(a, grid, s); break;
        case 4: launch_conv_grad_w<4>(a, grid, s); break;
        case 5: launch_conv_grad_w<5>(a, grid, s); break;
        case 6: launch_conv_grad_w<6>(a, grid, s); break;
        default: launch_conv_grad_w<7>(a, grid, s); break;
    }
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    conv_grad_w_reduce_kernel<<<dim3((q + 31) / 32, St, nprob), 256, 0, s>>>(a);
    count_launches(2);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);

    // inverse transforms: "samples" are (tap, row block i), paired s with s + St; "row blocks" are the q column
    // blocks, which is the transposed layer's output geometry; float32 out, no bias, no activation
    Extent ew;
    ew.B = ew.Bo = taps * p;
    ew.Bh = ew.Bho = St;
    ew.H = ew.Ho = 1;
    ew.W = ew.Wo = taps * p;
    ew.Nh = St;
    const int keep = T->y_dtype;
    T->y_dtype = CIRC_F32;
    rc = launch_output_ifft(T, yop, grad_w, ew, s, true);
    T->y_dtype = keep;
    return rc;
}

}  // extern "C"
