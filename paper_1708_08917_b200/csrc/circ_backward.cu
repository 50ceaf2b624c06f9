// Backward pass of the fully-connected layer (Algorithm 2): gradients with respect to the input and
// to the defining vectors, from g = dL/da.
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
        wt[idx] = w[((size_t)i * q + j) * k + ((k - t) & (k - 1))];
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

static int build_transposed(Layer* L) {
    if (L->transposed) return CIRC_OK;
    const int p = L->geo.p, q = L->geo.q, k = L->geo.k;
    float* wt = nullptr;
    const size_t count = (size_t)p * q * k;
    if (cudaMalloc(&wt, count * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        set_error(CIRC_ERR_ALLOC, "allocation of the transposed weights (%zu bytes) failed", count * sizeof(float));
        return CIRC_ERR_ALLOC;
    }
    long blocks = (long)((count + 255) / 256);
    if (blocks > 148L * 32) blocks = 148L * 32;
    transpose_reverse_kernel<<<(unsigned)blocks, 256>>>(L->w_dev, wt, p, q, k);
    count_launches(1);
    Layer* T = nullptr;
    if (cudaDeviceSynchronize() == cudaSuccess) T = make_layer(0, L->n, L->m, k, 1, 1, 0, wt);  // copies wt, computes spectra
    cudaFree(wt);
    if (!T) return circ_last_code() != CIRC_OK ? circ_last_code() : CIRC_ERR_CUDA;
    if (L->convention != 0) {
        T->convention = L->convention;
        int rc = launch_precompute(T, 0);
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
        const size_t x_floats = ((size_t)2 * e.Bh * L->n + 63) & ~(size_t)63;
        const size_t g_floats = ((size_t)2 * e.Bh * L->m + 63) & ~(size_t)63;
        const size_t y_floats = (size_t)2 * Ph * L->n;
        if ((rc = ensure_workspace(L, (x_floats + g_floats + y_floats) * sizeof(float) + 512)) != CIRC_OK) return rc;
        float* xop = static_cast<float*>(L->ws);
        float* gop = xop + x_floats;
        float* yop = gop + g_floats;
        // transforms: x with this layer's geometry (n, q); g with the transposed layer's (its n is m, its q is p)
        if ((rc = launch_input_fft(L, x, xop, 0, e, s)) != CIRC_OK) return rc;
        if ((rc = launch_input_fft(T, grad_a, gop, 0, e, s)) != CIRC_OK) return rc;
        GradWArgs a;
        a.gop = gop; a.xop = xop; a.yop = yop;
        a.p = p; a.q = q; a.k = k; a.cols = 2 * e.Bh; a.Ph = Ph; a.convention = L->convention;
        a.scale = 1.0f / (float)k;
        dim3 grid((q + 15) / 16, (Ph + 15) / 16, num_problems(k));
        grad_w_spectrum_kernel<<<grid, 256, 0, s>>>(a);
        count_launches(1);
        CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
        // inverse transforms over (i, j): "samples" are the p row blocks, "row blocks" the q column blocks,
        // which is the transposed layer's geometry (its m is n, its p is q); no bias, no activation
        Extent ew;
        ew.B = ew.Bo = p;
        ew.Bh = ew.Bho = Ph;
        ew.H = ew.Ho = 1;
        ew.W = ew.Wo = p;
        ew.Nh = Ph;
        if ((rc = launch_output_ifft(T, yop, grad_w, ew, s)) != CIRC_OK) return rc;
    }
    return CIRC_OK;
}

}  // extern "C"
