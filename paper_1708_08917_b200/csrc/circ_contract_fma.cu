// S2 / C2 on the float32 FMA pipes: for every problem (frequency bin, see circ_common.cuh)
//     Y[col][row] = sum_kk A[row][kk] * X[col(kk)][kk]
// This is sum_j FFT(w_ij) o FFT(x_j) of Algorithm 1 for all row blocks i at once, written as a
// small dense product per frequency.  For convolutions the contraction index also runs over the
// filter taps, and the column of X is the input pixel the tap points at (zero outside the image):
// Eq. 6 evaluated per frequency, without materialising the unfolded matrix of Sec. 3.2.
//
// Plain shared-memory tiling: 64 x 64 output tile, 16-deep slices, 4 x 4 outputs per thread.
// It is the general fallback; large batches go to the tensor-core contraction instead.
#include "circ_common.cuh"

namespace circ {

constexpr int BM = 64, BN = 64, BK = 16;

struct ContractArgs {
    const float* a;
    const float* x;
    float* y;
    int p, q, k, taps, r, pad;
    int cols_in, cols_out;  // 2*Bh, 2*Bho
    int H, W, Ho, Wo;
    int pdl_late;           // issue the dependent-launch trigger before the stores instead of first thing
};

template <bool CONV>
__global__ void __launch_bounds__(256) contract_fma_kernel(ContractArgs g) {
    if (!g.pdl_late) pdl_trigger();
    pdl_wait();     // X is written by the transform kernel before this one
    const int prob = blockIdx.z;
    const bool real = problem_is_real(prob);
    const int M = real ? g.p : 2 * g.p;
    const int Kq = real ? g.q : 2 * g.q;  // contraction length per tap
    const int Kd = Kq * g.taps;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    if (m0 >= M) return;

    const size_t a_real = (size_t)g.p * g.q * g.taps;
    const float* A = g.a + problem_offset(prob, a_real, 4 * a_real);
    const size_t xin_real = (size_t)g.cols_in * g.q;
    const float* X = g.x + problem_offset(prob, xin_real, 2 * xin_real);
    const size_t y_real = (size_t)g.cols_out * g.p;
    float* Y = g.y + problem_offset(prob, y_real, 2 * y_real);

    __shared__ float As[BK][BM + 4];
    __shared__ float Xs[BK][BN + 4];

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;  // tx -> rows (m), ty -> columns (n)
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    // loader mapping: each thread brings 4 elements of A and 4 of X per slice
    const int lk = tid % BK, lr = tid / BK;  // lr in [0,16)

    // decode the output columns this thread loads for (CONV only)
    int ccol[4], cho[4], cwo[4], cimg[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int col = n0 + lr + 16 * u;
        ccol[u] = col;
        if (CONV) {
            const int hw = g.Ho * g.Wo;
            cimg[u] = col / hw;
            const int rem = col % hw;
            cho[u] = rem / g.Wo;
            cwo[u] = rem % g.Wo;
        }
    }

    for (int k0 = 0; k0 < Kd; k0 += BK) {
        const int kk = k0 + lk;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int row = m0 + lr + 16 * u;
            As[lk][lr + 16 * u] = (row < M && kk < Kd) ? __ldg(A + (size_t)row * Kd + kk) : 0.f;
        }
        int tap = 0, kq = kk;
        if (CONV) {
            tap = kk / Kq;
            kq = kk % Kq;
        }
        const int di = CONV ? tap / g.r - g.pad : 0, dj = CONV ? tap % g.r - g.pad : 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float val = 0.f;
            if (ccol[u] < g.cols_out && kk < Kd) {
                if (CONV) {
                    const int hi = cho[u] + di, wi = cwo[u] + dj;
                    if (hi >= 0 && hi < g.H && wi >= 0 && wi < g.W)
                        val = __ldg(X + ((size_t)cimg[u] * g.H * g.W + (size_t)hi * g.W + wi) * Kq + kq);
                } else {
                    val = __ldg(X + (size_t)ccol[u] * Kq + kq);
                }
            }
            Xs[lk][lr + 16 * u] = val;
        }
        __syncthreads();
#pragma unroll
        for (int s = 0; s < BK; ++s) {
            float av[4], xv[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) av[a] = As[s][tx + 16 * a];
#pragma unroll
            for (int b = 0; b < 4; ++b) xv[b] = Xs[s][ty + 16 * b];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], xv[b], acc[a][b]);
        }
        __syncthreads();
    }
    if (g.pdl_late) pdl_trigger();
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int col = n0 + ty + 16 * b;
        if (col >= g.cols_out) continue;
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int row = m0 + tx + 16 * a;
            if (row < M) Y[(size_t)col * M + row] = acc[a][b];
        }
    }
}

int launch_contract_fma(const Layer* L, const float* xop, float* yop, const Extent& ext, cudaStream_t stream) {
    if (!L->a_f32) {
        set_error(CIRC_ERR_ARG, "the float32 operand of the staged contraction has not been built");
        return CIRC_ERR_ARG;
    }
    ContractArgs g;
    g.a = L->a_f32;
    g.x = xop;
    g.y = yop;
    g.p = L->geo.p; g.q = L->geo.q; g.k = L->geo.k; g.taps = L->geo.taps; g.r = L->geo.r; g.pad = L->geo.pad;
    g.cols_in = 2 * ext.Bh;
    g.cols_out = 2 * ext.Bho;
    g.H = ext.H; g.W = ext.W; g.Ho = ext.Ho; g.Wo = ext.Wo;
    g.pdl_late = dependent_launches() == PDL_LATE;
    dim3 grid((g.cols_out + BN - 1) / BN, (2 * g.p + BM - 1) / BM, num_problems(g.k));
    if (L->kind == 1)
        launch_kernel(dependent_launches(), contract_fma_kernel<true>, grid, dim3(256), 0, stream, g);
    else
        launch_kernel(dependent_launches(), contract_fma_kernel<false>, grid, dim3(256), 0, stream, g);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
