// S0 -- weight-spectrum precompute (once per layer, off the forward path).
//
// The paper keeps FFT(w_ij) in memory instead of w_ij (Sec. 3.1, Sec. 4.2).  This kernel
// evaluates What_ij[g] = (1/k) sum_t w_ij[t] exp(-2 pi i g t / k) for g = 0 .. k/2 directly
// (O(k) per bin, float64, exact argument reduction), folds the inverse transform's 1/k into
// it, conjugates it for circulant convention 1, and writes it in both stored layouts:
//
//   w_stream [tap][i][j][k]      packed half spectrum per block, for the fused streaming kernel:
//                                slot 0 = (Re What[0], Re What[k/2]); slot s = (Re, Im) What[s], 0 < s < k/2
//   a_f32    per problem [M][Kd] embedded real operand of the per-frequency contraction
//                                (layout described in circ_common.cuh)
#include "circ_common.cuh"

namespace circ {

__global__ void precompute_spectra_kernel(const float* __restrict__ w, float* __restrict__ w_stream,
                                          float* __restrict__ a_f32, __nv_bfloat16* __restrict__ a_bf16,
                                          Geometry geo, int convention, long total) {
    const int k = geo.k, p = geo.p, q = geo.q, taps = geo.taps;
    const int bins = k / 2 + 1;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int g = (int)(idx % bins);
        long blk = idx / bins;  // (tap * p + i) * q + j
        const int j = (int)(blk % q);
        const int i = (int)((blk / q) % p);
        const int tap = (int)(blk / ((long)p * q));
        const float* wv = w + blk * geo.ku;     // defining vectors are stored at the caller's block size
        double re = 0.0, im = 0.0;
        // Convention 1 is W[r][c] = w[(c - r) mod ku] = w'[(r - c) mod ku] with w' the index-reversed vector.  At
        // ku == k the reversal is the conjugate spectrum; an embedded block must be reversed before it is padded.
        const bool reverse = convention == 1 && geo.ku != k;
        for (int t = 0; t < geo.ku; ++t) {      // (zero padding up to k adds nothing)
            const int ph = (g * t) & (k - 1);  // exact reduction of g t / k
            double s, c;
            sincospi(-2.0 * (double)ph / (double)k, &s, &c);
            const double wt = (double)wv[reverse && t ? geo.ku - t : t];
            re += wt * c;
            im += wt * s;
        }
        re /= (double)k;
        im /= (double)k;
        if (convention == 1 && !reverse) im = -im;
        if (g == 0 || g == k / 2) im = 0.0;
        const float fre = (float)re, fim = (float)im;

        // packed half spectrum
        float* ws = w_stream + blk * k;
        if (g == 0) {
            ws[0] = fre;
        } else if (g == k / 2) {
            ws[1] = fre;
        } else {
            ws[2 * g] = fre;
            ws[2 * g + 1] = fim;
        }

        // embedded operand
        const int prob = problem_of_bin(g, k);
        const size_t real_sz = (size_t)p * q * taps, cplx_sz = 4 * real_sz;
        const size_t base = problem_offset(prob, real_sz, cplx_sz);
        if (problem_is_real(prob)) {
            const size_t kd = (size_t)q * taps;
            const size_t at = base + (size_t)i * kd + (size_t)tap * q + j;
            if (a_f32) a_f32[at] = fre;
        } else {
            const size_t kd = (size_t)2 * q * taps;
            // rows 2i (real part of the output) and 2i+1 (imaginary part); columns 2j (Re Z) and 2j+1 (Im Z)
            const size_t r0 = base + (size_t)(2 * i) * kd + (size_t)tap * 2 * q;
            const size_t r1 = base + (size_t)(2 * i + 1) * kd + (size_t)tap * 2 * q;
            if (a_f32) {
                a_f32[r0 + 2 * j] = fre;
                a_f32[r0 + 2 * j + 1] = -fim;
                a_f32[r1 + 2 * j] = fim;
                a_f32[r1 + 2 * j + 1] = fre;
            }
        }
        // split bfloat16 operand for the tensor-core contraction: [problem][row][hi|lo][tap][Kq]
        if (a_bf16) {
            const size_t rsz = (size_t)p * taps * 2 * q;  // one real problem, hi and lo
            const size_t b0 = problem_offset(prob, rsz, 4 * rsz);
            auto put = [&](size_t row, int kq, int kk, float val) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(val);
                const __nv_bfloat16 lo = __float2bfloat16_rn(val - __bfloat162float(hi));
                const size_t at = b0 + (row * 2 * taps + (size_t)tap) * kq + kk;
                a_bf16[at] = hi;
                a_bf16[at + (size_t)taps * kq] = lo;
            };
            if (problem_is_real(prob)) {
                put(i, q, j, fre);
            } else {
                put((size_t)2 * i, 2 * q, 2 * j, fre);
                put((size_t)2 * i, 2 * q, 2 * j + 1, -fim);
                put((size_t)2 * i + 1, 2 * q, 2 * j, fim);
                put((size_t)2 * i + 1, 2 * q, 2 * j + 1, fre);
            }
        }
    }
}

// Reduced-precision copy of the streamed spectra (Sec. 4.3 stores 16-bit spectra; here bfloat16, round to nearest even).
__global__ void round_stream_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t count) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = __float2bfloat16_rn(src[i]);
}

int launch_round_stream(Layer* L, cudaStream_t stream) {
    const size_t count = (size_t)L->geo.taps * L->geo.p * L->geo.q * L->geo.k;
    size_t blocks = (count + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    round_stream_kernel<<<(unsigned)blocks, 256, 0, stream>>>(L->w_stream, L->w_stream_bf16, count);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int launch_precompute(Layer* L, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const long total = (long)g.taps * g.p * g.q * (g.k / 2 + 1);
    const int threads = 256;
    long blocks = (total + threads - 1) / threads;
    if (blocks > 148L * 64) blocks = 148L * 64;
    precompute_spectra_kernel<<<(unsigned)blocks, threads, 0, stream>>>(L->w_dev, L->w_stream, L->a_f32, L->a_bf16, g,
                                                                       L->convention, total);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    if (L->w_stream_bf16) return launch_round_stream(L, stream);
    return CIRC_OK;
}

}  // namespace circ
