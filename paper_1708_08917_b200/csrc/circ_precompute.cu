// S0 -- weight-spectrum precompute (once per layer, off the forward path).
//
// The paper keeps FFT(w_ij) in memory instead of w_ij (Sec. 3.1, Sec. 4.2).  precompute_stream_kernel
// evaluates What_ij[g] = (1/k) sum_t w_ij[t] exp(-2 pi i g t / k) for g = 0 .. k/2 directly
// (O(k) per bin, float64, exact argument reduction), folds the inverse transform's 1/k into
// it, conjugates it for circulant convention 1, and writes the one canonical stored form:
//
//   w_stream [tap][i][j][k]      packed half spectrum per block (m n / k floats, the method's storage figure):
//                                slot 0 = (Re What[0], Re What[k/2]); slot s = (Re, Im) What[s], 0 < s < k/2
//
// Every other stored form is a re-arrangement of exactly these float32 values, made by spectrum_forms_kernel
// the first time a kernel variant that reads it runs (circ_api.cu, ensure_forms):
//
//   a_f32    per problem [M][Kd]  embedded real operand [Wr -Wi; Wi Wr] of the FMA contraction (circ_common.cuh)
//   a_bf16   the same as split bfloat16 (hi | lo), [problem][row][hi|lo][tap][Kq], for the tensor cores
//   a_twin   split bfloat16 with every complex value stored ONCE: complex problems have p rows of
//            (Wr, Wi) pairs, [problem][row i][hi|lo][tap][2q]; the contraction then multiplies them with two
//            column groups of X, (Zr, -Zi) for the real part of the result and (Zi, Zr) for the imaginary part
#include "circ_common.cuh"

namespace circ {

__global__ void precompute_stream_kernel(const float* __restrict__ w, float* __restrict__ w_stream, Geometry geo, int convention,
                                         long total) {
    const int k = geo.k, p = geo.p, q = geo.q;
    const int bins = k / 2 + 1;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int g = (int)(idx % bins);
        const long blk = idx / bins;  // (tap * p + i) * q + j
        (void)p; (void)q;
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
        float* ws = w_stream + blk * k;
        if (g == 0) {
            ws[0] = (float)re;
        } else if (g == k / 2) {
            ws[1] = (float)re;
        } else {
            ws[2 * g] = (float)re;
            ws[2 * g + 1] = (float)im;
        }
    }
}

// Packed half spectra -> the operand layouts of the staged contractions (any of the three outputs may be null).
__global__ void spectrum_forms_kernel(const float* __restrict__ w_stream, float* __restrict__ a_f32, __nv_bfloat16* __restrict__ a_bf16,
                                      __nv_bfloat16* __restrict__ a_twin, Geometry geo, long total) {
    const int k = geo.k, p = geo.p, q = geo.q, taps = geo.taps;
    const int bins = k / 2 + 1;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int g = (int)(idx % bins);
        long blk = idx / bins;  // (tap * p + i) * q + j
        const int j = (int)(blk % q);
        const int i = (int)((blk / q) % p);
        const int tap = (int)(blk / ((long)p * q));
        const float* ws = w_stream + blk * k;
        const float fre = g == 0 ? ws[0] : g == k / 2 ? ws[1] : ws[2 * g];
        const float fim = (g == 0 || g == k / 2) ? 0.f : ws[2 * g + 1];

        const int prob = problem_of_bin(g, k);
        if (a_f32) {
            const size_t real_sz = (size_t)p * q * taps, cplx_sz = 4 * real_sz;
            const size_t base = problem_offset(prob, real_sz, cplx_sz);
            if (problem_is_real(prob)) {
                a_f32[base + (size_t)i * q * taps + (size_t)tap * q + j] = fre;
            } else {
                const size_t kd = (size_t)2 * q * taps;
                // rows 2i (real part of the output) and 2i+1 (imaginary part); columns 2j (Re Z) and 2j+1 (Im Z)
                const size_t r0 = base + (size_t)(2 * i) * kd + (size_t)tap * 2 * q;
                const size_t r1 = base + (size_t)(2 * i + 1) * kd + (size_t)tap * 2 * q;
                a_f32[r0 + 2 * j] = fre;
                a_f32[r0 + 2 * j + 1] = -fim;
                a_f32[r1 + 2 * j] = fim;
                a_f32[r1 + 2 * j + 1] = fre;
            }
        }
        // split bfloat16 operands: [problem][row][hi|lo][tap][Kq], runs padded to a multiple of 8 entries (the buffers
        // were zeroed first when that adds entries)
        const int qs = padded_q(q);
        const size_t rsz = (size_t)p * taps * 2 * qs;  // one real problem, hi and lo
        auto put = [&](__nv_bfloat16* a, size_t b0, size_t row, int kq, int kk, float val) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(val);
            const __nv_bfloat16 lo = __float2bfloat16_rn(val - __bfloat162float(hi));
            const size_t at = b0 + (row * 2 * taps + (size_t)tap) * kq + kk;
            a[at] = hi;
            a[at + (size_t)taps * kq] = lo;
        };
        if (a_bf16) {
            const size_t b0 = problem_offset(prob, rsz, 4 * rsz);
            if (problem_is_real(prob)) {
                put(a_bf16, b0, i, qs, j, fre);
            } else {
                put(a_bf16, b0, (size_t)2 * i, 2 * qs, 2 * j, fre);
                put(a_bf16, b0, (size_t)2 * i, 2 * qs, 2 * j + 1, -fim);
                put(a_bf16, b0, (size_t)2 * i + 1, 2 * qs, 2 * j, fim);
                put(a_bf16, b0, (size_t)2 * i + 1, 2 * qs, 2 * j + 1, fre);
            }
        }
        if (a_twin) {
            const size_t b0 = problem_offset(prob, rsz, 2 * rsz);
            if (problem_is_real(prob)) {
                put(a_twin, b0, i, qs, j, fre);
            } else {
                put(a_twin, b0, i, 2 * qs, 2 * j, fre);
                put(a_twin, b0, i, 2 * qs, 2 * j + 1, fim);
            }
        }
    }
}

// Conjugate the packed spectra in place: the other circulant convention of a power-of-two block (w real).
__global__ void conjugate_stream_kernel(float* __restrict__ w_stream, int k, size_t count) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x) {
        const int s = (int)(i % (size_t)k);
        if (s >= 2 && (s & 1)) w_stream[i] = -w_stream[i];
    }
}

// Defining vectors back from the packed spectra of a power-of-two block (float64 sums; the stored spectra are
// float32, so the vectors come back to float32 rounding).  Used when a later call needs w again (the transposed
// layer of the backward pass) after the retained copy was released.
__global__ void defining_vectors_kernel(const float* __restrict__ w_stream, float* __restrict__ w, int k, int convention, size_t count) {
    for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < count; idx += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(idx % (size_t)k);
        const float* ws = w_stream + (idx - t);
        double acc = (double)ws[0] + ((t & 1) ? -(double)ws[1] : (double)ws[1]);
        for (int g = 1; g < k / 2; ++g) {
            const int ph = (g * t) & (k - 1);
            double s, c;
            sincospi(2.0 * (double)ph / (double)k, &s, &c);
            const double im = convention == 1 ? -(double)ws[2 * g + 1] : (double)ws[2 * g + 1];
            acc += 2.0 * ((double)ws[2 * g] * c - im * s);
        }
        w[idx] = (float)acc;
    }
}

// Reduced-precision copy of the streamed spectra (Sec. 4.3 stores 16-bit spectra; here bfloat16, round to nearest even).
__global__ void round_stream_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t count) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = __float2bfloat16_rn(src[i]);
}

static unsigned grid_for(size_t count, int threads) {
    size_t blocks = (count + threads - 1) / threads;
    if (blocks > 148 * 64) blocks = 148 * 64;
    if (blocks < 1) blocks = 1;
    return (unsigned)blocks;
}

int launch_round_stream(Layer* L, cudaStream_t stream) {
    const size_t count = (size_t)L->geo.taps * L->geo.p * L->geo.q * L->geo.k;
    round_stream_kernel<<<grid_for(count, 256), 256, 0, stream>>>(L->w_stream, L->w_stream_bf16, count);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

// w (defining vectors) -> w_stream, and whatever other stored forms the layer already holds.
int launch_precompute(Layer* L, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const long total = (long)g.taps * g.p * g.q * (g.k / 2 + 1);
    precompute_stream_kernel<<<grid_for((size_t)total, 256), 256, 0, stream>>>(L->w_dev, L->w_stream, g, L->convention, total);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return launch_spectrum_forms(L, L->a_f32, L->a_bf16, L->a_twin, stream);
}

// w_stream -> the given operand layouts (null pointers are skipped) and the bfloat16 stream when the layer has one.
int launch_spectrum_forms(Layer* L, float* a_f32, __nv_bfloat16* a_bf16, __nv_bfloat16* a_twin, cudaStream_t stream) {
    const Geometry& g = L->geo;
    if (a_f32 || a_bf16 || a_twin) {
        if (padded_q(g.q) != g.q) {     // the padding entries of the bfloat16 runs are zeros
            if (a_bf16) CIRC_CUDA_TRY(cudaMemsetAsync(a_bf16, 0, bf16_form_elems(L) * sizeof(__nv_bfloat16), stream), CIRC_ERR_CUDA);
            if (a_twin) CIRC_CUDA_TRY(cudaMemsetAsync(a_twin, 0, twin_elems(L) * sizeof(__nv_bfloat16), stream), CIRC_ERR_CUDA);
        }
        const long total = (long)g.taps * g.p * g.q * (g.k / 2 + 1);
        spectrum_forms_kernel<<<grid_for((size_t)total, 256), 256, 0, stream>>>(L->w_stream, a_f32, a_bf16, a_twin, g, total);
        count_launches(1);
        CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    }
    if (L->w_stream_bf16) return launch_round_stream(L, stream);
    return CIRC_OK;
}

int launch_conjugate_stream(Layer* L, cudaStream_t stream) {
    const size_t count = (size_t)L->geo.taps * L->geo.p * L->geo.q * L->geo.k;
    conjugate_stream_kernel<<<grid_for(count, 256), 256, 0, stream>>>(L->w_stream, L->geo.k, count);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int launch_defining_vectors(const Layer* L, float* w_out, cudaStream_t stream) {
    const size_t count = (size_t)L->geo.taps * L->geo.p * L->geo.q * L->geo.k;
    defining_vectors_kernel<<<grid_for(count, 256), 256, 0, stream>>>(L->w_stream, w_out, L->geo.k, L->convention, count);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
