// Pooling layer (Sec. 2.1: subsampling by a max, average or L2-norm over a window; Sec. 4.2: the peripheral computing
// block next to the transforms): x[N][H][W][C] -> y[N][Ho][Wo][C], whole windows only, no padding, each channel on its
// own.  Pure data movement with a comparison or an addition per element: one thread per output pixel and group of
// channels (16 bytes of them: 4 float32 or 8 bfloat16, so that a warp reads whole lines), window taps in a fixed order
// (row by row), float32 arithmetic, bfloat16 results rounded to nearest even.  Overlapping windows (stride < window)
// re-read their pixels from L1 / L2.
#include <cuda_bf16.h>

#include "circ_common.cuh"
#include "circ_io.cuh"

namespace circ {

template <int MODE>
__device__ __forceinline__ float pool_step(float acc, float v) {
    if constexpr (MODE == CIRC_POOL_MAX) return fmaxf(acc, v);
    if constexpr (MODE == CIRC_POOL_AVG) return acc + v;
    return fmaf(v, v, acc);
}
template <int MODE>
__device__ __forceinline__ float pool_finish(float acc, float inv_count) {
    if constexpr (MODE == CIRC_POOL_MAX) return acc;
    if constexpr (MODE == CIRC_POOL_AVG) return acc * inv_count;
    return sqrtf(acc);
}

// VEC channels per thread: 4 (float) / 8 (bfloat16) when C is a multiple of it and both pointers are 16-byte aligned, else 1.
// WIN: the window as a compile-time constant (2, 3: loops unrolled, all taps' loads in flight together) or 0 (runtime).
template <typename T, int VEC, int MODE, int WIN>
__global__ void __launch_bounds__(256) pool_kernel(const T* __restrict__ x, T* __restrict__ y, int H, int W, int C, int Ho, int Wo,
                                                    int window, int stride, float inv_count, long total) {
    const int cv = C / VEC;
    for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int c0 = (int)(idx % cv) * VEC;
        long pix = idx / cv;
        const int j = (int)(pix % Wo);
        pix /= Wo;
        const int i = (int)(pix % Ho);
        const long n = pix / Ho;
        float acc[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] = MODE == CIRC_POOL_MAX ? -INFINITY : 0.f;
        const T* base = x + (((size_t)n * H + (size_t)stride * i) * W + (size_t)stride * j) * C + c0;
        const int win = WIN ? WIN : window;
#pragma unroll
        for (int a = 0; a < win; ++a) {
            const T* row = base + (size_t)a * W * C;
#pragma unroll
            for (int b = 0; b < win; ++b) {
                const T* px = row + (size_t)b * C;
                if constexpr (VEC == 1) {
                    acc[0] = pool_step<MODE>(acc[0], to_float(*px));
                } else if constexpr (sizeof(T) == 4) {
                    const float4 v = __ldg(reinterpret_cast<const float4*>(px));
                    acc[0] = pool_step<MODE>(acc[0], v.x);
                    acc[1] = pool_step<MODE>(acc[1], v.y);
                    acc[2] = pool_step<MODE>(acc[2], v.z);
                    acc[3] = pool_step<MODE>(acc[3], v.w);
                } else {
                    const uint4 v = __ldg(reinterpret_cast<const uint4*>(px));
                    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {     // a bfloat16 is the upper half of a float
                        acc[2 * e] = pool_step<MODE>(acc[2 * e], __uint_as_float(w4[e] << 16));
                        acc[2 * e + 1] = pool_step<MODE>(acc[2 * e + 1], __uint_as_float(w4[e] & 0xffff0000u));
                    }
                }
            }
        }
        T* out = y + (((size_t)n * Ho + i) * Wo + j) * C + c0;
        if constexpr (VEC == 1) {
            store_one(out, pool_finish<MODE>(acc[0], inv_count));
        } else if constexpr (sizeof(T) == 4) {
            *reinterpret_cast<float4*>(out) = make_float4(pool_finish<MODE>(acc[0], inv_count), pool_finish<MODE>(acc[1], inv_count),
                                                          pool_finish<MODE>(acc[2], inv_count), pool_finish<MODE>(acc[3], inv_count));
        } else {
            uint32_t o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(pool_finish<MODE>(acc[2 * e], inv_count), pool_finish<MODE>(acc[2 * e + 1], inv_count));
                o[e] = *reinterpret_cast<const uint32_t*>(&pr);
            }
            *reinterpret_cast<uint4*>(out) = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

template <typename T, int VEC>
static void launch_mode(int mode, const T* x, T* y, int H, int W, int C, int Ho, int Wo, int window, int stride, long total, cudaStream_t s) {
    const long need = (total + 255) / 256;
    const unsigned blocks = (unsigned)(need < 148L * 32 ? need : 148L * 32);
    const float inv = 1.0f / (float)(window * window);
    auto go = [&](auto kernel) { kernel<<<blocks, 256, 0, s>>>(x, y, H, W, C, Ho, Wo, window, stride, inv, total); };
#define CIRC_POOL_WIN(MODE)                                       \
    if (window == 2) go(pool_kernel<T, VEC, MODE, 2>);            \
    else if (window == 3) go(pool_kernel<T, VEC, MODE, 3>);       \
    else go(pool_kernel<T, VEC, MODE, 0>);
    if (mode == CIRC_POOL_MAX) {
        CIRC_POOL_WIN(CIRC_POOL_MAX)
    } else if (mode == CIRC_POOL_AVG) {
        CIRC_POOL_WIN(CIRC_POOL_AVG)
    } else {
        CIRC_POOL_WIN(CIRC_POOL_L2)
    }
#undef CIRC_POOL_WIN
}

}  // namespace circ

using namespace circ;

extern "C" int circ_pool_forward(const void* x, void* y, int N, int H, int W, int C, int window, int stride, int mode, int dtype,
                                 void* stream) {
    if (!x || !y) {
        set_error(CIRC_ERR_ARG, "x or y is NULL");
        return CIRC_ERR_ARG;
    }
    if ((mode != CIRC_POOL_MAX && mode != CIRC_POOL_AVG && mode != CIRC_POOL_L2) || (dtype != CIRC_F32 && dtype != CIRC_BF16)) {
        set_error(CIRC_ERR_ARG, "bad pooling mode %d or element type %d", mode, dtype);
        return CIRC_ERR_ARG;
    }
    if (N < 1 || H < 1 || W < 1 || C < 1 || window < 1 || stride < 1 || window > H || window > W || window > 64) {
        set_error(CIRC_ERR_SHAPE, "bad pooling shape N=%d H=%d W=%d C=%d window=%d stride=%d", N, H, W, C, window, stride);
        return CIRC_ERR_SHAPE;
    }
    const int Ho = (H - window) / stride + 1, Wo = (W - window) / stride + 1;
    const size_t esz = dtype == CIRC_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & (esz - 1)) {
        set_error(CIRC_ERR_ARG, "x and y must be aligned to their element size");
        return CIRC_ERR_ARG;
    }
    const bool aligned16 = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15u) == 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long pixels = (long)N * Ho * Wo;
    if (dtype == CIRC_F32) {
        const float* xf = static_cast<const float*>(x);
        float* yf = static_cast<float*>(y);
        if (aligned16 && C % 4 == 0)
            launch_mode<float, 4>(mode, xf, yf, H, W, C, Ho, Wo, window, stride, pixels * (C / 4), s);
        else
            launch_mode<float, 1>(mode, xf, yf, H, W, C, Ho, Wo, window, stride, pixels * C, s);
    } else {
        const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
        __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(y);
        if (aligned16 && C % 8 == 0)
            launch_mode<__nv_bfloat16, 8>(mode, xb, yb, H, W, C, Ho, Wo, window, stride, pixels * (C / 8), s);
        else
            launch_mode<__nv_bfloat16, 1>(mode, xb, yb, H, W, C, Ho, Wo, window, stride, pixels * C, s);
    }
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}
