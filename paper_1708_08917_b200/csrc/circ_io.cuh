// Vector loads / stores of runs of E consecutive elements (float32 or bfloat16 in memory,
// float32 in registers).  bfloat16 stores round to nearest even.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace circ {

template <int E>
__device__ __forceinline__ void load_run(const float* __restrict__ src, float (&out)[E]) {
#pragma unroll
    for (int r = 0; r < E; r += 4) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(src + r));
        out[r] = t.x; out[r + 1] = t.y; out[r + 2] = t.z; out[r + 3] = t.w;
    }
}
template <int E>
__device__ __forceinline__ void load_run(const __nv_bfloat16* __restrict__ src, float (&out)[E]) {
    if constexpr (E % 8 == 0) {
#pragma unroll
        for (int r = 0; r < E; r += 8) {
            const uint4 t = __ldg(reinterpret_cast<const uint4*>(src + r));
            const uint32_t u[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                out[r + 2 * h] = __uint_as_float(u[h] << 16);
                out[r + 2 * h + 1] = __uint_as_float(u[h] & 0xffff0000u);
            }
        }
    } else {  // E == 4
        const uint2 t = __ldg(reinterpret_cast<const uint2*>(src));
        out[0] = __uint_as_float(t.x << 16); out[1] = __uint_as_float(t.x & 0xffff0000u);
        out[2] = __uint_as_float(t.y << 16); out[3] = __uint_as_float(t.y & 0xffff0000u);
    }
}
// The same from shared memory (plain loads: the read-only data path of load_run is for global memory).
template <int E>
__device__ __forceinline__ void load_run_shared(const float* src, float (&out)[E]) {
#pragma unroll
    for (int r = 0; r < E; r += 4) {
        const float4 t = *reinterpret_cast<const float4*>(src + r);
        out[r] = t.x; out[r + 1] = t.y; out[r + 2] = t.z; out[r + 3] = t.w;
    }
}
template <int E>
__device__ __forceinline__ void load_run_shared(const __nv_bfloat16* src, float (&out)[E]) {
    if constexpr (E % 8 == 0) {
#pragma unroll
        for (int r = 0; r < E; r += 8) {
            const uint4 t = *reinterpret_cast<const uint4*>(src + r);
            const uint32_t u[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                out[r + 2 * h] = __uint_as_float(u[h] << 16);
                out[r + 2 * h + 1] = __uint_as_float(u[h] & 0xffff0000u);
            }
        }
    } else {  // E == 4
        const uint2 t = *reinterpret_cast<const uint2*>(src);
        out[0] = __uint_as_float(t.x << 16); out[1] = __uint_as_float(t.x & 0xffff0000u);
        out[2] = __uint_as_float(t.y << 16); out[3] = __uint_as_float(t.y & 0xffff0000u);
    }
}
template <int E>
__device__ __forceinline__ void store_run(float* dst, const float (&v)[E]) {
#pragma unroll
    for (int r = 0; r < E; r += 4) *reinterpret_cast<float4*>(dst + r) = make_float4(v[r], v[r + 1], v[r + 2], v[r + 3]);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);  // round to nearest even
    return *reinterpret_cast<const uint32_t*>(&t);
}
template <int E>
__device__ __forceinline__ void store_run(__nv_bfloat16* dst, const float (&v)[E]) {
    if constexpr (E % 8 == 0) {
#pragma unroll
        for (int r = 0; r < E; r += 8)
            *reinterpret_cast<uint4*>(dst + r) = make_uint4(pack_bf16(v[r], v[r + 1]), pack_bf16(v[r + 2], v[r + 3]),
                                                            pack_bf16(v[r + 4], v[r + 5]), pack_bf16(v[r + 6], v[r + 7]));
    } else {
        *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
    }
}

__device__ __forceinline__ uint32_t bf16_pair(float lo, float hi) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&t);
}
// Split two float32 values into bfloat16 high parts (returned, packed) and low parts (`lo_pair`):
// v = hi + lo up to 2^-17 relative, which is what the three-pass tensor-core product needs.
__device__ __forceinline__ uint32_t bf16_split_pair(float a, float b, uint32_t& lo_pair) {
    const uint32_t hi = bf16_pair(a, b);
    lo_pair = bf16_pair(a - __uint_as_float(hi << 16), b - __uint_as_float(hi & 0xffff0000u));
    return hi;
}

// Single elements (the unaligned paths of embedded block sizes).
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void store_one(float* dst, float v) { *dst = v; }
__device__ __forceinline__ void store_one(__nv_bfloat16* dst, float v) { *dst = __float2bfloat16_rn(v); }

}  // namespace circ
