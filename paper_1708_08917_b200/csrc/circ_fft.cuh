// Register / warp-shuffle complex FFTs of size K = 4 .. 1024 (powers of two).
//
// The layer needs real transforms of real signals (Sec. 4.1: real inputs give a
// conjugate-symmetric spectrum, so half of it is redundant).  That redundancy is
// used here in its classical equivalent form: two real signals u, v are carried
// through ONE complex transform as z = u + i v.  Multiplying the spectrum of z
// by the spectrum of a real weight vector and transforming back gives
// (w (*) u) + i (w (*) v), so no split / merge pass is ever needed and the
// butterfly count per real signal is that of a half-size complex transform.
//
// A transform of size K is spread over L lanes of a warp, E points per lane
// (K = L * E, E <= 16; sizes above 512 take E = K / 32 so that L stays one warp: the larger block is
// built from the same small in-register transform plus more cross-lane butterfly levels, Sec. 4.1).  Lane l holds the contiguous samples z[E*l .. E*l+E-1],
// so global loads and stores are 16-byte vectors.  With f = f2 + L*f1:
//
//   Z[f2 + L f1] = sum_r w_E^(r f1) * [ w_K^(r f2) * ( sum_l w_L^(l f2) z[E l + r] ) ]
//
//   forward : (1) size-L decimation-in-frequency FFT across lanes, one xor-shuffle
//                 butterfly level per stage (the recursive halving of Sec. 4.1)
//             (2) twiddle w_K^(r f2)     (3) size-E FFT inside the thread's registers
//   inverse : the same three steps undone in reverse order with conjugate twiddles.
//
// The cross-lane stage leaves lane order bit-reversed: lane s of a group holds
// f2 = bitrev_L(s).  Nothing reorders it, because the inverse transform starts
// from that same placement; the products in between are pointwise.
// Neither direction normalises: the 1/K lives in the stored weight spectra.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace circ {

// EMAX bounds the points per lane.  16 keeps the shuffle count low (throughput); a small EMAX spreads a
// transform over more lanes, which shortens every thread's dependent chain when the whole problem is
// too small to fill the machine (latency).
template <int K, int EMAX = 16>
struct FftShape {
    static_assert(K >= 4 && K <= 1024 && (K & (K - 1)) == 0, "block size must be a power of two in [4,1024]");
    static_assert(EMAX == 4 || EMAX == 8 || EMAX == 16, "points per lane: 4, 8 or 16");
    static constexpr int E = K / 32 > EMAX ? K / 32 : (K < EMAX ? K : EMAX);  // points per lane (at most 32 lanes)
    static constexpr int L = K / E;                // lanes per transform
    static_assert(L <= 32, "a transform must fit one warp");
    static constexpr int LOG_L = L == 1 ? 0 : L == 2 ? 1 : L == 4 ? 2 : L == 8 ? 3 : L == 16 ? 4 : 5;
};

__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
// a * conj(b)
__device__ __forceinline__ float2 cmulc(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, a.y * b.y), fmaf(a.y, b.x, -a.x * b.y));
}

// Multiply by exp(-+ 2 pi i IDX / 16) with the trivial cases resolved at compile time
// (INV selects the + sign).  IDX in [0, 8).
template <int IDX, bool INV>
__device__ __forceinline__ float2 mul_w16(float2 a) {
    constexpr float C1 = 0.92387953251128675613f;  // cos(pi/8)
    constexpr float S1 = 0.38268343236508977173f;  // sin(pi/8)
    constexpr float C2 = 0.70710678118654752440f;  // cos(pi/4)
    if constexpr (IDX == 0) {
        return a;
    } else if constexpr (IDX == 4) {  // -+ i
        return INV ? make_float2(-a.y, a.x) : make_float2(a.y, -a.x);
    } else if constexpr (IDX == 2) {  // (1 -+ i) / sqrt2
        return INV ? make_float2(C2 * (a.x - a.y), C2 * (a.x + a.y)) : make_float2(C2 * (a.x + a.y), C2 * (a.y - a.x));
    } else if constexpr (IDX == 6) {  // (-1 -+ i) / sqrt2
        return INV ? make_float2(-C2 * (a.x + a.y), C2 * (a.x - a.y)) : make_float2(C2 * (a.y - a.x), -C2 * (a.x + a.y));
    } else {
        constexpr float c = IDX == 1 ? C1 : IDX == 3 ? S1 : IDX == 5 ? -S1 : -C1;
        constexpr float s = IDX == 1 ? S1 : IDX == 3 ? C1 : IDX == 5 ? C1 : S1;  // sin(2 pi IDX / 16)
        // forward: (c - i s); inverse: (c + i s)
        return INV ? make_float2(fmaf(a.x, c, -a.y * s), fmaf(a.x, s, a.y * c))
                   : make_float2(fmaf(a.x, c, a.y * s), fmaf(a.y, c, -a.x * s));
    }
}

// Multiply by exp(-+ 2 pi i IDX / 32), IDX in [0, 16): the last level of a 32-point in-register transform.
template <int IDX, bool INV>
__device__ __forceinline__ float2 mul_w32(float2 a) {
    if constexpr ((IDX & 1) == 0) {
        return mul_w16<IDX / 2, INV>(a);
    } else {
        constexpr float C[4] = {0.98078528040323044913f, 0.83146961230254523708f, 0.55557023301960222474f,
                                0.19509032201612826785f};   // cos(pi/16), cos(3pi/16), cos(5pi/16), cos(7pi/16)
        constexpr int h = (IDX & 7) >> 1;                   // IDX = 1,3,5,7 -> 0..3; IDX = 9,11,13,15 -> 0..3
        // first quadrant: (cos, sin) = (C[h], C[3-h]); second quadrant (IDX > 8): (-C[3-h], C[h])
        constexpr float c = IDX < 8 ? C[h] : -C[3 - h];
        constexpr float s = IDX < 8 ? C[3 - h] : C[h];
        return INV ? make_float2(fmaf(a.x, c, -a.y * s), fmaf(a.x, s, a.y * c))
                   : make_float2(fmaf(a.x, c, a.y * s), fmaf(a.y, c, -a.x * s));
    }
}

template <int E>
__host__ __device__ constexpr int bitrev_const(int i) {
    int r = 0;
    for (int b = 1; b < E; b <<= 1) {
        r = (r << 1) | (i & 1);
        i >>= 1;
    }
    return r;
}

// One decimation-in-time level: butterflies of span HALF on t[0..E), twiddle index J handled at compile time.
template <int E, int HALF, int J, bool INV>
struct DitLevel {
    static __device__ __forceinline__ void run(float2 (&t)[E]) {
#pragma unroll
        for (int g = 0; g < E; g += 2 * HALF) {
            float2 a = t[g + J];
            float2 b = mul_w32<J*(16 / HALF), INV>(t[g + J + HALF]);
            t[g + J] = cadd(a, b);
            t[g + J + HALF] = csub(a, b);
        }
        if constexpr (J + 1 < HALF) DitLevel<E, HALF, J + 1, INV>::run(t);
    }
};

template <int E, int HALF, bool INV>
struct DitStages {
    static __device__ __forceinline__ void run(float2 (&t)[E]) {
        DitLevel<E, HALF, 0, INV>::run(t);
        if constexpr (2 * HALF < E) DitStages<E, 2 * HALF, INV>::run(t);
    }
};

// Size-E FFT held entirely in one thread's registers, natural order in and out.
template <int E, bool INV>
__device__ __forceinline__ void fft_registers(float2 (&v)[E]) {
    float2 t[E];
#pragma unroll
    for (int i = 0; i < E; ++i) t[i] = v[bitrev_const<E>(i)];
    DitStages<E, 1, INV>::run(t);
#pragma unroll
    for (int i = 0; i < E; ++i) v[i] = t[i];
}

// Position of this lane's frequency residue: lane s of an L-lane group holds f2 = bitrev_L(s).
template <int K, int EMAX = 16>
__device__ __forceinline__ int lane_residue(int lane_in_group) {
    constexpr int LOG_L = FftShape<K, EMAX>::LOG_L;
    if constexpr (LOG_L == 0) {
        return 0;
    } else {
        return (int)(__brev((unsigned)lane_in_group) >> (32 - LOG_L));
    }
}

// Forward transform.  In: v[r] = z[E*l + r].  Out: v[f1] = Z[f2 + L*f1], f2 = lane_residue(l).
// tw[n] = exp(-2 pi i n / K), n < K (shared or global memory).  Every lane of the warp must call.
template <int K, int EMAX = 16>
__device__ __forceinline__ void fft_forward(float2 (&v)[FftShape<K, EMAX>::E], int l, const float2* __restrict__ tw) {
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L;
    if constexpr (L > 1) {
#pragma unroll
        for (int s = L / 2; s >= 1; s >>= 1) {
            // butterfly partner is lane l ^ s.  Lower lane: v + o.  Upper lane: (o - v) * w.
            // Written branch-free: d = o + sign * v, then d * w' with w' = w (upper) or 1 (lower).
            const bool upper = (l & s) != 0;
            const float sign = upper ? -1.f : 1.f;
            const float2 wt = tw[(l & (s - 1)) * (K / (2 * s))];
            const float2 w = upper ? wt : make_float2(1.f, 0.f);
#pragma unroll
            for (int r = 0; r < E; ++r) {
                float2 d;
                d.x = fmaf(sign, v[r].x, __shfl_xor_sync(0xffffffffu, v[r].x, s));
                d.y = fmaf(sign, v[r].y, __shfl_xor_sync(0xffffffffu, v[r].y, s));
                v[r] = cmul(d, w);
            }
        }
        const int f2 = lane_residue<K, EMAX>(l);
#pragma unroll
        for (int r = 1; r < E; ++r) v[r] = cmul(v[r], tw[(r * f2) & (K - 1)]);
    }
    fft_registers<E, false>(v);
}

// Inverse transform (unnormalised).  In: v[f1] = Y[f2 + L*f1].  Out: v[r] = K * y[E*l + r].
template <int K, int EMAX = 16>
__device__ __forceinline__ void fft_inverse(float2 (&v)[FftShape<K, EMAX>::E], int l, const float2* __restrict__ tw) {
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L;
    fft_registers<E, true>(v);
    if constexpr (L > 1) {
        const int f2 = lane_residue<K, EMAX>(l);
#pragma unroll
        for (int r = 1; r < E; ++r) v[r] = cmulc(v[r], tw[(r * f2) & (K - 1)]);
#pragma unroll
        for (int s = 1; s < L; s <<= 1) {
            // inverse of the forward butterfly: t = v * conj(w') ; lower: t + o, upper: o - t
            const bool upper = (l & s) != 0;
            const float sign = upper ? -1.f : 1.f;
            const float2 wt = tw[(l & (s - 1)) * (K / (2 * s))];
            const float2 w = upper ? wt : make_float2(1.f, 0.f);
#pragma unroll
            for (int r = 0; r < E; ++r) {
                const float2 t = cmulc(v[r], w);
                v[r].x = fmaf(sign, t.x, __shfl_xor_sync(0xffffffffu, t.x, s));
                v[r].y = fmaf(sign, t.y, __shfl_xor_sync(0xffffffffu, t.y, s));
            }
        }
    }
}

// Fill a shared-memory twiddle table tw[n] = exp(-2 pi i n / K).  Computed in place (sincospif takes
// the argument in units of pi, so the reduction is exact) rather than fetched: a table in global
// memory would put one more dependent memory round trip at the head of every kernel.
template <int K>
__device__ __forceinline__ void load_twiddles(float2* tw) {
    for (int n = threadIdx.x; n < K; n += blockDim.x) {
        float s, c;
        sincospif(-2.0f * (float)n / (float)K, &s, &c);
        tw[n] = make_float2(c, s);
    }
}

}  // namespace circ
