// S3 for large forwards: inverse transforms + bias + activation with the transform done in two in-register passes
// around ONE exchange through shared memory, and the output tile written by TMA.  The mirror image of
// circ_input_bulk.cu: with n = E2 l + r and f = f2 + L2 f1,
//
//     y[E2 l + r] = sum_f2 w_L2^-(l f2) * [ w_K^-(r f2) * ( sum_f1 w_E2^-(r f1) Y[f2 + L2 f1] ) ]      (unnormalised)
//
//   staging  a tile is 32 transforms (pair c, row block i): 32 consecutive row blocks of a pair (p >= 32) or 32 / p whole
//            pairs.  For every complex problem g the (Re, Im) pairs of the tile's transforms are one contiguous run of
//            Y[g][col][2 i ..], so ONE TMA box over (run, column, problem) brings all bins 0 < f < K/2 of the tile, a second
//            one (column Bho + c) the mirror bins, two small ones the real bins; completion is counted on an mbarrier
//            (bounded wait, error word).  Thread blocks are persistent and the tile is double-buffered.  (Loading the
//            bins with per-thread loads, one tile ahead, kept too few bytes in flight: 71 us against 25 us for the
//            input kernel on the same 134 MB.)
//   loads    lane = transform, warp = f2: a thread takes the E2 bins f2 + L2 f1 of its transform from the staged tile
//            (mirror bins conjugated).
//   pass A   E2-point inverse transform over f1 in registers, conjugate twiddle w_K^-(r f2) (warp-uniform, kept in
//            registers), written to the exchange area [transform][f2][r].
//   pass B   L2 threads per transform, thread (transform, t) holds r = R1 t .. and all f2: size-L2 inverse transforms
//            in registers give y[E2 l + r] of both samples of the pair; bias, activation, rounding; written to the
//            output tile with the 128-byte swizzle that a TMA store expects.  The exchange area is the input tile's own
//            memory (every thread has taken its bins by then).
//   store    one thread writes the tile with two cp.async.bulk.tensor stores (the rows of the pairs' first samples, the
//            rows of their second samples; rows past the batch are clipped by the copy), double-buffered.
#include <type_traits>

#include "circ_tc.cuh"
#include "circ_fft.cuh"
#include "circ_io.cuh"

namespace circ {

template <int K, typename TOUT>
struct OutBulk {
    static_assert(K >= 32 && K <= 256 && (K & (K - 1)) == 0, "K = 32 .. 256");
    static_assert(K * sizeof(TOUT) >= 128, "a transform fills at least one 128-byte swizzle row");
    static constexpr int E2 = K <= 64 ? 8 : 16;          // bins per thread in pass A
    static constexpr int L2 = K / E2;                    // size of the pass-B transform = threads per transform = warps
    static constexpr int R1 = E2 / L2 > 0 ? E2 / L2 : 1; // values of r per thread in pass B
    static_assert(L2 * R1 == E2 && L2 >= 4, "pass B gives every thread K / L2 points; at least four warps");
    static constexpr int TT = 32;                        // transforms per tile: the lanes of pass A
    static constexpr int NT = 32 * L2;
    static constexpr int CE = 128 / (int)sizeof(TOUT);   // elements per 128-byte chunk
    static constexpr size_t HALF = (size_t)TT * K * sizeof(TOUT);    // the first (or second) samples' rows of an output tile
    static constexpr size_t OUT = 2 * HALF;                          // one output tile
    static constexpr int NC = K / 2 - 1;                             // complex problems
    static constexpr size_t IN_C = (size_t)NC * TT * sizeof(float2); // the bins 0 < f < K/2 of a tile (and as much for the mirror bins)
    static constexpr size_t IN_R = (size_t)2 * TT * sizeof(float);   // the two real bins of a tile, one column group
    static constexpr int EXP = (K + 2) * (int)sizeof(float2);        // exchange area: bytes per transform
    static constexpr size_t EX = (size_t)TT * EXP;
    static constexpr size_t IN_RAW = 2 * IN_C + 2 * IN_R;
    static constexpr size_t IN = ((IN_RAW > EX ? IN_RAW : EX) + 1023) & ~(size_t)1023;   // an input tile, later the exchange area
    static constexpr int NOUT = 2 * IN + 2 * OUT + sizeof(float2) * K + 2048 <= 220 * 1024 ? 2 : 1;   // output tiles in shared memory
    static constexpr size_t SMEM = 1024 + 2 * IN + NOUT * OUT + sizeof(float2) * K + 64;
};

// Element e of tile-local transform tr in a staging half, at the position the TMA store's 128-byte swizzle expects.
template <int K, typename TOUT>
__device__ __forceinline__ TOUT* staging(unsigned char* half, int tr, int e) {
    const uint32_t off = (uint32_t)(tr * K + e) * (uint32_t)sizeof(TOUT);
    const uint32_t row = off >> 7, chunk = (off >> 4) & 7u;
    return reinterpret_cast<TOUT*>(half + (row << 7) + (((chunk ^ (row & 7u)) << 4) | (off & 15u)));
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, const void* src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

template <int K, typename TOUT>
__global__ void __launch_bounds__(OutBulk<K, TOUT>::NT)
output_ifft_tma_kernel(const __grid_constant__ CUtensorMap map_yc, const __grid_constant__ CUtensorMap map_yr,
                       const __grid_constant__ CUtensorMap map_y, const float* __restrict__ bias, int relu, int p, int Bho, int ntiles,
                       int* status, int pdl_late, int no_copy) {
    using S = OutBulk<K, TOUT>;
    const uint32_t spin_limit = no_copy ? (1u << 12) : kSpinLimit;   // no_copy: fault injection (tests only)
    constexpr int L2 = S::L2, R1 = S::R1, E2 = S::E2, TT = S::TT;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* in0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* out0 = in0 + 2 * S::IN;
    float2* tw = reinterpret_cast<float2*>(out0 + S::NOUT * S::OUT);
    uint64_t* full = reinterpret_cast<uint64_t*>(tw + K);             // [2]
    const int tid = threadIdx.x, lane = tid & 31;
    const int f2w = tid >> 5;                            // pass A: this thread's f2 (warp-uniform); its transform of the tile is `lane`

    load_twiddles<K>(tw);
    if (tid == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_yc) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_yr) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_y) : "memory");
        for (int b = 0; b < 2; ++b) mbar_init(&full[b], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!pdl_late) pdl_trigger();
    pdl_wait();     // Y is written by the contraction kernel before this one
    __syncthreads();
    float2 twr[E2];
#pragma unroll
    for (int r = 0; r < E2; ++r) twr[r] = tw[(r * f2w) & (K - 1)];

    // Tiles: p >= 32: tile = (pair c, 32 consecutive row blocks); p < 32: tile = 32 / p consecutive pairs.
    const int tiles_per_row = p >= TT ? p / TT : 1, rows_per_tile = p >= TT ? 1 : TT / p;
    auto tile_origin = [&](int tile, int& c0, int& i0) {
        if (p >= TT) {
            c0 = tile / tiles_per_row;
            i0 = (tile - c0 * tiles_per_row) * TT;
        } else {
            c0 = tile * rows_per_tile;
            i0 = 0;
        }
    };
    // one thread fetches a tile: [complex bins: NC x 32 pairs][mirror bins: the same from column Bho + c][real bins of
    // column c: 2 x 32 floats][real bins of column Bho + c]
    auto fetch = [&](int tile, int b) {
        if (tid != 0) return;
        int c0, i0;
        tile_origin(tile, c0, i0);
        unsigned char* dst = in0 + (size_t)b * S::IN;
        mbar_expect_tx(&full[b], (uint32_t)S::IN_RAW);
        if (no_copy) return;                             // the bytes were announced, nothing is in flight: the wait runs out
        tma_load_4d(dst, &map_yc, &full[b], 2 * i0, c0, 0, 0);
        tma_load_4d(dst + S::IN_C, &map_yc, &full[b], 2 * i0, Bho + c0, 0, 0);
        tma_load_4d(dst + 2 * S::IN_C, &map_yr, &full[b], i0, c0, 0, 0);
        tma_load_4d(dst + 2 * S::IN_C + S::IN_R, &map_yr, &full[b], i0, Bho + c0, 0, 0);
    };

    int tile = blockIdx.x;
    if (tile < ntiles) fetch(tile, 0);
    if (tile + (int)gridDim.x < ntiles) fetch(tile + (int)gridDim.x, 1);
    bool ok = true;
    int it = 0;
    for (; tile < ntiles; tile += gridDim.x, ++it) {
        const int b = it & 1;
        unsigned char* in = in0 + (size_t)b * S::IN;
        unsigned char* out = out0 + (size_t)(S::NOUT == 2 ? b : 0) * S::OUT;
        int c0, i0;
        tile_origin(tile, c0, i0);
        ok = mbar_wait_plain(&full[b], (uint32_t)(it >> 1) & 1u, spin_limit);
        ok = __syncthreads_and(ok);
        if (!ok) break;
        // ---- this thread's bins: Y[f2 + L2 f1] of transform `lane`, then pass A ----------------------------------
        float2 v[E2];
        {
            const float2* cplx = reinterpret_cast<const float2*>(in);
            const float2* mirr = reinterpret_cast<const float2*>(in + S::IN_C);
            const float* re0 = reinterpret_cast<const float*>(in + 2 * S::IN_C);
            const float* re1 = reinterpret_cast<const float*>(in + 2 * S::IN_C + S::IN_R);
#pragma unroll
            for (int f1 = 0; f1 < E2; ++f1) {
                const int f = f2w + L2 * f1;             // warp-uniform
                if (f == 0 || f == K / 2) {
                    const int pr = f == 0 ? 0 : TT;      // problem 0 / problem 1
                    v[f1] = make_float2(re0[pr + lane], re1[pr + lane]);
                } else if (f < K / 2) {
                    v[f1] = cplx[(f - 1) * TT + lane];
                } else {
                    const float2 z = mirr[(K - f - 1) * TT + lane];
                    v[f1] = make_float2(z.x, -z.y);      // mirror bins are stored as conjugates
                }
            }
        }
        __syncthreads();                                 // every thread has its bins: the input tile becomes the exchange area
        fft_registers<E2, true>(v);
        {
            float4* mine = reinterpret_cast<float4*>(in + (size_t)lane * S::EXP) + f2w * (E2 / 2);
#pragma unroll
            for (int r = 0; r < E2; r += 2) {
                const float2 a = r == 0 ? v[0] : cmulc(v[r], twr[r]);
                const float2 c2 = cmulc(v[r + 1], twr[r + 1]);
                mine[r / 2] = make_float4(a.x, a.y, c2.x, c2.y);
            }
        }
        if (S::NOUT == 1 && tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the one output tile: its last stores have read it
        __syncthreads();
        // ---- pass B: thread (transform, t): R1 values of r, all f2 ----------------------------------------------
        {
            const int tr = tid / L2, t = tid % L2;
            const int i = p >= TT ? i0 + tr : tr % p;
            const float2* ex = reinterpret_cast<const float2*>(in + (size_t)tr * S::EXP);
            float2 a[R1][L2];
#pragma unroll
            for (int f2 = 0; f2 < L2; ++f2)
#pragma unroll
                for (int e = 0; e < R1; ++e) a[e][f2] = ex[f2 * E2 + R1 * t + e];
#pragma unroll
            for (int e = 0; e < R1; ++e) fft_registers<L2, true>(a[e]);
#pragma unroll
            for (int l = 0; l < L2; ++l) {
                const int at = E2 * l + R1 * t;          // R1 <= 2 consecutive outputs: inside one 16-byte chunk
                TOUT* d0 = staging<K, TOUT>(out, tr, at);
                TOUT* d1 = staging<K, TOUT>(out + S::HALF, tr, at);
#pragma unroll
                for (int e = 0; e < R1; ++e) {
                    const float bb = bias ? __ldg(bias + (size_t)i * K + at + e) : 0.f;
                    float o0 = a[e][l].x + bb, o1 = a[e][l].y + bb;
                    if (relu) {
                        o0 = fmaxf(o0, 0.f);
                        o1 = fmaxf(o1, 0.f);
                    }
                    store_one(d0 + e, o0);
                    store_one(d1 + e, o1);
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the output tile is read, the input tile rewritten, by the copy engine
        __syncthreads();
        const int next2 = tile + 2 * (int)gridDim.x;
        if (tid == 0) {
            // with two output tiles: the other one is written in the next tile, the stores issued from it (a whole tile
            // ago) must have read it; the barriers of the next tile order this wait before those writes
            if (S::NOUT == 2) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            tma_store_4d(&map_y, out, 0, i0 * (K / S::CE), c0, 0);
            tma_store_4d(&map_y, out + S::HALF, 0, i0 * (K / S::CE), c0 + Bho, 0);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        if (next2 < ntiles) fetch(next2, b);             // this tile's memory is free: refill it two tiles ahead
        if (pdl_late && tile + (int)gridDim.x >= ntiles) pdl_trigger();
    }
    if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores done before the block's memory goes away
    if (!ok) {
        // a wait gave up: report it, and give the copies in flight a bounded wait to land before the memory goes away
        if (tid == 0) atomicExch(status, 1);
        if (!no_copy) {
            mbar_wait_plain(&full[it & 1], (uint32_t)(it >> 1) & 1u, 1u << 16);
            mbar_wait_plain(&full[(it + 1) & 1], (uint32_t)((it + 1) >> 1) & 1u, 1u << 16);
        }
    }
}

__device__ __forceinline__ uint32_t pack_bf16_pair(float a, float b) {      // a in the low half: the lower address
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// ---- short blocks (K = 4, 8, 16): one thread per transform ---------------------------------------------------------
// A transform of at most 16 points fits one thread's registers, so there is no exchange: a tile is 128 transforms (pair c,
// 128 consecutive row blocks), staged by the same four TMA boxes; thread t takes the K/2 + 1 bins of transform t
// (consecutive threads = consecutive (Re, Im) pairs), does the K-point inverse transform, adds bias, applies the
// activation and writes its 2 x K outputs as 16-byte pieces into the swizzled output tile, which leaves by two TMA
// stores.  Tiles are a few KB, so several thread blocks per SM keep enough bytes in flight.
template <int K, typename TOUT>
struct OutSmall {
    static_assert(K >= 4 && K <= 16 && (K & (K - 1)) == 0, "K = 4, 8, 16");
    static_assert(K * sizeof(TOUT) >= 16, "a transform's outputs are whole 16-byte pieces");
    static constexpr int TT = 128;                       // transforms per tile = threads per block
    static constexpr int CE = 128 / (int)sizeof(TOUT);
    static constexpr size_t HALF = (size_t)TT * K * sizeof(TOUT);    // a multiple of 1024
    static constexpr size_t OUT = 2 * HALF;
    static constexpr int NC = K / 2 - 1;
    static constexpr size_t IN_C = (size_t)NC * TT * sizeof(float2);
    static constexpr size_t IN_R = (size_t)2 * TT * sizeof(float);
    static constexpr size_t IN_RAW = 2 * IN_C + 2 * IN_R;
    static constexpr size_t IN = (IN_RAW + 1023) & ~(size_t)1023;
    static constexpr size_t SMEM = 1024 + 2 * IN + 2 * OUT + 64;
};

template <int K, typename TOUT>
__global__ void __launch_bounds__(OutSmall<K, TOUT>::TT)
output_ifft_tma_small_kernel(const __grid_constant__ CUtensorMap map_yc, const __grid_constant__ CUtensorMap map_yr,
                             const __grid_constant__ CUtensorMap map_y, const float* __restrict__ bias, int relu, int p, int Bho,
                             int ntiles, int* status, int pdl_late, int no_copy) {
    using S = OutSmall<K, TOUT>;
    const uint32_t spin_limit = no_copy ? (1u << 12) : kSpinLimit;   // no_copy: fault injection (tests only)
    constexpr int TT = S::TT, NC = S::NC;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* in0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* out0 = in0 + 2 * S::IN;
    uint64_t* full = reinterpret_cast<uint64_t*>(out0 + 2 * S::OUT);  // [2]
    const int tid = threadIdx.x;

    if (tid == 0) {
        if (NC > 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_yc) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_yr) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_y) : "memory");
        for (int b = 0; b < 2; ++b) mbar_init(&full[b], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!pdl_late) pdl_trigger();
    pdl_wait();     // Y is written by the contraction kernel before this one
    __syncthreads();

    const int tiles_per_row = p / TT;                    // p is a multiple of 128
    auto fetch = [&](int tile, int b) {
        if (tid != 0) return;
        const int c0 = tile / tiles_per_row, i0 = (tile - c0 * tiles_per_row) * TT;
        unsigned char* dst = in0 + (size_t)b * S::IN;
        mbar_expect_tx(&full[b], (uint32_t)S::IN_RAW);
        if (no_copy) return;                             // the bytes were announced, nothing is in flight: the wait runs out
        if (NC > 0) {
            tma_load_4d(dst, &map_yc, &full[b], 2 * i0, c0, 0, 0);
            tma_load_4d(dst + S::IN_C, &map_yc, &full[b], 2 * i0, Bho + c0, 0, 0);
        }
        tma_load_4d(dst + 2 * S::IN_C, &map_yr, &full[b], i0, c0, 0, 0);
        tma_load_4d(dst + 2 * S::IN_C + S::IN_R, &map_yr, &full[b], i0, Bho + c0, 0, 0);
    };

    int tile = blockIdx.x;
    if (tile < ntiles) fetch(tile, 0);
    if (tile + (int)gridDim.x < ntiles) fetch(tile + (int)gridDim.x, 1);
    bool ok = true;
    int it = 0;
    for (; tile < ntiles; tile += gridDim.x, ++it) {
        const int b = it & 1;
        unsigned char* in = in0 + (size_t)b * S::IN;
        unsigned char* out = out0 + (size_t)b * S::OUT;
        const int c0 = tile / tiles_per_row, i0 = (tile - c0 * tiles_per_row) * TT;
        ok = mbar_wait_plain(&full[b], (uint32_t)(it >> 1) & 1u, spin_limit);
        ok = __syncthreads_and(ok);
        if (!ok) break;
        float2 v[K];
        {
            const float2* cplx = reinterpret_cast<const float2*>(in);
            const float2* mirr = reinterpret_cast<const float2*>(in + S::IN_C);
            const float* re0 = reinterpret_cast<const float*>(in + 2 * S::IN_C);
            const float* re1 = reinterpret_cast<const float*>(in + 2 * S::IN_C + S::IN_R);
            v[0] = make_float2(re0[tid], re1[tid]);
            v[K / 2] = make_float2(re0[TT + tid], re1[TT + tid]);
#pragma unroll
            for (int f = 1; f < K / 2; ++f) {
                v[f] = cplx[(f - 1) * TT + tid];
                const float2 z = mirr[(f - 1) * TT + tid];
                v[K - f] = make_float2(z.x, -z.y);       // mirror bins are stored as conjugates
            }
        }
        fft_registers<K, true>(v);
        // the output tile of two tiles ago was handed to the copy engine by thread 0, which waited for those stores to
        // have read it before the barrier above: it may be rewritten
        {
            const int i = i0 + tid;
            constexpr int PER = 16 / (int)sizeof(TOUT);  // outputs per 16-byte piece
#pragma unroll
            for (int e0 = 0; e0 < K; e0 += PER) {
                float o0[PER], o1[PER];
#pragma unroll
                for (int e = 0; e < PER; ++e) {
                    const float bb = bias ? __ldg(bias + (size_t)i * K + e0 + e) : 0.f;
                    o0[e] = v[e0 + e].x + bb;
                    o1[e] = v[e0 + e].y + bb;
                    if (relu) {
                        o0[e] = fmaxf(o0[e], 0.f);
                        o1[e] = fmaxf(o1[e], 0.f);
                    }
                }
                TOUT* d0 = staging<K, TOUT>(out, tid, e0);
                TOUT* d1 = staging<K, TOUT>(out + S::HALF, tid, e0);
                if constexpr (std::is_same<TOUT, float>::value) {
                    *reinterpret_cast<float4*>(d0) = make_float4(o0[0], o0[1], o0[2], o0[3]);
                    *reinterpret_cast<float4*>(d1) = make_float4(o1[0], o1[1], o1[2], o1[3]);
                } else {
                    uint4 a, c;
                    a.x = pack_bf16_pair(o0[0], o0[1]); a.y = pack_bf16_pair(o0[2], o0[3]);
                    a.z = pack_bf16_pair(o0[4], o0[5]); a.w = pack_bf16_pair(o0[6], o0[7]);
                    c.x = pack_bf16_pair(o1[0], o1[1]); c.y = pack_bf16_pair(o1[2], o1[3]);
                    c.z = pack_bf16_pair(o1[4], o1[5]); c.w = pack_bf16_pair(o1[6], o1[7]);
                    *reinterpret_cast<uint4*>(d0) = a;
                    *reinterpret_cast<uint4*>(d1) = c;
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the output tile is read, the input tile rewritten, by the copy engine
        __syncthreads();
        const int next2 = tile + 2 * (int)gridDim.x;
        if (tid == 0) {
            tma_store_4d(&map_y, out, 0, i0 * K / S::CE, c0, 0);
            tma_store_4d(&map_y, out + S::HALF, 0, i0 * K / S::CE, c0 + Bho, 0);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            // the other output tile is written during the next tile: the stores issued from it (a tile ago) must have read it
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        }
        if (next2 < ntiles) fetch(next2, b);             // this tile's input memory is free: refill it two tiles ahead
        if (pdl_late && tile + (int)gridDim.x >= ntiles) pdl_trigger();
    }
    if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores done before the block's memory goes away
    if (!ok) {
        if (tid == 0) atomicExch(status, 1);
        if (!no_copy) {
            mbar_wait_plain(&full[it & 1], (uint32_t)(it >> 1) & 1u, 1u << 16);
            mbar_wait_plain(&full[(it + 1) & 1], (uint32_t)((it + 1) >> 1) & 1u, 1u << 16);
        }
    }
}

template <int K, typename TOUT>
static int launch_one(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream) {
    using S = OutBulk<K, TOUT>;
    auto kernel = output_ifft_tma_kernel<K, TOUT>;
    static thread_local int configured_device = -1;
    static thread_local int per_sm = 1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        CIRC_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::SMEM), CIRC_ERR_CUDA);
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, S::NT, S::SMEM) != cudaSuccess || per_sm < 1) {
            cudaGetLastError();
            per_sm = 1;
        }
        configured_device = dev;
    }
    const int p = L->geo.p;
    const int rows = p >= S::TT ? 1 : S::TT / p;             // pairs per tile
    const size_t cols = (size_t)2 * ext.Bho, real_sz = cols * p;
    CUtensorMap map_yc, map_yr, map_y;
    int rc;
    {
        // complex problems of Y: [problem][column][2p floats]; one box = the tile's pairs of all problems
        cuuint64_t dims[4] = {(cuuint64_t)2 * p, (cuuint64_t)cols, (cuuint64_t)S::NC, 1};
        cuuint64_t str[3] = {(cuuint64_t)2 * p * 4, (cuuint64_t)2 * real_sz * 4, (cuuint64_t)2 * real_sz * 4 * S::NC};
        cuuint32_t box[4] = {(cuuint32_t)(2 * S::TT / rows), (cuuint32_t)rows, (cuuint32_t)S::NC, 1};
        if ((rc = encode_tensor_map(&map_yc, const_cast<float*>(yop) + 2 * real_sz, 4, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                    CU_TENSOR_MAP_SWIZZLE_NONE)) != CIRC_OK)
            return rc;
    }
    {
        // real problems: [problem][column][p floats]
        cuuint64_t dims[4] = {(cuuint64_t)p, (cuuint64_t)cols, 2, 1};
        cuuint64_t str[3] = {(cuuint64_t)p * 4, (cuuint64_t)real_sz * 4, (cuuint64_t)2 * real_sz * 4};
        cuuint32_t box[4] = {(cuuint32_t)(S::TT / rows), (cuuint32_t)rows, 2, 1};
        if ((rc = encode_tensor_map(&map_yr, const_cast<float*>(yop), 4, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                    CU_TENSOR_MAP_SWIZZLE_NONE)) != CIRC_OK)
            return rc;
    }
    {
        // y as [row][128-byte chunk][chunk elements]; one box = the tile's transforms of one sample per pair
        cuuint64_t dims[4] = {(cuuint64_t)S::CE, (cuuint64_t)(L->m / S::CE), (cuuint64_t)ext.Bo, 1};
        cuuint64_t str[3] = {128, (cuuint64_t)L->m * sizeof(TOUT), (cuuint64_t)L->m * sizeof(TOUT) * ext.Bo};
        cuuint32_t box[4] = {(cuuint32_t)S::CE, (cuuint32_t)(S::TT * K / S::CE / rows), (cuuint32_t)rows, 1};
        if ((rc = encode_tensor_map(&map_y, y, 4, dims, str, box,
                                    sizeof(TOUT) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16)) != CIRC_OK)
            return rc;
    }
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, L->device);
    const long ntiles = p >= S::TT ? (long)ext.Bho * (p / S::TT) : (long)ext.Bho / (S::TT / p);
    if (ntiles >= (1L << 31)) {
        set_error(CIRC_ERR_SHAPE, "too many transforms");
        return CIRC_ERR_SHAPE;
    }
    const long resident = (long)sms * per_sm;
    const unsigned blocks = (unsigned)(ntiles < resident ? ntiles : resident);
    launch_kernel(dependent_launches(), kernel, dim3(blocks), dim3(S::NT), S::SMEM, stream, map_yc, map_yr, map_y,
                  static_cast<const float*>(L->bias_dev), L->relu, p, ext.Bho, (int)ntiles, L->dev_status, (int)(dependent_launches() == PDL_LATE),
                  (int)(L->inject == INJECT_BULK_NO_COPY));
    return CIRC_OK;
}

template <int K, typename TOUT>
static int launch_small(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream) {
    using S = OutSmall<K, TOUT>;
    auto kernel = output_ifft_tma_small_kernel<K, TOUT>;
    static thread_local int configured_device = -1;
    static thread_local int per_sm = 1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        CIRC_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::SMEM), CIRC_ERR_CUDA);
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, S::TT, S::SMEM) != cudaSuccess || per_sm < 1) {
            cudaGetLastError();
            per_sm = 1;
        }
        configured_device = dev;
    }
    const int p = L->geo.p;
    const size_t cols = (size_t)2 * ext.Bho, real_sz = cols * p;
    CUtensorMap map_yc, map_yr, map_y;
    int rc;
    {
        // complex problems of Y: [problem][column][2p floats]; one box = the tile's 128 (Re, Im) pairs of all problems
        // (K = 4 has one complex problem; the dimensions stay valid for the encoder when there is none)
        const int nc = S::NC > 0 ? S::NC : 1;
        cuuint64_t dims[4] = {(cuuint64_t)2 * p, (cuuint64_t)cols, (cuuint64_t)nc, 1};
        cuuint64_t str[3] = {(cuuint64_t)2 * p * 4, (cuuint64_t)2 * real_sz * 4, (cuuint64_t)2 * real_sz * 4 * nc};
        cuuint32_t box[4] = {(cuuint32_t)(2 * S::TT), 1, (cuuint32_t)nc, 1};
        if ((rc = encode_tensor_map(&map_yc, const_cast<float*>(yop) + 2 * real_sz, 4, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                    CU_TENSOR_MAP_SWIZZLE_NONE)) != CIRC_OK)
            return rc;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)p, (cuuint64_t)cols, 2, 1};
        cuuint64_t str[3] = {(cuuint64_t)p * 4, (cuuint64_t)real_sz * 4, (cuuint64_t)2 * real_sz * 4};
        cuuint32_t box[4] = {(cuuint32_t)S::TT, 1, 2, 1};
        if ((rc = encode_tensor_map(&map_yr, const_cast<float*>(yop), 4, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                    CU_TENSOR_MAP_SWIZZLE_NONE)) != CIRC_OK)
            return rc;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)S::CE, (cuuint64_t)(L->m / S::CE), (cuuint64_t)ext.Bo, 1};
        cuuint64_t str[3] = {128, (cuuint64_t)L->m * sizeof(TOUT), (cuuint64_t)L->m * sizeof(TOUT) * ext.Bo};
        cuuint32_t box[4] = {(cuuint32_t)S::CE, (cuuint32_t)(S::TT * K / S::CE), 1, 1};
        if ((rc = encode_tensor_map(&map_y, y, 4, dims, str, box,
                                    sizeof(TOUT) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16)) != CIRC_OK)
            return rc;
    }
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, L->device);
    const long ntiles = (long)ext.Bho * (p / S::TT);
    if (ntiles >= (1L << 31)) {
        set_error(CIRC_ERR_SHAPE, "too many transforms");
        return CIRC_ERR_SHAPE;
    }
    const long resident = (long)sms * per_sm;
    const unsigned blocks = (unsigned)(ntiles < resident ? ntiles : resident);
    launch_kernel(dependent_launches(), kernel, dim3(blocks), dim3(S::TT), S::SMEM, stream, map_yc, map_yr, map_y,
                  static_cast<const float*>(L->bias_dev), L->relu, p, ext.Bho, (int)ntiles, L->dev_status, (int)(dependent_launches() == PDL_LATE),
                  (int)(L->inject == INJECT_BULK_NO_COPY));
    return CIRC_OK;
}

template <int K>
static int launch_small_k(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream) {
    if (L->y_dtype == CIRC_BF16) {
        if constexpr (K >= 8) return launch_small<K, __nv_bfloat16>(L, yop, y, ext, stream);
        set_error(CIRC_ERR_UNSUPPORTED, "bfloat16 blocks of 4 are not served by the TMA-written inverse transforms");
        return CIRC_ERR_UNSUPPORTED;
    }
    return launch_small<K, float>(L, yop, y, ext, stream);
}

template <int K>
static int launch_k(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream) {
    if (L->y_dtype == CIRC_BF16) {
        if constexpr (K >= 64) return launch_one<K, __nv_bfloat16>(L, yop, y, ext, stream);
        set_error(CIRC_ERR_UNSUPPORTED, "bfloat16 blocks below 64 are not served by the TMA-written inverse transforms");
        return CIRC_ERR_UNSUPPORTED;
    }
    return launch_one<K, float>(L, yop, y, ext, stream);
}

// Large forwards of power-of-two blocks whose transform fills at least one 128-byte row of y (float32: k >= 32,
// bfloat16: k >= 64), up to k = 256, with row-block counts that tile evenly: p a multiple of 32, or a divisor of it with
// whole tiles of pairs (a partial tile's box would reach into the rows of the second samples); and short blocks
// (float32 k = 4 .. 16, bfloat16 k = 8, 16) with p a multiple of the 128 transforms of their tiles.
// Y as one array in the interleaved layout (not the copies or the separate real / imaginary parts that the
// row-streaming contraction leaves: those forwards have few columns and little to transform).
bool output_ifft_tma_supported(const Layer* L, const void* y, const Extent& ext) {
    const int k = L->geo.k, p = L->geo.p;
    const bool common = L->kind == 0 && !embedded(L->geo) && (long)ext.Bho * p >= 148L * 64 && (reinterpret_cast<uintptr_t>(y) & 15u) == 0 &&
                        L->dev_status != nullptr && tensor_map_encoder() != nullptr;
    if (!common) return false;
    if (k <= 16)   // short blocks: tiles of 128 row blocks; a transform's outputs are at least one 16-byte piece
        return k >= (L->y_dtype == CIRC_BF16 ? 8 : 4) && p % 128 == 0;
    const int kmin = L->y_dtype == CIRC_BF16 ? 64 : 32;
    const bool tiles_evenly = p % 32 == 0 || (p % 4 == 0 && 32 % p == 0 && ext.Bho % (32 / p) == 0);
    return k >= kmin && k <= 256 && tiles_evenly;
}

int launch_output_ifft_tma(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream) {
    int rc;
    switch (L->geo.k) {
        case 4: rc = launch_small_k<4>(L, yop, y, ext, stream); break;
        case 8: rc = launch_small_k<8>(L, yop, y, ext, stream); break;
        case 16: rc = launch_small_k<16>(L, yop, y, ext, stream); break;
        case 32: rc = launch_k<32>(L, yop, y, ext, stream); break;
        case 64: rc = launch_k<64>(L, yop, y, ext, stream); break;
        case 128: rc = launch_k<128>(L, yop, y, ext, stream); break;
        case 256: rc = launch_k<256>(L, yop, y, ext, stream); break;
        default: set_error(CIRC_ERR_SHAPE, "block size %d not served by the TMA-written inverse transforms", L->geo.k); return CIRC_ERR_SHAPE;
    }
    if (rc != CIRC_OK) return rc;
    L->last_kernels[2] = KERNEL_S3_TMA;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
