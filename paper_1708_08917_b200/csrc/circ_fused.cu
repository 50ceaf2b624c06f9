// S4 -- the whole fully-connected forward pass in one launch, for small batches.
//
// At batch 1..8 the layer is bound by reading the weight spectra once (m*n/k floats), so this
// kernel is organised around that stream (Algorithm 1 with the loops reordered so that every
// FFT(w_ij) is touched exactly once and every x_j / a_i is transformed once).  The grid is
// (column splits C) x (row groups): thread block (cs, rg) owns the row blocks of group rg and the
// column blocks of slice cs; the C blocks of a row group form a thread-block cluster.
//
//   phase A  the block transforms its slice of the input (q / C blocks, up to PAIRS sample pairs) into
//            shared memory; the loads of several passes are in flight at once.  Spectra are stored per
//            block as lo[s] = Z[s] and hi[s] = Z[k - s] (hi[0] = Z[k/2]) for s < k/2, the order of the
//            packed weight spectra.
//   phase B  the block's (row block, column sub-slice) units are dealt to its warps; a warp streams
//            What_ij as coalesced 16-byte loads (two packed bins per load; the first loads are issued
//            before phase A, they do not depend on x) and accumulates Yhat_i[f] += What_ij[f] Z_j[f]
//            for bins f and k - f in registers; lanes are combined by warp shuffles.
//   phase C  one inverse transform per (row block, pair): the partial spectra of all sub-slices of
//            all C blocks are added in a fixed order (bitwise repeatable; the other blocks' partial
//            sums are read through distributed shared memory, no atomics), then bias + ReLU and
//            vector stores of y.  The row blocks of a group are dealt to its C blocks.
// Splitting the columns fills the machine when there are fewer row blocks than SMs (k = 256 at
// n = 16384 has 64) and divides the input transforms, which every block of the unsplit kernel repeated.
#include <cooperative_groups.h>

#include <type_traits>

#include "circ_common.cuh"
#include "circ_fft.cuh"
#include "circ_io.cuh"

namespace circ {

constexpr int kFusedThreads = 512;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kMaxFusedSmem = 200 * 1024;

struct FusedArgs {
    const void* x;
    void* y;
    const void* w_stream;   // float or __nv_bfloat16, the kernel's WT
    const float* bias;
    int relu, x_bf16, y_bf16;
    int m, n, p, q, batch, Bh;
    int rows_per_cta;
    int jsplit;  // column sub-slices per row block inside a thread block (power of two)
    int csplit;  // column slices = thread blocks per cluster (1, 2, 4 or 8)
    int qs;      // column blocks per slice
};

// shared memory: twiddles, the spectra of the block's input slice, the partial output spectra
__host__ __device__ inline size_t fused_smem_bytes(int k, int qs, int pairs, int rows_per_cta, int jsplit) {
    return sizeof(float2) * ((size_t)k + (size_t)pairs * qs * k + (size_t)jsplit * rows_per_cta * pairs * k);
}

// Four consecutive packed spectrum values (two slots) as stored and as float4.
template <typename WT>
struct WeightVec;
template <>
struct WeightVec<float> {
    using raw = float4;
    static __device__ __forceinline__ raw load(const float* blk, int idx) { return __ldg(reinterpret_cast<const float4*>(blk) + idx); }
    static __device__ __forceinline__ raw zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
    static __device__ __forceinline__ float4 widen(raw r) { return r; }
};
template <>
struct WeightVec<__nv_bfloat16> {
    using raw = uint2;
    static __device__ __forceinline__ raw load(const __nv_bfloat16* blk, int idx) { return __ldg(reinterpret_cast<const uint2*>(blk) + idx); }
    static __device__ __forceinline__ raw zero() { return make_uint2(0u, 0u); }
    static __device__ __forceinline__ float4 widen(raw r) {   // a bfloat16 is the upper half of a float
        return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u), __uint_as_float(r.y << 16),
                           __uint_as_float(r.y & 0xffff0000u));
    }
};

template <int K, int PAIRS, typename WT>
__global__ void __launch_bounds__(kFusedThreads, 1) fused_fc_kernel(FusedArgs a) {
    namespace cg = cooperative_groups;
    // transforms here are latency, not throughput: few points per lane keep every thread's chain short
    constexpr int EMAX = K <= 8 ? 16 : (K <= 128 ? 4 : 8);
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L, TT = kFusedThreads / L;
    constexpr int H = K / 2;                    // packed slots per block
    constexpr int G = K / 4;                    // threads that cover one block with 16-byte loads
    constexpr int NU = G > 32 ? G / 32 : 1;     // 16-byte loads per thread and block
    constexpr int BPW = G >= 32 ? 1 : 32 / G;   // blocks per warp-wide load
    // weight loads in flight per thread (the same bytes in flight for either storage type)
    constexpr int UNROLL = (PAIRS == 1 ? 8 : PAIRS == 2 ? 4 : 2) / (NU > 1 ? 2 : 1) * (int)(sizeof(float) / sizeof(WT));
    constexpr int DEPTH = E <= 4 ? 4 : 2;       // passes of phase A whose loads are in flight together
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2* tw = reinterpret_cast<float2*>(smem_raw);
    float2* zlo = tw + K;                                      // [PAIRS][qs][H]  Z[s]
    float2* zhi = zlo + (size_t)PAIRS * a.qs * H;              // [PAIRS][qs][H]  Z[k-s], slot 0 = Z[k/2]
    float2* part = zhi + (size_t)PAIRS * a.qs * H;             // [jsplit][rows][PAIRS][K]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cs = blockIdx.x;                                 // column slice = rank in the cluster
    const int jb = cs * a.qs, je = min(a.q, jb + a.qs);        // this block's column blocks
    const int qn = max(je - jb, 0);
    const int i0 = blockIdx.y * a.rows_per_cta;
    const int rows = min(a.rows_per_cta, a.p - i0);
    load_twiddles<K>(tw);

    // ---- phase B set-up: units (row block, column sub-slice) dealt to the warps -------------------
    const int JS = a.jsplit;
    const int units = rows * JS;
    const int u0 = G >= 32 ? lane : lane % G;   // first packed-slot pair of this thread
    const int jsub = G >= 32 ? 0 : lane / G;
    const int per_slice = ((qn + JS * BPW - 1) / (JS * BPW)) * BPW;
    typedef typename WeightVec<WT>::raw Raw;
    // one chunk = UNROLL warp-wide loads of a unit, starting at column block j (relative to jb)
    auto load_chunk = [&](int unit, int j, Raw (&wv)[UNROLL][NU]) {
        const int row = unit / JS, slice = unit - row * JS;
        const int send = min(qn, (slice + 1) * per_slice);
        const WT* wrow = static_cast<const WT*>(a.w_stream) + ((size_t)(i0 + row) * a.q + jb) * K;
#pragma unroll
        for (int s = 0; s < UNROLL; ++s) {
            const int jj = j + s * BPW;
#pragma unroll
            for (int t = 0; t < NU; ++t)
                wv[s][t] = jj < send ? WeightVec<WT>::load(wrow + (size_t)jj * K, u0 + 32 * t) : WeightVec<WT>::zero();
        }
    };
    int unit = warp;                                            // this warp's current unit and position in it
    int jpos = (unit % JS) * per_slice + jsub;
    Raw wcur[UNROLL][NU];
    // the weights do not depend on x: their first loads go out before the input is even read
    // (they do not depend on an earlier kernel either, so they need not wait for it)
    if (unit < units) load_chunk(unit, jpos, wcur);
    pdl_trigger();
    pdl_wait();     // x may come from the kernel before
    __syncthreads();

    // ---- phase A: Z_j for the block's column blocks -----------------------------------------------
    {
        const int gi = tid / L, l = tid % L;
        const int f2 = lane_residue<K, EMAX>(l);
        const int total = PAIRS * qn;
        float re[DEPTH][E], im[DEPTH][E];
        auto fetch = [&](int base, float (&r_)[E], float (&i_)[E]) {
            const int T = base + gi;
#pragma unroll
            for (int r = 0; r < E; ++r) r_[r] = i_[r] = 0.f;
            if (T < total) {
                const int c = T / qn, j = T - c * qn;
                if (c < a.Bh) {
                    const size_t off0 = (size_t)c * a.n + (size_t)(jb + j) * K + E * l;
                    const size_t off1 = (size_t)(c + a.Bh) * a.n + (size_t)(jb + j) * K + E * l;
                    if (a.x_bf16) {
                        load_run<E>(static_cast<const __nv_bfloat16*>(a.x) + off0, r_);
                        if (c + a.Bh < a.batch) load_run<E>(static_cast<const __nv_bfloat16*>(a.x) + off1, i_);
                    } else {
                        load_run<E>(static_cast<const float*>(a.x) + off0, r_);
                        if (c + a.Bh < a.batch) load_run<E>(static_cast<const float*>(a.x) + off1, i_);
                    }
                }
            }
        };
#pragma unroll
        for (int d = 0; d < DEPTH; ++d) fetch(d * TT, re[d], im[d]);
        for (int base = 0; base < total; base += DEPTH * TT) {
#pragma unroll
            for (int d = 0; d < DEPTH; ++d) {
                const int T = base + d * TT + gi;
                float2 v[E];
#pragma unroll
                for (int r = 0; r < E; ++r) v[r] = make_float2(re[d][r], im[d][r]);
                if (base + (d + DEPTH) * TT < total) fetch(base + (d + DEPTH) * TT, re[d], im[d]);   // next round's loads
                if (base + d * TT < total) {        // uniform over the block: whole passes only
                    fft_forward<K, EMAX>(v, l, tw);
                    if (T < total) {
                        float2* dlo = zlo + (size_t)T * H;
                        float2* dhi = zhi + (size_t)T * H;
#pragma unroll
                        for (int f1 = 0; f1 < E; ++f1) {
                            const int f = f2 + L * f1;
                            if (f < H) dlo[f] = v[f1];
                            else dhi[f == H ? 0 : K - f] = v[f1];
                        }
                    }
                }
            }
        }
    }
    __syncthreads();

    // ---- phase B: stream the weight spectra ----------------------------------------------------
    {
        float2 acc[PAIRS][NU][4];
        auto clear = [&]() {
#pragma unroll
            for (int c = 0; c < PAIRS; ++c)
#pragma unroll
                for (int t = 0; t < NU; ++t)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[c][t][e] = make_float2(0.f, 0.f);
        };
        auto multiply = [&](int j, const Raw (&wv)[UNROLL][NU]) {
#pragma unroll
            for (int s = 0; s < UNROLL; ++s) {
                const int jj = min(j + s * BPW, qn - 1);  // tail iterations multiply zeros
#pragma unroll
                for (int t = 0; t < NU; ++t) {
                    const int u = u0 + 32 * t;
                    const bool dc = (u == 0);
                    const float4 w = WeightVec<WT>::widen(wv[s][t]);
                    // slot 2u: (a0, b0); slot 2u+1: (a1, b1).  The first slot of a block packs the two real bins.
                    const float a0 = w.x, b0 = dc ? 0.f : w.y, h0 = dc ? w.y : w.x;
                    const float a1 = w.z, b1 = w.w;
#pragma unroll
                    for (int c = 0; c < PAIRS; ++c) {
                        const size_t zoff = ((size_t)c * qn + jj) * H + 2 * u;
                        const float4 zl = *reinterpret_cast<const float4*>(zlo + zoff);
                        const float4 zh = *reinterpret_cast<const float4*>(zhi + zoff);
                        float2* ac = acc[c][t];
                        ac[0].x = fmaf(a0, zl.x, fmaf(-b0, zl.y, ac[0].x));
                        ac[0].y = fmaf(a0, zl.y, fmaf(b0, zl.x, ac[0].y));
                        ac[1].x = fmaf(a1, zl.z, fmaf(-b1, zl.w, ac[1].x));
                        ac[1].y = fmaf(a1, zl.w, fmaf(b1, zl.z, ac[1].y));
                        ac[2].x = fmaf(h0, zh.x, fmaf(b0, zh.y, ac[2].x));
                        ac[2].y = fmaf(h0, zh.y, fmaf(-b0, zh.x, ac[2].y));
                        ac[3].x = fmaf(a1, zh.z, fmaf(b1, zh.w, ac[3].x));
                        ac[3].y = fmaf(a1, zh.w, fmaf(-b1, zh.z, ac[3].y));
                    }
                }
            }
        };
        auto flush = [&](int un) {
            // combine the lanes that worked on different column blocks for the same bins
#pragma unroll
            for (int c = 0; c < PAIRS; ++c)
#pragma unroll
                for (int t = 0; t < NU; ++t)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float2 v = acc[c][t][e];
#pragma unroll
                        for (int off = G; off < 32; off <<= 1) {
                            v.x += __shfl_xor_sync(0xffffffffu, v.x, off);
                            v.y += __shfl_xor_sync(0xffffffffu, v.y, off);
                        }
                        acc[c][t][e] = v;
                    }
            if (jsub == 0) {
                const int row = un / JS, slice = un - row * JS;
#pragma unroll
                for (int c = 0; c < PAIRS; ++c) {
                    float2* dst = part + (((size_t)slice * a.rows_per_cta + row) * PAIRS + c) * K;
#pragma unroll
                    for (int t = 0; t < NU; ++t) {
                        const int u = u0 + 32 * t;
                        dst[2 * u] = acc[c][t][0];
                        dst[2 * u + 1] = acc[c][t][1];
                        dst[u == 0 ? H : K - 2 * u] = acc[c][t][2];
                        dst[K - 2 * u - 1] = acc[c][t][3];
                    }
                }
            }
        };
        // One step: issue the loads of the chunk after this one (into `fill`), multiply this one (`use`).
        // Returns false when the warp has no chunk left.
        clear();
        auto step = [&](const Raw (&use)[UNROLL][NU], Raw (&fill)[UNROLL][NU]) -> bool {
            const int slice = unit % JS;
            const int send = min(qn, (slice + 1) * per_slice);
            int nunit = unit, njpos = jpos + BPW * UNROLL;
            const bool last_of_unit = njpos - jsub >= send;          // warp-uniform
            if (last_of_unit) {
                nunit = unit + kFusedWarps;
                njpos = (nunit % JS) * per_slice + jsub;
            }
            const bool more = nunit < units;
            if (more) load_chunk(nunit, njpos, fill);
            multiply(jpos, use);
            if (last_of_unit) {
                flush(unit);
                clear();
            }
            unit = nunit;
            jpos = njpos;
            return more;
        };
        if (unit < units) {
            Raw wnext[UNROLL][NU];
            while (step(wcur, wnext) && step(wnext, wcur)) {}
        }
    }
    __syncthreads();
    cg::cluster_group cluster = cg::this_cluster();
    if (a.csplit > 1) cluster.sync();            // every block's partial spectra are complete and visible

    // ---- phase C: inverse transforms, bias, activation -----------------------------------------
    {
        const int gi = tid / L, l = tid % L;
        const int f2 = lane_residue<K, EMAX>(l);
        // the row blocks of the group are dealt to the cluster's blocks: this one takes cs, cs + C, ...
        const int my_rows = rows > cs ? (rows - cs + a.csplit - 1) / a.csplit : 0;
        const int total = my_rows * PAIRS;
        for (int base = 0; base < total; base += TT) {
            const int T = base + gi;
            const bool live = T < total;
            const int row = live ? cs + (T / PAIRS) * a.csplit : 0, c = live ? T % PAIRS : 0;
            const int col = (i0 + row) * K + E * l;
            float bv[E];
#pragma unroll
            for (int r = 0; r < E; ++r) bv[r] = 0.f;
            if (live && a.bias) load_run<E>(a.bias + col, bv);
            float2 v[E];
#pragma unroll
            for (int f1 = 0; f1 < E; ++f1) v[f1] = make_float2(0.f, 0.f);
            if (live) {
                for (int rk = 0; rk < a.csplit; ++rk) {       // fixed order: bitwise repeatable
                    const float2* rpart = a.csplit > 1 ? cluster.map_shared_rank(part, rk) : part;
                    for (int sl = 0; sl < JS; ++sl) {
                        const float2* src = rpart + (((size_t)sl * a.rows_per_cta + row) * PAIRS + c) * K;
#pragma unroll
                        for (int f1 = 0; f1 < E; ++f1) {
                            const float2 t = src[f2 + L * f1];
                            v[f1].x += t.x;
                            v[f1].y += t.y;
                        }
                    }
                }
            }
            fft_inverse<K, EMAX>(v, l, tw);
            if (!live || c >= a.Bh) continue;
            float re[E], im[E];
#pragma unroll
            for (int r = 0; r < E; ++r) {
                re[r] = v[r].x + bv[r];
                im[r] = v[r].y + bv[r];
                if (a.relu) {
                    re[r] = fmaxf(re[r], 0.f);
                    im[r] = fmaxf(im[r], 0.f);
                }
            }
            const size_t o0 = (size_t)c * a.m + col, o1 = (size_t)(c + a.Bh) * a.m + col;
            if (a.y_bf16) {
                store_run<E>(static_cast<__nv_bfloat16*>(a.y) + o0, re);
                if (c + a.Bh < a.batch) store_run<E>(static_cast<__nv_bfloat16*>(a.y) + o1, im);
            } else {
                store_run<E>(static_cast<float*>(a.y) + o0, re);
                if (c + a.Bh < a.batch) store_run<E>(static_cast<float*>(a.y) + o1, im);
            }
        }
    }
    if (a.csplit > 1) cluster.sync();            // no block leaves while its partial spectra may still be read
}

static int pairs_for(int batch) {
    const int bh = (batch + 1) / 2;
    return bh <= 1 ? 1 : bh <= 2 ? 2 : 4;
}

struct FusedPlan {
    int rows;     // row blocks per thread block
    int jsplit;   // column sub-slices per row block inside a thread block
    int csplit;   // column slices (thread blocks per cluster)
    int qs;       // column blocks per slice
    size_t smem;
    bool ok;
};

// How many clusters of `c` thread blocks of this kernel the device can hold at once (one 512-thread block with the
// largest shared-memory request per SM; clusters cannot straddle GPCs, so this is less than SMs / c).
static int resident_clusters(int device, int c) {
    static int cache[64][4];
    static bool known[64] = {};
    const int slot = c == 1 ? 0 : c == 2 ? 1 : c == 4 ? 2 : 3;
    if (device < 0 || device >= 64) return 16;
    if (!known[device]) {
        int sms = 148;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        cudaFuncSetAttribute(fused_fc_kernel<64, 1, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxFusedSmem);
        for (int i = 0, cc = 1; i < 4; ++i, cc *= 2) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)cc, (unsigned)sms);
            cfg.blockDim = dim3(kFusedThreads);
            cfg.dynamicSmemBytes = kMaxFusedSmem;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)cc;
            attr[0].val.clusterDim.y = attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, fused_fc_kernel<64, 1, float>, &cfg) != cudaSuccess || n < 1) {
                cudaGetLastError();
                n = cc == 1 ? sms : (sms / cc) * 3 / 4;      // a guess on the safe side
                if (n < 1) n = 1;
            }
            cache[device][i] = n;
        }
        known[device] = true;
    }
    return cache[device][slot];
}

// Row groups x column slices.  Among the cluster sizes 1, 2, 4, 8 that divide q and fit shared memory, take the one
// with the least estimated time per thread block, in microseconds:
//   weight stream   bytes of the block's spectra / its SM's share of the memory bandwidth (44 KB per microsecond),
//                   stretched by the imbalance of the (row, sub-slice) units over the warps;
//   input transforms 0.7 us per pass of 512 threads (more for blocks of 128 points and up, whose transforms span a warp);
//   cluster         launch and two cluster barriers: 0.8 / 1.2 / 3.0 us for 2 / 4 / 8 blocks.
// Measured on B200 (cold, one forward per graph node), C = 1 / 2 / 4 / 8: n = 16384, batch 1: k = 4: 46.6 / 46.6 / 58.1 /
// 65.9 us, k = 16: 20.7 / 20.0 / 18.9 / 22.3, k = 64: 12.0 / 10.2 / 9.5 / 11.0, k = 256: 12.5 / 9.8 / 8.4 / 9.0;
// n = 4096: k = 4: 7.0 / 7.5 / 8.1 / 12.3, k = 64: 4.2 / 4.9 / 5.2 / 6.1; 256 x 256, k = 16: 2.9 / 3.7 / 4.1 / 4.8.
// Row groups never exceed the clusters that are resident at once.
static FusedPlan plan(const Layer* L, int pairs) {
    const int p = L->geo.p, q = L->geo.q, k = L->geo.k;
    const int bpw = k >= 128 ? 1 : 128 / k;                                         // column blocks per warp-wide load
    const int chunk = bpw * ((pairs == 1 ? 8 : pairs == 2 ? 4 : 2) / (k >= 256 ? 2 : 1));   // column blocks per chunk of loads
    const int lanes = k <= 8 ? 1 : (k <= 128 ? k / 4 : 32);                         // lanes per transform in this kernel
    const int tt = kFusedThreads / lanes;                                           // transforms per pass
    const double pass_us = 0.7 * (k >= 256 ? 3.0 : k >= 128 ? 2.0 : 1.0);
    const double wbytes = L->w_dtype == CIRC_BF16 && L->w_stream_bf16 ? 2.0 : 4.0;
    FusedPlan best = {};
    double best_cost = -1.0;
    for (int c = 1; c <= 8; c *= 2) {
        if (q % c) break;
        if (L->fused_split && c != L->fused_split) continue;
        const int groups = resident_clusters(L->device, c);
        const int r = (p + groups - 1) / groups;
        const int qs = q / c;
        // sub-slices: the smallest power of two that deals the (row, sub-slice) units evenly to the warps, as long
        // as a sub-slice still fills a chunk of loads and the partial sums fit
        int js = 1;
        while (js < kFusedWarps && (r * js) % kFusedWarps != 0 && qs / (2 * js) >= chunk) js *= 2;
        while (js > 1 && fused_smem_bytes(k, qs, pairs, r, js) > (size_t)kMaxFusedSmem) js /= 2;
        const size_t smem = fused_smem_bytes(k, qs, pairs, r, js);
        if (smem > (size_t)kMaxFusedSmem) continue;
        const long units_per_warp = ((long)r * js + kFusedWarps - 1) / kFusedWarps;
        const double stream_us = (double)units_per_warp * ((qs + js - 1) / js) * k * wbytes * kFusedWarps / 44000.0;
        const double passes = (double)(((long)pairs * qs + tt - 1) / tt);
        const double cluster_us = c == 1 ? 0.0 : c == 2 ? 0.8 : c == 4 ? 1.2 : 3.0;
        const double cost = stream_us + passes * pass_us + cluster_us;
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = FusedPlan{r, js, c, qs, smem, true};
        }
    }
    return best;
}

bool fused_fc_supported(const Layer* L, int batch) {
    if (L->kind != 0 || batch < 1 || batch > 8 || L->geo.k > 256 || embedded(L->geo)) return false;   // larger or embedded blocks: the staged path
    return plan(L, pairs_for(batch)).ok;
}

// With 5 to 8 samples every CTA transforms four sample pairs of the whole input, and for long blocks on a wide
// layer that redundant work outweighs the single launch.  Measured (4096 x 4096, batch 8, one launch against the
// three-launch tensor path): k = 4: 12.3 / 19.9 us, k = 16: 9.6 / 10.8, k = 64: 10.3 / 8.1, k = 256: 13.3 / 12.4;
// 2048 x 2048, k = 64: 6.9 / 7.0; batch 4 at k = 64: 6.8 / 7.3.
bool fused_fc_preferred(const Layer* L, int batch, bool tensor_ok) {
    if (!fused_fc_supported(L, batch)) return false;
    if (tensor_ok && batch >= 5 && L->geo.k >= 64 && L->n >= 4096) return false;
    return true;
}

template <int K, int PAIRS, typename WT>
static int launch_one(const FusedArgs& a, dim3 grid, size_t smem, cudaStream_t stream) {
    static thread_local int configured_device = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        CIRC_CUDA_TRY(cudaFuncSetAttribute(fused_fc_kernel<K, PAIRS, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kMaxFusedSmem),
                      CIRC_ERR_CUDA);
        configured_device = dev;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;     // the column slices of a row group (plain loads and
    attr[1].val.clusterDim.x = (unsigned)a.csplit;        // distributed shared memory only: no multicast copies)
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.csplit > 1 ? 2 : 1;
    CIRC_CUDA_TRY(cudaLaunchKernelEx(&cfg, fused_fc_kernel<K, PAIRS, WT>, a), CIRC_ERR_CUDA);
    return CIRC_OK;
}

template <int K, typename WT>
static int launch_w(const FusedArgs& a, int pairs, dim3 grid, size_t smem, cudaStream_t stream) {
    switch (pairs) {
        case 1: return launch_one<K, 1, WT>(a, grid, smem, stream);
        case 2: return launch_one<K, 2, WT>(a, grid, smem, stream);
        default: return launch_one<K, 4, WT>(a, grid, smem, stream);
    }
}

template <int K>
static int launch_k(const FusedArgs& a, bool bf16_spectra, int pairs, dim3 grid, size_t smem, cudaStream_t stream) {
    return bf16_spectra ? launch_w<K, __nv_bfloat16>(a, pairs, grid, smem, stream) : launch_w<K, float>(a, pairs, grid, smem, stream);
}

int launch_fused_fc(const Layer* L, const void* x, void* y, int batch, cudaStream_t stream) {
    const int pairs = pairs_for(batch);
    FusedArgs a;
    a.x = x;
    a.y = y;
    const bool wb = L->w_dtype == CIRC_BF16 && L->w_stream_bf16;
    a.w_stream = wb ? static_cast<const void*>(L->w_stream_bf16) : static_cast<const void*>(L->w_stream);
    a.bias = L->bias_dev;
    a.relu = L->relu;
    a.x_bf16 = L->x_dtype == CIRC_BF16;
    a.y_bf16 = L->y_dtype == CIRC_BF16;
    a.m = L->m; a.n = L->n; a.p = L->geo.p; a.q = L->geo.q;
    a.batch = batch;
    a.Bh = (batch + 1) / 2;
    const FusedPlan pl = plan(L, pairs);
    if (!pl.ok) {
        set_error(CIRC_ERR_UNSUPPORTED, "the one-launch kernel cannot hold this layer's input spectra in shared memory");
        return CIRC_ERR_UNSUPPORTED;
    }
    a.rows_per_cta = pl.rows;
    a.jsplit = pl.jsplit;
    a.csplit = pl.csplit;
    a.qs = pl.qs;
    const dim3 grid((unsigned)pl.csplit, (unsigned)((a.p + pl.rows - 1) / pl.rows));
    const size_t smem = pl.smem;
    int rc;
    switch (L->geo.k) {
        case 4: rc = launch_k<4>(a, wb, pairs, grid, smem, stream); break;
        case 8: rc = launch_k<8>(a, wb, pairs, grid, smem, stream); break;
        case 16: rc = launch_k<16>(a, wb, pairs, grid, smem, stream); break;
        case 32: rc = launch_k<32>(a, wb, pairs, grid, smem, stream); break;
        case 64: rc = launch_k<64>(a, wb, pairs, grid, smem, stream); break;
        case 128: rc = launch_k<128>(a, wb, pairs, grid, smem, stream); break;
        case 256: rc = launch_k<256>(a, wb, pairs, grid, smem, stream); break;
        default: set_error(CIRC_ERR_SHAPE, "block size %d not supported", L->geo.k); return CIRC_ERR_SHAPE;
    }
    if (rc != CIRC_OK) return rc;
    L->last_kernels[0] = KERNEL_S4_FUSED;
    L->last_kernels[1] = pl.csplit;
    L->last_kernels[2] = pl.rows;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
