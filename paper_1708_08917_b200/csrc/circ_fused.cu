// S4 -- the whole fully-connected forward pass in one launch, for small batches.
//
// At batch 1..8 the layer is bound by reading the weight spectra once (m*n/k floats), so this
// kernel is organised around that stream (Algorithm 1 with the loops reordered so that every
// FFT(w_ij) is touched exactly once and every x_j / a_i is transformed once):
//
//   phase A  every CTA transforms the whole input (q blocks, up to PAIRS sample pairs) into shared
//            memory.  Spectra are stored per block as lo[s] = Z[s] and hi[s] = Z[k - s]
//            (hi[0] = Z[k/2]) for s < k/2, which is the order the packed weight spectra use.
//   phase B  each CTA owns a few row blocks i; its warps split the column blocks j, stream
//            What_ij as coalesced 16-byte loads (two packed bins per load), and accumulate
//            Yhat_i[f] += What_ij[f] Z_j[f] for bins f and k - f in registers; partial sums are
//            combined by warp shuffles and a fixed-order sum over warps (bitwise repeatable).
//   phase C  one inverse transform per (row block, pair), bias + ReLU, vector stores of y.
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
    int jsplit;  // warps that share one row block (power of two, divides the warp count)
};

__host__ __device__ inline size_t fused_smem_bytes(int k, int q, int pairs, int rows_per_cta, int jsplit) {
    return sizeof(float2) * ((size_t)k + (size_t)pairs * q * k + (size_t)jsplit * rows_per_cta * pairs * k);
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
    // transforms here are latency, not throughput: few points per lane keep every thread's chain short
    constexpr int EMAX = K <= 8 ? 16 : (K <= 128 ? 4 : 8);
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L, TT = kFusedThreads / L;
    constexpr int H = K / 2;                    // packed slots per block
    constexpr int G = K / 4;                    // threads that cover one block with 16-byte loads
    constexpr int NU = G > 32 ? G / 32 : 1;     // 16-byte loads per thread and block
    constexpr int BPW = G >= 32 ? 1 : 32 / G;   // blocks per warp-wide load
    // weight loads in flight per thread (the same bytes in flight for either storage type)
    constexpr int UNROLL = (PAIRS == 1 ? 8 : PAIRS == 2 ? 4 : 2) / (NU > 1 ? 2 : 1) * (int)(sizeof(float) / sizeof(WT));
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2* tw = reinterpret_cast<float2*>(smem_raw);
    float2* zlo = tw + K;                                      // [PAIRS][q][H]  Z[s]
    float2* zhi = zlo + (size_t)PAIRS * a.q * H;               // [PAIRS][q][H]  Z[k-s], slot 0 = Z[k/2]
    float2* part = zhi + (size_t)PAIRS * a.q * H;              // [jsplit][rows][PAIRS][K]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = a.q;
    load_twiddles<K>(tw);
    pdl_trigger();
    pdl_wait();     // x may come from the kernel before
    __syncthreads();

    // ---- phase A: Z_j for all column blocks ----------------------------------------------------
    {
        const int gi = tid / L, l = tid % L;
        const int f2 = lane_residue<K, EMAX>(l);
        const int total = PAIRS * q;
        for (int base = 0; base < total; base += TT) {
            const int T = base + gi;
            const int c = T / q, j = T - c * q;
            float2 v[E];
            float re[E], im[E];
#pragma unroll
            for (int r = 0; r < E; ++r) re[r] = im[r] = 0.f;
            if (T < total && c < a.Bh) {
                const size_t off0 = (size_t)c * a.n + (size_t)j * K + E * l;
                const size_t off1 = (size_t)(c + a.Bh) * a.n + (size_t)j * K + E * l;
                if (a.x_bf16) {
                    load_run<E>(static_cast<const __nv_bfloat16*>(a.x) + off0, re);
                    if (c + a.Bh < a.batch) load_run<E>(static_cast<const __nv_bfloat16*>(a.x) + off1, im);
                } else {
                    load_run<E>(static_cast<const float*>(a.x) + off0, re);
                    if (c + a.Bh < a.batch) load_run<E>(static_cast<const float*>(a.x) + off1, im);
                }
            }
#pragma unroll
            for (int r = 0; r < E; ++r) v[r] = make_float2(re[r], im[r]);
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
    __syncthreads();

    // ---- phase B: stream the weight spectra ----------------------------------------------------
    const int i0 = blockIdx.x * a.rows_per_cta;
    const int rows = min(a.rows_per_cta, a.p - i0);
    {
        const int JS = a.jsplit;
        const int slice = warp % JS, row_first = warp / JS, row_step = kFusedWarps / JS;
        const int u0 = G >= 32 ? lane : lane % G;   // first packed-slot pair of this thread
        const int jsub = G >= 32 ? 0 : lane / G;
        const int per_slice = ((q + JS * BPW - 1) / (JS * BPW)) * BPW;
        const int jb = slice * per_slice, je = min(q, jb + per_slice);
        for (int row = row_first; row < rows; row += row_step) {
            const WT* wrow = static_cast<const WT*>(a.w_stream) + (size_t)(i0 + row) * q * K;
            float2 acc[PAIRS][NU][4];
#pragma unroll
            for (int c = 0; c < PAIRS; ++c)
#pragma unroll
                for (int t = 0; t < NU; ++t)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[c][t][e] = make_float2(0.f, 0.f);

            for (int j = jb + jsub; j < je; j += BPW * UNROLL) {
                typename WeightVec<WT>::raw wv[UNROLL][NU];
#pragma unroll
                for (int s = 0; s < UNROLL; ++s) {
                    const int jj = j + s * BPW;
#pragma unroll
                    for (int t = 0; t < NU; ++t)
                        wv[s][t] = jj < je ? WeightVec<WT>::load(wrow + (size_t)jj * K, u0 + 32 * t) : WeightVec<WT>::zero();
                }
#pragma unroll
                for (int s = 0; s < UNROLL; ++s) {
                    const int jj = min(j + s * BPW, q - 1);  // tail iterations multiply zeros
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
                            const size_t zoff = ((size_t)c * q + jj) * H + 2 * u;
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
            }
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
        }
    }
    __syncthreads();

    // ---- phase C: inverse transforms, bias, activation -----------------------------------------
    {
        const int gi = tid / L, l = tid % L;
        const int f2 = lane_residue<K, EMAX>(l);
        const int total = rows * PAIRS;
        for (int base = 0; base < total; base += TT) {
            const int T = base + gi;
            const bool live = T < total;
            const int row = live ? T / PAIRS : 0, c = live ? T % PAIRS : 0;
            float2 v[E];
#pragma unroll
            for (int f1 = 0; f1 < E; ++f1) v[f1] = make_float2(0.f, 0.f);
            if (live) {
                for (int sl = 0; sl < a.jsplit; ++sl) {   // fixed order: bitwise repeatable
                    const float2* src = part + (((size_t)sl * a.rows_per_cta + row) * PAIRS + c) * K;
#pragma unroll
                    for (int f1 = 0; f1 < E; ++f1) {
                        const float2 t = src[f2 + L * f1];
                        v[f1].x += t.x;
                        v[f1].y += t.y;
                    }
                }
            }
            fft_inverse<K, EMAX>(v, l, tw);
            if (!live || c >= a.Bh) continue;
            const int col = (i0 + row) * K + E * l;
            float re[E], im[E];
#pragma unroll
            for (int r = 0; r < E; ++r) {
                const float b = a.bias ? __ldg(a.bias + col + r) : 0.f;
                re[r] = v[r].x + b;
                im[r] = v[r].y + b;
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
}

static int pairs_for(int batch) {
    const int bh = (batch + 1) / 2;
    return bh <= 1 ? 1 : bh <= 2 ? 2 : 4;
}

static void plan(const Layer* L, int pairs, int* rows, int* jsplit) {
    // one CTA per SM; when a CTA has fewer row blocks than warps, several warps share a row block
    int r = (L->geo.p + 147) / 148;
    if (r < 1) r = 1;
    int js = 1;
    while (js * 2 * r <= kFusedWarps) js *= 2;
    while (js > 1 && fused_smem_bytes(L->geo.k, L->geo.q, pairs, r, js) > (size_t)kMaxFusedSmem) js /= 2;
    *rows = r;
    *jsplit = js;
}

bool fused_fc_supported(const Layer* L, int batch) {
    if (L->kind != 0 || batch < 1 || batch > 8 || L->geo.k > 256 || embedded(L->geo)) return false;   // larger or embedded blocks: the staged path
    const int pairs = pairs_for(batch);
    int rows, js;
    plan(L, pairs, &rows, &js);
    return fused_smem_bytes(L->geo.k, L->geo.q, pairs, rows, js) <= (size_t)kMaxFusedSmem;
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
static int launch_one(const FusedArgs& a, unsigned grid, size_t smem, cudaStream_t stream) {
    static thread_local int configured_device = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        CIRC_CUDA_TRY(cudaFuncSetAttribute(fused_fc_kernel<K, PAIRS, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kMaxFusedSmem),
                      CIRC_ERR_CUDA);
        configured_device = dev;
    }
    launch_kernel(true, fused_fc_kernel<K, PAIRS, WT>, dim3(grid), dim3(kFusedThreads), smem, stream, a);
    return CIRC_OK;
}

template <int K, typename WT>
static int launch_w(const FusedArgs& a, int pairs, unsigned grid, size_t smem, cudaStream_t stream) {
    switch (pairs) {
        case 1: return launch_one<K, 1, WT>(a, grid, smem, stream);
        case 2: return launch_one<K, 2, WT>(a, grid, smem, stream);
        default: return launch_one<K, 4, WT>(a, grid, smem, stream);
    }
}

template <int K>
static int launch_k(const FusedArgs& a, bool bf16_spectra, int pairs, unsigned grid, size_t smem, cudaStream_t stream) {
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
    plan(L, pairs, &a.rows_per_cta, &a.jsplit);
    const unsigned grid = (unsigned)((a.p + a.rows_per_cta - 1) / a.rows_per_cta);
    const size_t smem = fused_smem_bytes(L->geo.k, a.q, pairs, a.rows_per_cta, a.jsplit);
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
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
