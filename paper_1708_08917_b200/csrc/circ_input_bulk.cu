// S1 for large forwards: input transforms with the tile staged by bulk asynchronous copies and the transform done
// in two in-register passes around ONE exchange through shared memory (no warp shuffles, no transposition pass).
//
// A transform of K = L2 x E2 points (K = 32 .. 256; E2 = 8 up to K = 64, else 16) is split as n = E2 l + r,
// f = f2 + L2 f1 (Sec. 4.1: the larger transform from smaller ones plus twiddles):
//
//     Z[f2 + L2 f1] = sum_r w_E2^(r f1) * [ w_K^(r f2) * ( sum_l w_L2^(l f2) z[E2 l + r] ) ]
//
//   staging  a thread block takes a tile of 32 transforms (pair c, column block j): 32 consecutive column blocks of one
//            row of x (q >= 32), or 32 / q whole rows (q < 32).  The K samples of row c are the real part and those of
//            row c + Bh the imaginary part (two real signals ride one complex transform), so a tile is two contiguous
//            pieces of x: ONE TMA box each (cp.async.bulk.tensor over x seen as [row][128-byte chunk][chunk elements],
//            128-byte swizzle, rows past the batch read as zeros), completion counted on an mbarrier (bounded wait,
//            error word).  (Per-transform bulk copies of 64 .. 256 bytes were tried first: too small to run at rate.)
//            The swizzle is what makes pass 1's strided reads of several transforms fall on different banks.  Thread
//            blocks are persistent and the tile is double-buffered: the next tile is in flight while this one is transformed.
//   pass 1   L2 threads per transform, thread (transform, t) holds r = R1 t .. R1 t + R1 - 1 (R1 = E2 / L2) for all l:
//            size-L2 transforms over l in registers, written to the exchange area [transform][f2][r].
//   pass 2   lane = transform, warp = f2: a thread reads the E2 values of its (transform, f2), multiplies by
//            w_K^(r f2) (warp-uniform, kept in registers across tiles), does the E2-point transform over r in
//            registers and holds Z[f2 + L2 f1], f1 = 0 .. E2 - 1.  The 32 lanes of a warp hold one frequency of 32
//            CONSECUTIVE transforms, which is a contiguous run of the operand X[problem][col][2 j ..]: every bin is
//            stored straight from registers as one 128-byte (bfloat16 pairs) or 256-byte (float32) line per warp.
// About as many instructions per complex point as the shuffle-based kernel of circ_staged.cu (69 against 70 at k = 64: the
// butterflies, the twiddles, the bfloat16 hi / lo split and the stores are the same work), but none of them waits on a
// shuffle or a conflicting shared-memory access: 32.5 -> 24.8 us for 134 MB at k = 64, 38 -> 27 us at k = 256.  The
// shuffle-based kernel keeps serving small forwards, k <= 16 (where it already runs at the copy rate) and >= 512, and
// embedded block sizes.
#include <type_traits>

#include "circ_tc.cuh"
#include "circ_fft.cuh"
#include "circ_io.cuh"

namespace circ {

constexpr uint32_t kInBulkSpinLimit = 1u << 22;   // bounded wait: polls before giving up

template <int K, typename TIN>
struct InBulk {
    static_assert(K >= 16 && K <= 256 && (K & (K - 1)) == 0, "K = 16 .. 256");
    static_assert(K * sizeof(TIN) >= 128, "a transform fills at least one 128-byte swizzle row");
    static constexpr int E2 = K <= 64 ? 8 : 16;          // points per thread in pass 2 (few registers: many warps per SM)
    static constexpr int L2 = K / E2;                    // size of the pass-1 transform = threads per transform = warps
    static constexpr int R1 = E2 / L2 > 0 ? E2 / L2 : 1; // values of r per thread in pass 1
    static_assert(L2 * R1 == E2 && L2 >= 4, "pass 1 gives every thread K / L2 points; at least four warps");
    static constexpr int TT = 32;                        // transforms per tile: the lanes of pass 2
    static constexpr int NT = 32 * L2;                   // threads per block
    static constexpr int CE = 128 / (int)sizeof(TIN);    // elements per 128-byte chunk
    static constexpr size_t HALF = (size_t)TT * K * sizeof(TIN);     // the real (or imaginary) rows of a tile: a multiple of 1024
    static constexpr size_t BUF = 2 * HALF;                          // one tile buffer
    static constexpr int EXP = (K + 2) * (int)sizeof(float2);        // exchange area: bytes per transform (16 mod 128: 16-byte reads of
    static constexpr size_t EX = (size_t)TT * EXP;                   //   eight transforms fall on different banks)
    static constexpr size_t SMEM = 1024 + 2 * BUF + EX + sizeof(float2) * K + 64;
};

// Element e of tile-local transform tr in a staged half (real or imaginary rows): the TMA wrote 128-byte rows whose
// 16-byte chunks are XOR-swizzled with the row index (the buffer is 1024-byte aligned).
template <int K, typename TIN>
__device__ __forceinline__ const TIN* staged(const unsigned char* half, int tr, int e) {
    const uint32_t off = (uint32_t)(tr * K + e) * (uint32_t)sizeof(TIN);
    const uint32_t row = off >> 7, chunk = (off >> 4) & 7u;
    return reinterpret_cast<const TIN*>(half + (row << 7) + (((chunk ^ (row & 7u)) << 4) | (off & 15u)));
}

__device__ __forceinline__ uint32_t inb_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool inb_wait(uint64_t* bar, uint32_t parity, uint32_t limit) {
    for (uint32_t it = 0; it < limit; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(inb_smem(bar)), "r"(parity) : "memory");
        if (ok) return true;
        if (it > 64) __nanosleep(64);
    }
    return false;
}

// XMODE / TWIN as in circ_staged.cu: 0 float32 operand, 1 split bfloat16 (hi | lo), 2 bfloat16; TWIN: complex problems get
// the two column groups (Zr, -Zi) and (Zi, Zr).
template <int K, typename TIN, int XMODE, bool TWIN>
__global__ void __launch_bounds__(InBulk<K, TIN>::NT)
input_fft_bulk_kernel(const __grid_constant__ CUtensorMap map_x, void* __restrict__ xop, int q, int B, int Bh, int ntiles,
                      int* status, int pdl_late) {
    using S = InBulk<K, TIN>;
    constexpr int L2 = S::L2, R1 = S::R1, E2 = S::E2, TT = S::TT;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* buf0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* exa = buf0 + 2 * S::BUF;
    float2* tw = reinterpret_cast<float2*>(exa + S::EX);
    uint64_t* full = reinterpret_cast<uint64_t*>(tw + K);             // [2]
    const int tid = threadIdx.x, lane = tid & 31;
    const int f2w = tid >> 5;                            // pass 2: this thread's f2 (warp-uniform); its transform of the tile is `lane`

    load_twiddles<K>(tw);
    if (tid == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        for (int b = 0; b < 2; ++b) mbar_init(&full[b], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!pdl_late) pdl_trigger();
    pdl_wait();     // x may come from the kernel before; the operand buffer may still be read by it
    __syncthreads();

    // Tiles: q >= 32: tile = (row c, 32 consecutive column blocks); q < 32: tile = 32 / q consecutive rows.
    const int tiles_per_row = q >= TT ? q / TT : 1, rows_per_tile = q >= TT ? 1 : TT / q;
    auto tile_origin = [&](int tile, int& c0, int& j0) {
        if (q >= TT) {
            c0 = tile / tiles_per_row;
            j0 = (tile - c0 * tiles_per_row) * TT;
        } else {
            c0 = tile * rows_per_tile;
            j0 = 0;
        }
    };
    // one thread fetches the two boxes of a tile: the rows' real parts (rows c) and imaginary parts (rows c + Bh; rows past
    // the batch, i.e. the second sample of the last pair of an odd batch, read as zeros)
    auto fetch = [&](int tile, int b) {
        if (tid != 0) return;
        int c0, j0;
        tile_origin(tile, c0, j0);
        unsigned char* dst = buf0 + (size_t)b * S::BUF;
        mbar_expect_tx(&full[b], (uint32_t)S::BUF);
        tma_load_4d(dst, &map_x, &full[b], 0, j0 * (K / S::CE), c0, 0);
        tma_load_4d(dst + S::HALF, &map_x, &full[b], 0, j0 * (K / S::CE), c0 + Bh, 0);
    };

    // twiddles of pass 2: w_K^(r f2), f2 = this warp
    float2 twr[E2];
#pragma unroll
    for (int r = 0; r < E2; ++r) twr[r] = tw[(r * f2w) & (K - 1)];

    const size_t cols = 2 * (size_t)Bh;
    constexpr int NPART = XMODE == 1 ? 2 : 1;
    const size_t real_sz = cols * q * NPART, cplx_sz = (TWIN ? 4 : 2) * real_sz;      // elements of a real / complex problem of X
    const size_t col_stride_c = (size_t)NPART * 2 * q, col_stride_r = (size_t)NPART * q;

    int tile = blockIdx.x;
    if (tile < ntiles) fetch(tile, 0);
    if (tile + (int)gridDim.x < ntiles) fetch(tile + (int)gridDim.x, 1);
    bool ok = true;
    int it = 0;
    for (; tile < ntiles; tile += gridDim.x, ++it) {
        const int b = it & 1;
        unsigned char* buf = buf0 + (size_t)b * S::BUF;
        ok = inb_wait(&full[b], (uint32_t)(it >> 1) & 1u, kInBulkSpinLimit);
        ok = __syncthreads_and(ok);
        if (!ok) break;
        int c0, j0;
        tile_origin(tile, c0, j0);

        float2 v[E2];
        {
            // ---- pass 1: thread (transform, t): R1 values of r, all l ------------------------------------
            const int tr = tid / L2, t = tid % L2;
            float2 a[R1][L2];
#pragma unroll
            for (int l = 0; l < L2; ++l) {
                // R1 <= 2 consecutive values: they stay inside one 16-byte chunk of the swizzled rows
                const TIN* re = staged<K, TIN>(buf, tr, E2 * l + R1 * t);
                const TIN* im = staged<K, TIN>(buf + S::HALF, tr, E2 * l + R1 * t);
#pragma unroll
                for (int e = 0; e < R1; ++e) a[e][l] = make_float2(to_float(re[e]), to_float(im[e]));
            }
#pragma unroll
            for (int e = 0; e < R1; ++e) fft_registers<L2, false>(a[e]);
            float2* ex = reinterpret_cast<float2*>(exa + (size_t)tr * S::EXP);
#pragma unroll
            for (int f2 = 0; f2 < L2; ++f2) {
                if constexpr (R1 >= 2) {
#pragma unroll
                    for (int e = 0; e < R1; e += 2)
                        *reinterpret_cast<float4*>(&ex[f2 * E2 + R1 * t + e]) = make_float4(a[e][f2].x, a[e][f2].y, a[e + 1][f2].x, a[e + 1][f2].y);
                } else {
                    ex[f2 * E2 + t] = a[0][f2];
                }
            }
            __syncthreads();
            // ---- pass 2: lane = transform, warp = f2 -------------------------------------------------------
            const float4* mine = reinterpret_cast<const float4*>(exa + (size_t)lane * S::EXP) + f2w * (E2 / 2);
#pragma unroll
            for (int r = 0; r < E2; r += 2) {
                const float4 two = mine[r / 2];
                v[r] = r == 0 ? make_float2(two.x, two.y) : cmul(make_float2(two.x, two.y), twr[r]);
                v[r + 1] = cmul(make_float2(two.z, two.w), twr[r + 1]);
            }
        }
        fft_registers<E2, false>(v);
        // this lane's transform: (pair c, column block j); rows past the pairs (q < 32, last tile) are not ours
        const int c = q >= TT ? c0 : c0 + lane / q, j = q >= TT ? j0 + lane : lane % q;
        // the tile's memory is free once every thread has taken its values: refill it two tiles ahead
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tile + 2 * (int)gridDim.x < ntiles) fetch(tile + 2 * (int)gridDim.x, b);
        if (pdl_late && tile + (int)gridDim.x >= ntiles) pdl_trigger();

        // ---- stores: bin f = warp + L2 f1 of transform (c, j); consecutive lanes = consecutive j ----------
        if (c >= Bh) continue;
#pragma unroll
        for (int f1 = 0; f1 < E2; ++f1) {
            const int f = f2w + L2 * f1;                        // warp-uniform
            float2 z = v[f1];
            if (f == 0 || f == K / 2) {
                // real bins: problem 0 / 1, column c takes the first signal's value, column Bh + c the second's
                const size_t base = (f == 0 ? 0 : real_sz) + (size_t)c * col_stride_r + j;
                const size_t other = (size_t)Bh * col_stride_r;
                if constexpr (XMODE == 0) {
                    float* xf = static_cast<float*>(xop);
                    xf[base] = z.x;
                    xf[base + other] = z.y;
                } else {
                    __nv_bfloat16* xb = static_cast<__nv_bfloat16*>(xop);
                    uint32_t lo;
                    const uint32_t hi = bf16_split_pair(z.x, z.y, lo);
                    xb[base] = __ushort_as_bfloat16((unsigned short)(hi & 0xffffu));
                    xb[base + other] = __ushort_as_bfloat16((unsigned short)(hi >> 16));
                    if constexpr (XMODE == 1) {
                        xb[base + q] = __ushort_as_bfloat16((unsigned short)(lo & 0xffffu));
                        xb[base + other + q] = __ushort_as_bfloat16((unsigned short)(lo >> 16));
                    }
                }
            } else {
                const bool mirror = f > K / 2;                  // stored as the conjugate, in the second column group
                const int g = mirror ? K - f : f;
                if (mirror) z.y = -z.y;
                const size_t base = 2 * real_sz + (size_t)(g - 1) * cplx_sz + ((size_t)(mirror ? Bh : 0) + c) * col_stride_c + 2 * (size_t)j;
                if constexpr (XMODE == 0) {
                    *reinterpret_cast<float2*>(static_cast<float*>(xop) + base) = z;
                } else {
                    __nv_bfloat16* d = static_cast<__nv_bfloat16*>(xop) + base;
                    uint32_t lo;
                    const uint32_t hi = bf16_split_pair(z.x, z.y, lo);
                    if constexpr (TWIN) {
                        __nv_bfloat16* d2 = d + cols * col_stride_c;
                        *reinterpret_cast<uint32_t*>(d) = hi ^ 0x80000000u;                      // (Zr, -Zi)
                        *reinterpret_cast<uint32_t*>(d2) = __byte_perm(hi, 0u, 0x1032);          // (Zi, Zr)
                        if constexpr (XMODE == 1) {
                            *reinterpret_cast<uint32_t*>(d + 2 * q) = lo ^ 0x80000000u;
                            *reinterpret_cast<uint32_t*>(d2 + 2 * q) = __byte_perm(lo, 0u, 0x1032);
                        }
                    } else {
                        *reinterpret_cast<uint32_t*>(d) = hi;
                        if constexpr (XMODE == 1) *reinterpret_cast<uint32_t*>(d + 2 * q) = lo;
                    }
                }
            }
        }
    }
    if (!ok) {
        // a wait gave up: report it, and give the copies in flight (this tile's and the next one's) a bounded wait
        // to land before the block's shared memory goes away
        if (tid == 0) atomicExch(status, 1);
        inb_wait(&full[it & 1], (uint32_t)(it >> 1) & 1u, 1u << 16);
        inb_wait(&full[(it + 1) & 1], (uint32_t)((it + 1) >> 1) & 1u, 1u << 16);
    }
}

template <int K, typename TIN, int XMODE, bool TWIN>
static int launch_one(const Layer* L, const void* x, void* xop, const Extent& ext, cudaStream_t stream) {
    using S = InBulk<K, TIN>;
    auto kernel = input_fft_bulk_kernel<K, TIN, XMODE, TWIN>;
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
    const int q = L->geo.q;
    // x as [row][128-byte chunk][chunk elements]; one box = the 32 transforms of a tile: 32 K / CE chunks of one row, or
    // 32 / q whole rows
    CUtensorMap map;
    {
        const int chunks_per_row = L->n / S::CE;
        const int rows = q >= S::TT ? 1 : S::TT / q;
        cuuint64_t dims[4] = {(cuuint64_t)S::CE, (cuuint64_t)chunks_per_row, (cuuint64_t)ext.B, 1};
        cuuint64_t str[3] = {128, (cuuint64_t)L->n * sizeof(TIN), (cuuint64_t)L->n * sizeof(TIN) * ext.B};
        cuuint32_t box[4] = {(cuuint32_t)S::CE, (cuuint32_t)(S::TT * K / S::CE / rows), (cuuint32_t)rows, 1};
        const int rc = encode_tensor_map(&map, const_cast<void*>(x), 4, dims, str, box,
                                         sizeof(TIN) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
        if (rc != CIRC_OK) return rc;
    }
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, L->device);
    const long ntiles = q >= S::TT ? (long)ext.Bh * (q / S::TT) : ((long)ext.Bh + S::TT / q - 1) / (S::TT / q);
    if (ntiles >= (1L << 31)) {
        set_error(CIRC_ERR_SHAPE, "too many transforms");
        return CIRC_ERR_SHAPE;
    }
    const long resident = (long)sms * per_sm;
    const unsigned blocks = (unsigned)(ntiles < resident ? ntiles : resident);
    launch_kernel(dependent_launches(), kernel, dim3(blocks), dim3(S::NT), S::SMEM, stream, map, xop, q, ext.B, ext.Bh, (int)ntiles,
                  L->dev_status, (int)(dependent_launches() == PDL_LATE));
    return CIRC_OK;
}

template <int K, typename TIN>
static int launch_t(const Layer* L, const void* x, void* xop, int xmode, bool twin, const Extent& ext, cudaStream_t stream) {
    if (xmode == 0) return launch_one<K, TIN, 0, false>(L, x, xop, ext, stream);
    if (xmode == 1) return twin ? launch_one<K, TIN, 1, true>(L, x, xop, ext, stream) : launch_one<K, TIN, 1, false>(L, x, xop, ext, stream);
    return twin ? launch_one<K, TIN, 2, true>(L, x, xop, ext, stream) : launch_one<K, TIN, 2, false>(L, x, xop, ext, stream);
}

template <int K>
static int launch_k(const Layer* L, const void* x, void* xop, int xmode, bool twin, const Extent& ext, cudaStream_t stream) {
    if (L->x_dtype == CIRC_BF16) {
        if constexpr (K >= 64) return launch_t<K, __nv_bfloat16>(L, x, xop, xmode, twin, ext, stream);
        set_error(CIRC_ERR_UNSUPPORTED, "bfloat16 blocks below 64 are not served by the TMA-staged input transforms");
        return CIRC_ERR_UNSUPPORTED;
    }
    return launch_t<K, float>(L, x, xop, xmode, twin, ext, stream);
}

// Large forwards of power-of-two blocks whose transform fills at least one 128-byte row (float32: k >= 32, bfloat16:
// k >= 64), up to k = 256, with column-block counts that tile evenly (q a multiple of 32, or a divisor of it).
bool input_fft_bulk_supported(const Layer* L, const void* x, long total) {
    const int k = L->geo.k, q = L->geo.q;
    const int kmin = L->x_dtype == CIRC_BF16 ? 64 : 32;
    return !embedded(L->geo) && k >= kmin && k <= 256 && (q % 32 == 0 || (32 % q == 0 && q % 8 == 0)) && total >= 148L * 64 &&
           (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && L->dev_status != nullptr && tensor_map_encoder() != nullptr;
}

int launch_input_fft_bulk(const Layer* L, const void* x, void* xop, int xmode, bool twin, const Extent& ext, cudaStream_t stream) {
    int rc;
    switch (L->geo.k) {
        case 32: rc = launch_k<32>(L, x, xop, xmode, twin, ext, stream); break;
        case 64: rc = launch_k<64>(L, x, xop, xmode, twin, ext, stream); break;
        case 128: rc = launch_k<128>(L, x, xop, xmode, twin, ext, stream); break;
        case 256: rc = launch_k<256>(L, x, xop, xmode, twin, ext, stream); break;
        default: set_error(CIRC_ERR_SHAPE, "block size %d not served by the bulk-staged input transforms", L->geo.k); return CIRC_ERR_SHAPE;
    }
    if (rc != CIRC_OK) return rc;
    L->last_kernels[0] = KERNEL_S1_BULK;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
