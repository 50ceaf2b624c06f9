// S2 on the tensor cores for fully-connected layers with FEW columns and MANY row blocks: the weight-streaming
// regime between the one-launch kernel (batch <= 8) and the large-batch contraction of circ_tensor.cu.
//
// There the forward is bound by reading the weight spectra once, and the large-batch kernel is a poor fit: it
// puts the batch columns on the 128-row side of the MMA, so with 64 columns half of every instruction is padding,
// and it has few, long tiles.  This kernel turns the product around,
//     Y^T[row][col] = sum_kk A[row][kk] * X[col][kk],
//   * 128 WEIGHT ROWS are the MMA's M dimension (tensor-memory lanes), the batch columns its N dimension
//     (16 .. 256, all columns of the problem in one tile), the contraction index is K;
//   * one tile = (frequency problem, 128 weight rows): every weight is fetched from memory exactly once, by TMA
//     (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into a ring of shared-memory stages that keeps about
//     100 KB of the weight stream in flight per SM; X (a few MB) is re-read per tile from the L2;
//   * float32 inputs: split bfloat16 operands and the three products hi*hi + hi*lo + lo*hi, as in circ_tensor.cu;
//   * the contraction range of a tile is cut into equal pieces (twice as many for a complex problem, whose range is
//     twice as long), one piece = one work unit, so that all SMs carry the same number of bytes: a forward like this
//     is bound by what one SM can pull in, and whole tiles of two lengths left half the machine waiting.  Each
//     piece writes its partial result to its own copy of Y; the inverse-transform kernel adds the copies in a fixed
//     order (bitwise repeatable, no atomics);
//   * the epilogue needs no turn-around: a lane of tensor memory is a weight row, rows are contiguous in
//     Y[col][row], so the 32 lanes of a warp store 128 contiguous bytes per column.
// With twin columns (circ_common.cuh: use_twin) a complex problem has p rows of (Wr, Wi) pairs and 2 x cols columns.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and tensor-memory owner, warps 2..5 = epilogue.  Every wait
// is bounded: on expiry the block records an error word, drains its copies, frees its tensor memory and returns.
#include "circ_tc.cuh"

namespace circ {

constexpr int kRowsThreads = 192;
constexpr int kRowsTile = 128;            // MMA M: weight rows per tile
constexpr int kRowsKBlock = 64;           // bf16 elements per stage along K (one 128-byte swizzle row)
constexpr int kRowsMaxStages = 8;

struct RowsArgs {
    float* yop;
    int* status;
    int p, q, k;
    int nsplit;              // parts of each operand: 2 (hi, lo) or 1
    int npass;               // products per K step: 3 (float32 inputs) or 1 (bfloat16 inputs)
    int cols_r, cols_c;      // columns of a real / complex problem (complex: twice the real ones with twin columns)
    int nr, nc;              // the same rounded up to the MMA's N granularity (16)
    int rows_c;              // rows of a complex problem: p (twin) or 2p (embedded)
    int nt_r, nt_c;          // 128-row tiles per real / complex problem
    int splits_r, splits_c;  // pieces of the contraction range of a real / complex tile
    int units_c;             // complex work units (tile x piece); they come first
    int tiles;               // all work units; thread blocks walk them with a grid stride
    long y_copy;             // floats between the copies of Y that the pieces write
    int stages;              // depth of the shared-memory ring
    uint32_t acc_cols;       // tensor-memory columns of one accumulator (power of two >= 32)
    uint32_t spin_limit;
    int pdl_late;
    int no_copy;             // fault injection (tests only): the producer announces its bytes but issues no copy
};

struct RowsTile {
    bool real;
    int prob_in_kind, prob, row0, Mg, Kq, cols, npad, piece, kb0, kb1;
};
__device__ __forceinline__ RowsTile rows_decode(const RowsArgs& g, int unit) {
    RowsTile t;
    t.real = unit >= g.units_c;
    int u = t.real ? unit - g.units_c : unit;
    const int splits = t.real ? g.splits_r : g.splits_c;
    t.piece = u % splits;
    u /= splits;
    const int nt = t.real ? g.nt_r : g.nt_c;
    t.prob_in_kind = u / nt;
    t.row0 = (u - t.prob_in_kind * nt) * kRowsTile;
    t.prob = t.real ? t.prob_in_kind : 2 + t.prob_in_kind;
    t.Mg = t.real ? g.p : g.rows_c;
    t.Kq = t.real ? g.q : 2 * g.q;
    t.cols = t.real ? g.cols_r : g.cols_c;
    t.npad = t.real ? g.nr : g.nc;
    const int kblocks = (t.Kq + kRowsKBlock - 1) / kRowsKBlock;
    t.kb0 = t.piece * kblocks / splits;         // even cut; the host never makes more pieces than K blocks: kb0 < kb1
    t.kb1 = (t.piece + 1) * kblocks / splits;
    return t;
}

// Instruction descriptor: bf16 x bf16 -> f32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t rows_instr_desc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kRowsTile >> 4) << 24);
}

__global__ void __launch_bounds__(kRowsThreads, 1)
contract_rows_kernel(const __grid_constant__ CUtensorMap map_a_real, const __grid_constant__ CUtensorMap map_a_cplx,
                     const __grid_constant__ CUtensorMap map_xhi_real, const __grid_constant__ CUtensorMap map_xlo_real,
                     const __grid_constant__ CUtensorMap map_xhi_cplx, const __grid_constant__ CUtensorMap map_xlo_cplx,
                     RowsArgs g) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t full_bar[kRowsMaxStages], empty_bar[kRowsMaxStages], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_max = g.nr > g.nc ? g.nr : g.nc;
    const uint32_t x_bytes = (uint32_t)n_max * 128;                 // one part of the X tile (all columns x 64 K)
    const uint32_t a_bytes = (uint32_t)kRowsTile * 128;             // one part of the weight tile
    const uint32_t stage_bytes = (uint32_t)g.nsplit * (x_bytes + a_bytes);
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const uint32_t tmem_cols = 2 * g.acc_cols;

    if (warp == 0 && lane == 0) {
        const CUtensorMap* maps[6] = {&map_a_real, &map_a_cplx, &map_xhi_real, &map_xhi_cplx, &map_xlo_real, &map_xlo_cplx};
#pragma unroll
        for (int i = 0; i < 6; ++i)
            if (i < 4 || g.nsplit == 2) asm volatile("prefetch.tensormap [%0];" ::"l"(maps[i]) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 4);         // one arrival per epilogue warp
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_base_slot, tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    if (!g.pdl_late) pdl_trigger();

    if (warp == 0) {
        // ---- TMA producer -----------------------------------------------------------------------
        if (lane == 0) {
            int s = 0, issued = 0;
            uint32_t par = 0;
            bool wrapped = false, ok = true;
            // The weights were written when the layer was made: their copies do not depend on the kernel before this
            // one.  The first trip around the ring therefore announces its bytes and fetches its weight tiles before
            // waiting for that kernel; the X tiles of those stages follow after the wait.
            int ahead = 0;
            if (!g.no_copy) {
                for (int tile = blockIdx.x; tile < g.tiles && ahead < g.stages; tile += gridDim.x) {
                    const RowsTile t = rows_decode(g, tile);
                    const uint32_t tx_bytes = (uint32_t)g.nsplit * ((uint32_t)t.npad * 128 + a_bytes);
                    for (int kb = t.kb0; kb < t.kb1 && ahead < g.stages; ++kb, ++ahead) {
                        unsigned char* as = ring + (size_t)ahead * stage_bytes + (size_t)g.nsplit * x_bytes;
                        mbar_expect_tx(&full_bar[ahead], tx_bytes);
                        tma_load_4d(as, t.real ? &map_a_real : &map_a_cplx, &full_bar[ahead], kb * kRowsKBlock, t.row0, 0, t.prob_in_kind);
                    }
                }
            }
            pdl_wait();                              // X is written by the transform kernel before this one
            int it = 0;
            for (int tile = blockIdx.x; tile < g.tiles && ok; tile += gridDim.x) {
                const RowsTile t = rows_decode(g, tile);
                const CUtensorMap* map_a = t.real ? &map_a_real : &map_a_cplx;
                const CUtensorMap* map_xhi = t.real ? &map_xhi_real : &map_xhi_cplx;
                const CUtensorMap* map_xlo = t.real ? &map_xlo_real : &map_xlo_cplx;
                const uint32_t tx_bytes = (uint32_t)g.nsplit * ((uint32_t)t.npad * 128 + a_bytes);
                for (int kb = t.kb0; kb < t.kb1; ++kb, ++it) {
                    if (wrapped) ok = mbar_wait(&empty_bar[s], par ^ 1u, &abort_flag, g.spin_limit);
                    if (!ok) break;
                    unsigned char* xs = ring + (size_t)s * stage_bytes;
                    unsigned char* as = xs + (size_t)g.nsplit * x_bytes;
                    if (it >= ahead) mbar_expect_tx(&full_bar[s], tx_bytes);
                    if (g.no_copy) {                 // fault injection: nothing is in flight, the consumer's wait runs out
                        ok = false;
                        issued = 0;
                        break;
                    }
                    // [part][row][128 B]: hi parts first, then lo parts
                    if (it >= ahead) tma_load_4d(as, map_a, &full_bar[s], kb * kRowsKBlock, t.row0, 0, t.prob_in_kind);
                    tma_load_4d(xs, map_xhi, &full_bar[s], kb * kRowsKBlock, 0, t.prob_in_kind, 0);
                    if (g.nsplit == 2) tma_load_4d(xs + x_bytes, map_xlo, &full_bar[s], kb * kRowsKBlock, 0, t.prob_in_kind, 0);
                    if (issued < g.stages) ++issued;
                    if (++s == g.stages) {
                        s = 0;
                        par ^= 1u;
                        wrapped = true;
                    }
                }
            }
            if (!ok) {
                // drain: every copy that was issued must land before the block may go away
                int ds = s;
                uint32_t dpar = par;
                for (int n = 0; n < issued; ++n) {
                    if (ds == 0) {
                        ds = g.stages;
                        dpar ^= 1u;
                    }
                    --ds;
                    for (uint32_t spin = 0; spin < g.spin_limit && !mbar_try_wait(&full_bar[ds], dpar); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer (all lanes walk the loop; one elected lane issues) ---------------------------
        const uint32_t leader = elect_one();
        int s = 0, buf = 0;
        uint32_t par = 0, acc_par = 0;
        bool acc_wrapped = false, ok = true;
        for (int tile = blockIdx.x; tile < g.tiles && ok; tile += gridDim.x) {
            const RowsTile t = rows_decode(g, tile);
            const uint32_t idesc = rows_instr_desc(t.npad);
            if (acc_wrapped) ok = mbar_wait(&acc_empty[buf], acc_par ^ 1u, &abort_flag, g.spin_limit);   // epilogue done with it
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)buf * g.acc_cols;
            uint32_t accumulate = 0;
            for (int kb = t.kb0; kb < t.kb1; ++kb) {
                ok = mbar_wait(&full_bar[s], par, &abort_flag, g.spin_limit);
                if (!ok) break;
                tc_fence_after();
                const uint32_t xs = smem_u32(ring + (size_t)s * stage_bytes);
                const uint32_t as = xs + (uint32_t)g.nsplit * x_bytes;
                const int krem = t.Kq - kb * kRowsKBlock;
                const int ksteps = krem >= kRowsKBlock ? kRowsKBlock / 16 : (krem + 15) / 16;   // the rest of the block is zero fill
                if (leader) {
                    // A operand of the MMA = weight tile (128 rows), B operand = X tile (N columns)
                    const uint64_t dwh = smem_desc_sw128(as), dxh = smem_desc_sw128(xs);
                    const uint64_t dwl = dwh + (uint64_t)(a_bytes >> 4), dxl = dxh + (uint64_t)(x_bytes >> 4);
                    for (int k4 = 0; k4 < ksteps; ++k4) {
                        tc_mma_bf16(d_tmem, dwh + 2 * k4, dxh + 2 * k4, idesc, accumulate);
                        accumulate = 1u;
                    }
                    if (g.npass == 3) {
                        for (int k4 = 0; k4 < ksteps; ++k4) tc_mma_bf16(d_tmem, dwl + 2 * k4, dxh + 2 * k4, idesc, 1u);
                        for (int k4 = 0; k4 < ksteps; ++k4) tc_mma_bf16(d_tmem, dwh + 2 * k4, dxl + 2 * k4, idesc, 1u);
                    }
                    tc_commit(&empty_bar[s]);   // stage free once these MMAs have read it
                    if (kb + 1 == t.kb1) tc_commit(&acc_full[buf]);   // accumulator complete
                }
                accumulate = 1u;
                if (++s == g.stages) {
                    s = 0;
                    par ^= 1u;
                }
            }
            if (++buf == 2) {
                buf = 0;
                acc_par ^= 1u;
                acc_wrapped = true;
            }
        }
    } else {
        // ---- epilogue: tensor memory -> registers -> Y[col][row] ------------------------------------
        // lane of tensor memory = weight row; the warp's 32 rows are contiguous in Y for every column
        const int quarter = warp & 3;                 // a warp may only read its own 32 lanes
        int buf = 0;
        uint32_t acc_par = 0;
        const size_t y_real = (size_t)g.cols_r * g.p;
        for (int tile = blockIdx.x; tile < g.tiles; tile += gridDim.x) {
            const RowsTile t = rows_decode(g, tile);
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[buf], acc_par, &abort_flag, g.spin_limit));  // warp-uniform
            if (!ok) break;
            tc_fence_after();
            const int row = t.row0 + quarter * 32 + lane;
            float* yrow = g.yop + (size_t)t.piece * g.y_copy + problem_offset(t.prob, y_real, 2 * y_real) + row;
            for (int c0 = 0; c0 < t.npad; c0 += 32) {
                uint32_t acc[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * g.acc_cols + (uint32_t)c0, acc);
                if (c0 + 32 >= t.npad) {
                    // last read of this accumulator: it may be overwritten by the tile after next
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[buf]);
                }
                if (row < t.Mg) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c0 + e < t.cols) yrow[(size_t)(c0 + e) * t.Mg] = __uint_as_float(acc[e]);
                }
            }
            if (++buf == 2) {
                buf = 0;
                acc_par ^= 1u;
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------
    if (g.pdl_late) pdl_trigger();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(g.status, 1);
}

// ---- host side ---------------------------------------------------------------------------------
static int rows_tiles(const Layer* L, bool twin) {
    const int p = L->geo.p, k = L->geo.k;
    const int rows_c = twin ? p : 2 * p;
    return 2 * ((p + kRowsTile - 1) / kRowsTile) + (k / 2 - 1) * ((rows_c + kRowsTile - 1) / kRowsTile);
}

// How the tensor-core contraction of a forward runs.  The row-streaming kernel serves a fully-connected forward
// when all columns of a problem fit one MMA (N <= 256) and there are enough 128-row tiles to keep the memory system
// busy; twin columns (weights read once, X twice) when the layer has at least twice as many row blocks as columns.
ContractionPlan plan_contraction(const Layer* L, const Extent& e) {
    ContractionPlan pl = {false, false};
    if (L->kind != 0) return pl;
    const long cols = 2L * e.Bh;
    const bool twin_ok = !L->no_twin && !embedded(L->geo) && L->geo.p >= 16 && (long)L->geo.p >= 2 * cols && L->geo.q % 8 == 0;
    const bool rows_ok = !L->no_rows_kernel;
    if (rows_ok && twin_ok && 2 * cols <= 256 && rows_tiles(L, true) >= 64) return ContractionPlan{true, true};
    if (rows_ok && cols <= 256 && rows_tiles(L, false) >= 64) return ContractionPlan{false, true};
    pl.twin = twin_ok && cols <= 512;
    return pl;
}

// Pieces per real and per complex tile.  A forward like this is bound by what one SM can take in (a ring of stages per
// SM, about 60 GB/s each on B200 whatever the depth beyond 130 KB in flight), so the pieces are chosen to give every SM
// the same number of bytes: for each pair of counts, the units (complex ones first) are dealt to the thread blocks with
// the kernel's grid stride and the block with the most bytes sets the time; every extra copy of Y costs the inverse
// transforms one more read of Y.  The cheapest pair wins.  (16384 x 16384, k = 4, batch 64, float32: equal-length
// pieces (1, 2): 62.2 us; byte-balanced (2, 5): 57.4 us.)
RowsPieces rows_pieces(const Layer* L, const Extent& e, bool twin) {
    const int p = L->geo.p, q = L->geo.q, k = L->geo.k;
    const int rows_c = twin ? p : 2 * p;
    const long tiles_r = 2L * ((p + kRowsTile - 1) / kRowsTile), tiles_c = (long)(k / 2 - 1) * ((rows_c + kRowsTile - 1) / kRowsTile);
    const int kblocks_r = (q + kRowsKBlock - 1) / kRowsKBlock, kblocks_c = (2 * q + kRowsKBlock - 1) / kRowsKBlock;
    const double parts = L->x_dtype == CIRC_BF16 ? 1.0 : 2.0;
    const double cols_r = 2.0 * e.Bh, cols_c = twin ? 2.0 * cols_r : cols_r;
    // bytes of one K block of a real / complex unit: the weight tile and the X tile
    const double blk_r = parts * 128.0 * (kRowsTile + cols_r), blk_c = parts * 128.0 * (kRowsTile + cols_c);
    const double y_bytes = 4.0 * cols_r * p * k;                  // one copy of Y
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, L->device);
    RowsPieces best = {1, 1};
    double best_cost = -1.0;
    for (int sr = 1; sr <= 4 && sr <= kblocks_r; ++sr) {
        for (int sc = 1; sc <= 8 && sc <= kblocks_c; ++sc) {
            if (tiles_c == 0 && sc > 1) break;
            const double ur = blk_r * ((kblocks_r + sr - 1) / sr), uc = blk_c * ((kblocks_c + sc - 1) / sc);
            const long nr = tiles_r * sr, nc = tiles_c * sc;
            const long n = nr + nc;
            const long full = n / sms, rest = n % sms;             // every block `full` units, the first `rest` one more
            auto unit_bytes = [&](long u) { return u < nc ? uc : ur; };
            double worst = 0.0;
            for (long b = 0; b < (n < sms ? n : sms); b += (sms > 8 ? (sms - 1) / 4 : 1)) {   // a few sample blocks, first and last included
                double t = 0.0;
                for (long j = 0; j < full + (b < rest ? 1 : 0); ++j) t += unit_bytes(b + j * sms);
                if (t > worst) worst = t;
            }
            const double cost = worst * sms + 2.0 * y_bytes * (sc > sr ? sc : sr);   // both in "bytes through the whole machine"
            if (best_cost < 0 || cost < best_cost * 0.97) {
                best_cost = cost;
                best = RowsPieces{sr, sc};
            }
        }
    }
    return best;
}

int launch_contract_rows(const Layer* L, const __nv_bfloat16* xb, float* yop, const Extent& ext, int nsplit, cudaStream_t stream, bool twin) {
    const int p = L->geo.p, q = padded_q(L->geo.q), k = L->geo.k;   // q: the (padded) run length of the operands
    const __nv_bfloat16* a_op = twin ? L->a_twin : L->a_bf16;
    if (!a_op || L->kind != 0) {
        set_error(CIRC_ERR_ARG, "the stored form of the spectra for this contraction has not been built, or not a fully-connected layer");
        return CIRC_ERR_ARG;
    }
    RowsArgs g;
    g.yop = yop;
    g.status = L->dev_status;
    g.p = p; g.q = q; g.k = k;
    g.nsplit = nsplit;
    g.npass = nsplit == 2 ? 3 : 1;
    g.cols_r = 2 * ext.Bh;
    g.cols_c = twin ? 2 * g.cols_r : g.cols_r;
    g.nr = (g.cols_r + 15) & ~15;
    g.nc = (g.cols_c + 15) & ~15;
    if (g.nc > 256) {
        set_error(CIRC_ERR_UNSUPPORTED, "%d columns do not fit one tile of the row-streaming contraction", g.cols_c);
        return CIRC_ERR_UNSUPPORTED;
    }
    g.rows_c = twin ? p : 2 * p;
    g.nt_r = (p + kRowsTile - 1) / kRowsTile;
    g.nt_c = (g.rows_c + kRowsTile - 1) / kRowsTile;
    const RowsPieces pieces = rows_pieces(L, ext, twin);
    g.splits_r = pieces.real;
    g.splits_c = pieces.cplx;
    g.units_c = (k / 2 - 1) * g.nt_c * g.splits_c;
    g.tiles = g.units_c + 2 * g.nt_r * g.splits_r;
    g.y_copy = (long)g.cols_r * p * k;           // all problems of Y: 2 real ones and k/2 - 1 complex ones of twice the size
    g.spin_limit = kSpinLimit;
    g.no_copy = L->inject == INJECT_TENSOR_NO_COPY;
    if (g.no_copy) g.spin_limit = 1u << 12;
    g.pdl_late = dependent_launches() == PDL_LATE;
    g.acc_cols = 32;
    while ((int)g.acc_cols < g.nc) g.acc_cols <<= 1;

    const size_t stage_bytes = (size_t)nsplit * ((size_t)g.nc * 128 + (size_t)kRowsTile * 128);
    g.stages = (int)((196 * 1024) / stage_bytes);
    if (g.stages > kRowsMaxStages) g.stages = kRowsMaxStages;
    if (g.stages < 2) {
        set_error(CIRC_ERR_UNSUPPORTED, "a stage of %zu bytes leaves no room for a ring", stage_bytes);
        return CIRC_ERR_UNSUPPORTED;
    }
    const size_t smem = (size_t)g.stages * stage_bytes + 1024;

    // tensor maps.  A: [problem][row][hi|lo][Kq]; X: [problem][col][hi|lo][Kq]
    CUtensorMap ma_r, ma_c, mxh_r, mxl_r, mxh_c, mxl_c;
    const size_t a_real_elems = (size_t)p * 2 * q;  // one real problem of A (hi and lo)
    int rc;
    {
        cuuint64_t dims[4] = {(cuuint64_t)q, (cuuint64_t)p, 2, 2};
        cuuint64_t str[3] = {(cuuint64_t)2 * q * 2, (cuuint64_t)q * 2, (cuuint64_t)a_real_elems * 2};
        cuuint32_t box[4] = {kRowsKBlock, kRowsTile, (cuuint32_t)nsplit, 1};
        if ((rc = encode_tensor_map(&ma_r, const_cast<__nv_bfloat16*>(a_op), 4, dims, str, box)) != CIRC_OK) return rc;
    }
    const int ncp = k / 2 - 1 > 0 ? k / 2 - 1 : 1;
    {
        cuuint64_t dims[4] = {(cuuint64_t)2 * q, (cuuint64_t)g.rows_c, 2, (cuuint64_t)ncp};
        cuuint64_t str[3] = {(cuuint64_t)2 * 2 * q * 2, (cuuint64_t)2 * q * 2, (cuuint64_t)(twin ? 2 : 4) * a_real_elems * 2};
        cuuint32_t box[4] = {kRowsKBlock, kRowsTile, (cuuint32_t)nsplit, 1};
        if ((rc = encode_tensor_map(&ma_c, const_cast<__nv_bfloat16*>(a_op) + 2 * a_real_elems, 4, dims, str, box)) != CIRC_OK) return rc;
    }
    const size_t x_real_elems = (size_t)g.cols_r * nsplit * q;
    __nv_bfloat16* xbase = const_cast<__nv_bfloat16*>(xb);
    {
        cuuint64_t dims[4] = {(cuuint64_t)q, (cuuint64_t)g.cols_r, 2, 1};
        cuuint64_t str[3] = {(cuuint64_t)nsplit * q * 2, (cuuint64_t)x_real_elems * 2, (cuuint64_t)2 * x_real_elems * 2};
        cuuint32_t box[4] = {kRowsKBlock, (cuuint32_t)g.nr, 1, 1};
        if ((rc = encode_tensor_map(&mxh_r, xbase, 4, dims, str, box)) != CIRC_OK) return rc;
        if ((rc = encode_tensor_map(&mxl_r, xbase + (nsplit == 2 ? q : 0), 4, dims, str, box)) != CIRC_OK) return rc;
    }
    {
        const size_t x_cplx_elems = (size_t)g.cols_c * nsplit * 2 * q;
        cuuint64_t dims[4] = {(cuuint64_t)2 * q, (cuuint64_t)g.cols_c, (cuuint64_t)ncp, 1};
        cuuint64_t str[3] = {(cuuint64_t)nsplit * 2 * q * 2, (cuuint64_t)x_cplx_elems * 2, (cuuint64_t)ncp * x_cplx_elems * 2};
        cuuint32_t box[4] = {kRowsKBlock, (cuuint32_t)g.nc, 1, 1};
        __nv_bfloat16* base = xbase + 2 * x_real_elems;
        if ((rc = encode_tensor_map(&mxh_c, base, 4, dims, str, box)) != CIRC_OK) return rc;
        if ((rc = encode_tensor_map(&mxl_c, base + (nsplit == 2 ? 2 * q : 0), 4, dims, str, box)) != CIRC_OK) return rc;
    }

    static thread_local int configured_device = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        CIRC_CUDA_TRY(cudaFuncSetAttribute(contract_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024), CIRC_ERR_CUDA);
        configured_device = dev;
    }
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, L->device);
    const unsigned grid = (unsigned)(g.tiles < sms ? g.tiles : sms);
    launch_kernel(dependent_launches(), contract_rows_kernel, dim3(grid), dim3(kRowsThreads), smem, stream, ma_r, ma_c, mxh_r, mxl_r, mxh_c,
                  mxl_c, g);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
