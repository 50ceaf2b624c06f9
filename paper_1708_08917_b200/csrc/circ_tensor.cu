// S2 / C2 on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory).
//
// For every frequency problem (circ_common.cuh) the contraction
//     Y[col][row] = sum_{tap, kk} A[row][tap][kk] * X[col shifted by tap][kk]
// is a dense product once the batch (or the pixel count) is large.  One CTA computes one
// 128-column x BN-row output tile:
//   * the 128 batch columns / output pixels are the MMA's M dimension (TMEM lanes),
//     the weight rows are its N dimension (TMEM columns), the contraction index is K;
//   * operands are bfloat16, K-major, fetched by TMA (cp.async.bulk.tensor, 128-byte swizzle,
//     no multicast) into a ring of shared-memory stages guarded by mbarriers;
//   * a convolution loads ONE input tile with its halo per K block -- a TMA box over the (W, H,
//     image) dimensions of X whose out-of-image pixels are the zero fill of the copy (Eq. 6 with
//     zero padding) -- and every filter tap multiplies a row-shifted view of that same tile
//     (the MMA's row index is the flattened halo-tile pixel index, so a tap is a start offset);
//   * float32 inputs use the split  a = a_hi + a_lo  (two bfloat16 values, 16 mantissa bits):
//     a stage holds the hi and lo parts of both operands for one K block and the three products
//     hi*hi + lo*hi + hi*lo go into the same float32 accumulator; bfloat16 inputs have the hi
//     part only and take the single hi*hi product.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 = epilogue
// (tcgen05.ld -> registers -> global).  Every wait is bounded: on expiry the CTA records an error
// word, drains its copies, frees its tensor memory and returns.
#include "circ_tc.cuh"

namespace circ {

constexpr int kTcThreads = 192;
constexpr int kTileCols = 128;            // MMA M: batch columns / pixels per tile
constexpr int kKBlock = 64;               // bf16 elements per stage along K (one 128-byte swizzle row)
constexpr int kMaxAcc = 8;           // accumulators in tensor memory (chosen per launch: as many as 512 columns hold)
constexpr int kMaxStages = 8;        // ring depth is chosen per launch (as many stages as shared memory holds)
constexpr int kStagePitch = 36;           // floats per row of the epilogue's 32 x 32 staging tiles (16-byte aligned, conflict-free)
constexpr int kStageOutBytes = 4 * 32 * kStagePitch * 4;   // one staging tile per epilogue warp

struct TcArgs {
    float* yop;
    int* status;
    int p, q, k, taps, r, pad;
    int nsplit;              // parts of X per column: 2 (hi, lo) or 1
    int npass;               // products per K block: 3 (float32 inputs) or 1 (bfloat16 inputs)
    int W, H, V;             // input image (FC: W = columns, H = V = 1)
    int Wo, Ho;              // output image
    int tw, th;              // output pixels per tile (tw wide, th high)
    int pitch;               // input tile row pitch in pixels: tw + r - 1 (halo included)
    int xrows;               // pixels of the input tile that the TMA box brings: pitch * (th + r - 1)
    int xalloc;              // pixels reserved per sub-tile of the input tile (whole swizzle groups)
    int xtail;               // pixels reserved behind the last sub-tile of a part, so that every tap's 128-row view stays inside the stage
    int tiles_w, tiles_h;    // tiles per image (real problems)
    int twin;                // complex problems in twin-column form: p rows, columns [real parts | imaginary parts]
    int Wo_c, tiles_w_c;     // output columns and column tiles of a complex problem (twice the real ones when twin)
    int bn_real, bn_cplx;    // rows per tile (multiple of 16, <= 256)
    int nt_real, nt_cplx;    // row tiles per problem
    int ctas_real;           // CTAs that serve the two real problems
    int stages;              // depth of the shared-memory ring (<= kMaxStages)
    int nacc;                // accumulators in tensor memory (2 .. kMaxAcc)
    long tiles;              // output tiles in total; CTAs walk them with a grid stride
    long cols_out;           // V * Ho * Wo
    uint32_t spin_limit;     // polls before a wait gives up (kSpinLimit; a few thousand under fault injection)
    int pdl_late;            // issue the dependent-launch trigger after the CTA's last tile instead of first thing
    int no_copy;             // fault injection (tests only): the producer announces its bytes but issues no copy
    int stride;              // strided convolution: output pixel (i, j) reads input pixels (stride i + di - pad, stride j + dj - pad)
    int sp, nph;             // phases per direction min(stride, r) and in all (sp * sp): the input tile comes as one
                             // sub-tile per phase (a, b) = (row, column) offset modulo the stride, each fetched by a
                             // strided TMA box; tap (di, dj) reads sub-tile (di % stride, dj % stride) shifted by
                             // (di / stride, dj / stride).  stride 1: one sub-tile, the tile with its halo.
};

// Instruction descriptor: bf16 x bf16 -> f32, both operands K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t instr_desc(int bn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kTileCols >> 4) << 24);
}

// Where a tile sits: which problem, which row tile, which spatial tile.
struct TileCoord {
    bool real;
    int prob_in_kind, prob, row0, bn, Mg, Kq, v, ho0, wo0, Wo;
};
// 32-bit arithmetic only: the roles that call this are single threads on the critical path
// (the host refuses launches with 2^31 tiles or more).
__device__ __forceinline__ TileCoord decode_tile(const TcArgs& g, long tile) {
    TileCoord t;
    unsigned cta = (unsigned)tile;
    // complex tiles (twice the contraction length) come first, so that a grid with more tiles than thread blocks
    // ends on the short ones
    const unsigned ctas_cplx = (unsigned)g.tiles - (unsigned)g.ctas_real;
    t.real = cta >= ctas_cplx;
    if (t.real) cta -= ctas_cplx;
    const unsigned tiles_w = (unsigned)(t.real ? g.tiles_w : g.tiles_w_c);
    const unsigned sp_tiles = (unsigned)(g.V * g.tiles_h) * tiles_w;
    const unsigned nt = (unsigned)(t.real ? g.nt_real : g.nt_cplx);
    const unsigned pr = cta / sp_tiles;              // problem * nt + row tile
    unsigned sp = cta - pr * sp_tiles;
    unsigned row_tile;
    if (nt == 1) {
        t.prob_in_kind = (int)pr;
        row_tile = 0;
    } else {
        t.prob_in_kind = (int)(pr / nt);
        row_tile = pr - (unsigned)t.prob_in_kind * nt;
    }
    const unsigned per_img = (unsigned)g.tiles_h * tiles_w;
    t.v = (int)(sp / per_img);
    sp -= (unsigned)t.v * per_img;
    const unsigned th_i = tiles_w == 1 ? sp : sp / tiles_w;
    const unsigned tw_i = sp - th_i * tiles_w;
    t.ho0 = (int)th_i * g.th;
    t.wo0 = (int)tw_i * g.tw;
    t.bn = t.real ? g.bn_real : g.bn_cplx;
    t.Mg = (t.real || g.twin) ? g.p : 2 * g.p;
    t.Kq = t.real ? g.q : 2 * g.q;
    t.Wo = t.real ? g.Wo : g.Wo_c;
    t.row0 = (int)row_tile * t.bn;
    t.prob = t.real ? t.prob_in_kind : 2 + t.prob_in_kind;
    return t;
}


// Issue the MMAs of one product (one X part against one A part) for all R x R taps of a K block.
// R is a compile-time filter size so that the tap loops unroll and the single issuing thread
// spends its time on tcgen05.mma, not on loop bookkeeping.  Descriptors differ only in their
// start-address field (16-byte units): 8 units per tile row, a_step per tap, 2 per K step.
template <int R, int KSTEPS>
__device__ __forceinline__ void issue_taps(uint32_t d_tmem, uint64_t dx, uint64_t da, uint64_t row_step, uint64_t a_step,
                                           uint32_t idesc, uint32_t& accumulate) {
#pragma unroll
    for (int di = 0; di < R; ++di) {
#pragma unroll
        for (int dj = 0; dj < R; ++dj) {
            const uint64_t x = dx + (uint64_t)di * row_step + (uint64_t)(dj * 8);
            const uint64_t w = da + (uint64_t)(di * R + dj) * a_step;
            tc_mma_bf16(d_tmem, x, w, idesc, accumulate);
#pragma unroll
            for (int k4 = 1; k4 < KSTEPS; ++k4) tc_mma_bf16(d_tmem, x + 2 * k4, w + 2 * k4, idesc, 1u);
            accumulate = 1u;
        }
    }
}
template <int R>
__device__ __forceinline__ void issue_taps_k(int ksteps, uint32_t d_tmem, uint64_t dx, uint64_t da, uint64_t row_step,
                                             uint64_t a_step, uint32_t idesc, uint32_t& accumulate) {
    switch (ksteps) {
        case 1: issue_taps<R, 1>(d_tmem, dx, da, row_step, a_step, idesc, accumulate); break;
        case 2: issue_taps<R, 2>(d_tmem, dx, da, row_step, a_step, idesc, accumulate); break;
        case 3: issue_taps<R, 3>(d_tmem, dx, da, row_step, a_step, idesc, accumulate); break;
        default: issue_taps<R, 4>(d_tmem, dx, da, row_step, a_step, idesc, accumulate); break;
    }
}

// Persistent: each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...  The three roles run
// ahead of one another: the producer keeps the shared-memory ring full across tile boundaries, the
// MMA warp cycles through the accumulators in tensor memory (2 to 8, as many as its 512 columns hold), and
// the epilogue warps drain one accumulator while the following tiles' products are being formed in the others.
__global__ void __launch_bounds__(kTcThreads, 1)
contract_tc_kernel(const __grid_constant__ CUtensorMap map_a_real, const __grid_constant__ CUtensorMap map_a_cplx,
                   const __grid_constant__ CUtensorMap map_xhi_real, const __grid_constant__ CUtensorMap map_xlo_real,
                   const __grid_constant__ CUtensorMap map_xhi_cplx, const __grid_constant__ CUtensorMap map_xlo_cplx,
                   TcArgs g) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], acc_full[kMaxAcc], acc_empty[kMaxAcc];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // stage ring, 1024-byte aligned (the swizzle pattern repeats every 1024 bytes); every stage has room
    // for the input tile and for all taps' weight tiles of the widest row tile
    const int bn_max = g.bn_real > g.bn_cplx ? g.bn_real : g.bn_cplx;
    const uint32_t xph_bytes = (uint32_t)g.xalloc * 128;                                  // one sub-tile (phase) of one part of the input tile
    const uint32_t x_bytes = (uint32_t)g.nph * xph_bytes + (uint32_t)g.xtail * 128;       // one part (hi or lo) of the input tile
    const uint32_t stage_bytes = (uint32_t)g.nsplit * (x_bytes + (uint32_t)g.taps * (uint32_t)bn_max * 128);
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    uint32_t acc_cols = 32;                      // columns of one accumulator
    while ((int)acc_cols < bn_max) acc_cols <<= 1;
    const uint32_t tmem_cols = (uint32_t)g.nacc * acc_cols;   // a power of two, <= 512 columns

    if (warp == 0 && lane == 0) {
        // start fetching the copy descriptors now; the first TMA would otherwise wait for them
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
        for (int b = 0; b < g.nacc; ++b) {
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
    pdl_wait();     // X is written by the transform kernel before this one; Y may still be read by an earlier one

    if (warp == 0) {
        // ---- TMA producer -----------------------------------------------------------------------
        if (lane == 0) {
            // ring position: stage s, and the parity of the current trip around the ring.  Counters
            // only -- no divisions on this thread's critical path.
            int s = 0, issued = 0;
            uint32_t par = 0;
            bool wrapped = false, ok = true;
            for (long tile = blockIdx.x; tile < g.tiles && ok; tile += gridDim.x) {
                const TileCoord t = decode_tile(g, tile);
                const CUtensorMap* map_a = t.real ? &map_a_real : &map_a_cplx;
                const CUtensorMap* map_xhi = t.real ? &map_xhi_real : &map_xhi_cplx;
                const CUtensorMap* map_xlo = t.real ? &map_xlo_real : &map_xlo_cplx;
                const uint32_t a_bytes = (uint32_t)t.bn * 128;           // one tap's weight tile
                const uint32_t tx_bytes = (uint32_t)g.nsplit * ((uint32_t)g.nph * (uint32_t)g.xrows * 128 + (uint32_t)g.taps * a_bytes);
                const int kblocks = (t.Kq + kKBlock - 1) / kKBlock;
                // one iteration = one K block: input tile (hi [, lo]) and all taps' weight tiles (hi [, lo])
                {
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (wrapped) ok = mbar_wait(&empty_bar[s], par ^ 1u, &abort_flag, g.spin_limit);
                        if (!ok) break;
                        unsigned char* xs = ring + (size_t)s * stage_bytes;
                        unsigned char* as = xs + (size_t)g.nsplit * x_bytes;
                        mbar_expect_tx(&full_bar[s], tx_bytes);
                        if (g.no_copy) {                 // fault injection: nothing is in flight, the consumer's wait runs out
                            ok = false;
                            issued = 0;
                            break;
                        }
                        // input tile with its halo: starts pad pixels before the output tile (negative and
                        // out-of-image coordinates read the zero fill)
                        for (int ph = 0; ph < g.nph; ++ph) {
                            const int pa = ph / g.sp, pb = ph - pa * g.sp;
                            const int w0 = g.stride * t.wo0 - g.pad + pb, h0 = g.stride * t.ho0 - g.pad + pa;
                            tma_load_5d(xs + ph * xph_bytes, map_xhi, &full_bar[s], kb * kKBlock, w0, h0, t.v, t.prob_in_kind);
                            if (g.nsplit == 2)
                                tma_load_5d(xs + x_bytes + ph * xph_bytes, map_xlo, &full_bar[s], kb * kKBlock, w0, h0, t.v, t.prob_in_kind);
                        }
                        // one box brings every tap's weight tile, hi parts first, then lo parts: [part][row][128 B]
                        tma_load_4d(as, map_a, &full_bar[s], kb * kKBlock, t.row0, 0, t.prob_in_kind);
                        if (issued < g.stages) ++issued;
                        if (++s == g.stages) {
                            s = 0;
                            par ^= 1u;
                            wrapped = true;
                        }
                    }
                }
            }
            if (!ok) {
                // drain: every copy that was issued must land before the CTA may go away.  The last
                // `issued` stages, walking backwards from the current ring position.
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
        {
            const uint32_t leader = elect_one();
            int s = 0;
            uint32_t par = 0;
            int buf = 0;
            uint32_t acc_par = 0;                 // parity of the accumulator pair's current use
            bool acc_wrapped = false, ok = true;
            for (long tile = blockIdx.x; tile < g.tiles && ok; tile += gridDim.x) {
                const TileCoord t = decode_tile(g, tile);
                const uint32_t a_bytes = (uint32_t)t.bn * 128;
                const uint32_t idesc = instr_desc(t.bn);
                const int kblocks = (t.Kq + kKBlock - 1) / kKBlock;
                if (acc_wrapped) ok = mbar_wait(&acc_empty[buf], acc_par ^ 1u, &abort_flag, g.spin_limit);   // epilogue done with it
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * acc_cols;
                uint32_t accumulate = 0;
                {
                    for (int kb = 0; kb < kblocks; ++kb) {
                        ok = mbar_wait(&full_bar[s], par, &abort_flag, g.spin_limit);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t xs = smem_u32(ring + (size_t)s * stage_bytes);
                        const uint32_t as = xs + (uint32_t)g.nsplit * x_bytes;
                        const uint32_t a_lo = as + (uint32_t)g.taps * a_bytes;   // lo parts of the weight tiles
                        const int krem = t.Kq - kb * kKBlock;                    // valid contraction entries in this block
                        if (leader) {
                        if (g.taps == 1 && krem >= kKBlock) {
                            // fully-connected fast path: four K steps of 16 per product
                            const uint64_t dxh = smem_desc_sw128(xs), dah = smem_desc_sw128(as);
                            tc_mma_bf16(d_tmem, dxh, dah, idesc, accumulate);
                            tc_mma_bf16(d_tmem, dxh + 2, dah + 2, idesc, 1u);
                            tc_mma_bf16(d_tmem, dxh + 4, dah + 4, idesc, 1u);
                            tc_mma_bf16(d_tmem, dxh + 6, dah + 6, idesc, 1u);
                            if (g.npass == 3) {
                                const uint64_t dxl = smem_desc_sw128(xs + x_bytes), dal = smem_desc_sw128(a_lo);
#pragma unroll
                                for (int k4 = 0; k4 < 4; ++k4) tc_mma_bf16(d_tmem, dxh + 2 * k4, dal + 2 * k4, idesc, 1u);
#pragma unroll
                                for (int k4 = 0; k4 < 4; ++k4) tc_mma_bf16(d_tmem, dxl + 2 * k4, dah + 2 * k4, idesc, 1u);
                            }
                            accumulate = 1u;
                        } else {
                            const int ksteps = krem >= kKBlock ? kKBlock / 16 : (krem + 15) / 16;   // the rest is zero fill
                            // descriptors differ only in their start-address field (16-byte units): build one per
                            // operand part and step it -- 8 units per tile row, a_bytes / 16 per tap, 2 per K step
                            const uint64_t dx_hi = smem_desc_sw128(xs), da_hi = smem_desc_sw128(as);
                            const uint64_t dx_lo = dx_hi + (uint64_t)(x_bytes >> 4);
                            const uint64_t da_lo = da_hi + (uint64_t)((uint32_t)g.taps * (a_bytes >> 4));
                            const uint64_t tap_step = (uint64_t)(a_bytes >> 4), row_step = (uint64_t)(g.pitch * 8);
                            for (int prod = 0; prod < g.npass; ++prod) {          // hi*hi, hi*lo(A), lo(X)*hi
                                const uint64_t dx = prod == 2 ? dx_lo : dx_hi;
                                const uint64_t da = prod == 1 ? da_lo : da_hi;
                                if (g.stride > 1) {
                                    // tap (di, dj) reads the sub-tile of phase (di % stride, dj % stride), shifted by the quotients
                                    uint64_t db = da;
                                    for (int di = 0; di < g.r; ++di) {
                                        const int pa = di % g.stride, qa = di / g.stride;
                                        for (int dj = 0; dj < g.r; ++dj, db += tap_step) {
                                            const int pb = dj % g.stride, qb = dj / g.stride;
                                            const uint64_t dxx = dx + (uint64_t)(pa * g.sp + pb) * (uint64_t)(xph_bytes >> 4) +
                                                                 (uint64_t)qa * row_step + (uint64_t)(qb * 8);
                                            tc_mma_bf16(d_tmem, dxx, db, idesc, accumulate);
                                            for (int k4 = 1; k4 < ksteps; ++k4)
                                                tc_mma_bf16(d_tmem, dxx + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), idesc, 1u);
                                            accumulate = 1u;
                                        }
                                    }
                                } else if (g.r == 3) {
                                    issue_taps_k<3>(ksteps, d_tmem, dx, da, row_step, tap_step, idesc, accumulate);
                                } else if (g.r == 1) {
                                    issue_taps_k<1>(ksteps, d_tmem, dx, da, row_step, tap_step, idesc, accumulate);
                                } else {
                                    uint64_t dx_row = dx, db = da;
                                    for (int di = 0; di < g.r; ++di, dx_row += row_step) {
                                        uint64_t dxx = dx_row;
                                        for (int dj = 0; dj < g.r; ++dj, dxx += 8, db += tap_step) {
                                            tc_mma_bf16(d_tmem, dxx, db, idesc, accumulate);
                                            for (int k4 = 1; k4 < ksteps; ++k4)   // 16 bf16 = 32 bytes per MMA step along K
                                                tc_mma_bf16(d_tmem, dxx + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), idesc, 1u);
                                            accumulate = 1u;
                                        }
                                    }
                                }
                            }
                        }
                        tc_commit(&empty_bar[s]);   // stage free once these MMAs have read it
                        if (kb + 1 == kblocks) tc_commit(&acc_full[buf]);   // accumulator complete
                        }
                        accumulate = 1u;
                        if (++s == g.stages) {
                            s = 0;
                            par ^= 1u;
                        }
                    }
                }
                if (++buf == g.nacc) {
                    buf = 0;
                    acc_par ^= 1u;
                    acc_wrapped = true;
                }
            }
        }
    } else {
        // ---- epilogue: TMEM -> registers -> shared memory -> Y[col][row] ----------------------------
        // A thread reads one TMEM lane = one column (pixel) of the tile, i.e. a run of rows that is
        // contiguous in Y, but the 32 lanes of a warp then hold 32 different memory lines.  The warp
        // therefore turns each 32 x 32 chunk around in shared memory and stores it with 8 lanes per
        // pixel (one 128-byte line per pixel, 512 contiguous bytes per instruction when the pixels
        // are neighbours), instead of 32 scattered 16-byte pieces per instruction.
        const int quarter = warp & 3;                 // a warp may only read its own 32 TMEM lanes
        float* stg = reinterpret_cast<float*>(ring + (size_t)g.stages * stage_bytes) + quarter * (32 * kStagePitch);
        const int sub = lane >> 3, seg = lane & 7;    // store phase: pixel sub + 4 * it of the warp, floats 4 seg .. 4 seg + 3
        // tile-independent position of the pixels this lane touches: row of the tile = flattened pixel
        // index at the input pitch
        uint32_t px_pos[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int rr = quarter * 32 + it * 4 + sub;
            const int h2 = rr / g.pitch;
            px_pos[it] = ((uint32_t)h2 << 16) | (uint32_t)(rr - h2 * g.pitch);
        }
        const int r = quarter * 32 + lane;            // the lane's own row (scalar path)
        const int hh = r / g.pitch, ww = r - hh * g.pitch;
        int buf = 0;
        uint32_t acc_par = 0;
        for (long tile = blockIdx.x; tile < g.tiles; tile += gridDim.x) {
            const TileCoord t = decode_tile(g, tile);
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[buf], acc_par, &abort_flag, g.spin_limit));  // warp-uniform
            if (!ok) break;
            tc_fence_after();
            const size_t y_real = (size_t)g.cols_out * g.p;
            float* ytile = g.yop + problem_offset(t.prob, y_real, 2 * y_real) + t.row0;
            const bool vec = (t.Mg & 3) == 0;         // rows come in whole float4 (row0, c0 and bn are multiples of 16)
            for (int c0 = 0; c0 < t.bn; c0 += 32) {
                uint32_t acc[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * acc_cols + (uint32_t)c0, acc);
                if (c0 + 32 >= t.bn) {
                    // last read of this accumulator: it may be overwritten by the tile after next
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[buf]);
                }
                // columns of this chunk that belong to the tile (its row tile may be narrower than 32
                // columns, and the last row tile may reach past the matrix)
                int nvalid = t.bn - c0;
                if (nvalid > t.Mg - t.row0 - c0) nvalid = t.Mg - t.row0 - c0;
                if (nvalid > 32) nvalid = 32;
                if (vec) {
                    float* mine = stg + lane * kStagePitch;
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        *reinterpret_cast<float4*>(mine + e) = make_float4(__uint_as_float(acc[e]), __uint_as_float(acc[e + 1]),
                                                                           __uint_as_float(acc[e + 2]), __uint_as_float(acc[e + 3]));
                    __syncwarp();
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int h2 = (int)(px_pos[it] >> 16), w2 = (int)(px_pos[it] & 0xffffu);
                        const int ho = t.ho0 + h2, wo = t.wo0 + w2;
                        if (h2 < g.th && w2 < g.tw && ho < g.Ho && wo < t.Wo && seg * 4 < nvalid) {
                            const float4 v = *reinterpret_cast<const float4*>(stg + (it * 4 + sub) * kStagePitch + seg * 4);
                            *reinterpret_cast<float4*>(ytile + ((size_t)((size_t)t.v * g.Ho + ho) * t.Wo + wo) * t.Mg + c0 + seg * 4) = v;
                        }
                    }
                    __syncwarp();
                } else {
                    const int ho = t.ho0 + hh, wo = t.wo0 + ww;
                    if (hh < g.th && ww < g.tw && ho < g.Ho && wo < t.Wo) {
                        float* yrow = ytile + ((size_t)((size_t)t.v * g.Ho + ho) * t.Wo + wo) * t.Mg;
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (e < nvalid) yrow[c0 + e] = __uint_as_float(acc[e]);
                    }
                }
            }
            if (++buf == g.nacc) {
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
static EncodeTiledFn encode_fn() { return tensor_map_encoder(); }
static int encode(CUtensorMap* map, void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes, const cuuint32_t* box,
                  const cuuint32_t* elem_strides = nullptr) {
    return encode_tensor_map(map, base, rank, dims, strides_bytes, box, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B,
                             elem_strides);
}

static int round_up16(int v) { return (v + 15) & ~15; }

// q a multiple of 4: the input transforms hand over four column blocks at a time; the operands' runs are padded to 8
bool tensor_supported(const Layer* L) { return (L->geo.q % 4) == 0 && encode_fn() != nullptr; }

// Ring depth, CTAs per SM and grid for a planned launch; maps = {A real, A complex, X hi real, X lo real, X hi complex, X lo complex}.
static int launch_planned(TcArgs& g, const CUtensorMap* maps, int nsplit, int taps, int kq_max, long ctas, cudaStream_t stream) {
    const int bn_max = g.bn_real > g.bn_cplx ? g.bn_real : g.bn_cplx;
    const size_t stage_bytes = (size_t)nsplit * (((size_t)g.nph * g.xalloc + g.xtail) * 128 + (size_t)taps * bn_max * 128);
    if (stage_bytes + 1024 > 199 * 1024) {
        set_error(CIRC_ERR_UNSUPPORTED, "filter taps x row tile do not fit one shared-memory stage (%zu bytes)", stage_bytes);
        return CIRC_ERR_UNSUPPORTED;
    }
    const int iters_max = (kq_max + kKBlock - 1) / kKBlock;
    g.stages = (int)((199 * 1024) / stage_bytes);
    if (g.stages > kMaxStages) g.stages = kMaxStages;
    if (g.stages > iters_max) g.stages = iters_max;
    // Persistent CTAs.  Short tiles (few ring iterations each) run two CTAs per SM, each with half of
    // the shared memory, so that one CTA's start-up and tail overlap the other's steady state; two
    // accumulators of bn_max columns per CTA keep both within the 512 columns of tensor memory.
    int ctas_per_sm = 1;
    {
        const int fit2 = (int)((93 * 1024) / stage_bytes);   // stages per CTA when two CTAs share an SM (ring + staging + reserve <= 114 KB each)
        if (ctas > 148 && iters_max <= 4 && bn_max <= 128 && fit2 >= 3) {
            ctas_per_sm = 2;                                  // only when each CTA still gets a ring of three or more
            if (g.stages > fit2) g.stages = fit2;
        }
        // the ring may run ahead into the next tile, so it is worth filling even when one tile needs fewer stages
        int deep = ctas_per_sm == 2 ? fit2 : (int)((198 * 1024) / stage_bytes);
        if (deep > kMaxStages) deep = kMaxStages;
        if (ctas > 148 * ctas_per_sm && deep > g.stages) g.stages = deep;
    }
    {
        // Accumulators: as many as tensor memory holds (512 columns per SM, shared by the CTAs on it).  With
        // small tiles the hand-over MMA -> epilogue -> MMA is a chain of barrier latencies; several
        // accumulators in flight take it off the critical path.
        int acc_cols = 32;
        while (acc_cols < bn_max) acc_cols <<= 1;
        g.nacc = (ctas_per_sm == 2 ? 256 : 512) / acc_cols;
        if (g.nacc > kMaxAcc) g.nacc = kMaxAcc;
    }
    const size_t smem = (size_t)g.stages * stage_bytes + 1024 + kStageOutBytes;
    static thread_local int configured_device = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        CIRC_CUDA_TRY(cudaFuncSetAttribute(contract_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024 + kStageOutBytes),
                      CIRC_ERR_CUDA);
        configured_device = dev;
    }
    if (ctas >= (1L << 31)) {
        set_error(CIRC_ERR_SHAPE, "too many output tiles (%ld)", ctas);
        return CIRC_ERR_SHAPE;
    }
    g.tiles = ctas;
    g.pdl_late = dependent_launches() == PDL_LATE;
    if (g.no_copy) g.spin_limit = 1u << 12;
    const unsigned grid = (unsigned)(ctas < 148 * ctas_per_sm ? ctas : 148 * ctas_per_sm);
    launch_kernel(dependent_launches(), contract_tc_kernel, dim3(grid), dim3(kTcThreads), smem, stream, maps[0], maps[1], maps[2], maps[3], maps[4],
                  maps[5], g);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int launch_contract_tc(const Layer* L, const __nv_bfloat16* xb, float* yop, const Extent& ext, int nsplit, cudaStream_t stream, bool twin) {
    const Geometry& geo = L->geo;
    const int p = geo.p, q = padded_q(geo.q), k = geo.k, taps = geo.taps;   // q: the (padded) run length of the operands
    TcArgs g;
    g.yop = yop;
    g.status = L->dev_status;
    g.p = p; g.q = q; g.k = k; g.taps = taps; g.r = geo.r; g.pad = geo.pad;
    g.nsplit = nsplit;
    g.npass = nsplit == 2 ? 3 : 1;
    g.spin_limit = kSpinLimit;
    g.no_copy = L->inject == INJECT_TENSOR_NO_COPY;
    if (L->kind == 1) {
        g.W = ext.W; g.H = ext.H; g.V = 2 * ext.Nh; g.Wo = ext.Wo; g.Ho = ext.Ho;
    } else {
        g.W = g.Wo = 2 * ext.Bh; g.H = g.Ho = 1; g.V = 1;
    }
    if (twin && L->kind != 0) {
        set_error(CIRC_ERR_UNSUPPORTED, "twin columns serve fully-connected layers only");
        return CIRC_ERR_UNSUPPORTED;
    }
    const __nv_bfloat16* a_op = twin ? L->a_twin : L->a_bf16;
    if (!a_op) {
        set_error(CIRC_ERR_ARG, "the stored form of the spectra for this contraction has not been built");
        return CIRC_ERR_ARG;
    }
    g.twin = twin ? 1 : 0;
    g.Wo_c = twin ? 2 * g.Wo : g.Wo;
    // strided convolution: tiles live in output-pixel space; each phase's sub-tile has (r - 1) / stride halo pixels
    g.stride = L->kind == 1 ? geo.stride : 1;
    g.sp = g.stride < geo.r ? g.stride : geo.r;
    g.nph = g.sp * g.sp;
    const int halo = (geo.r - 1) / g.stride;
    int tw_cap = kTileCols - halo;
    if (256 / g.stride - halo < tw_cap) tw_cap = 256 / g.stride - halo;   // a strided box spans pitch x stride pixels, at most 256
    for (;;) {
        g.tw = g.Wo_c < tw_cap ? g.Wo_c : tw_cap;   // the wider problem kind sets the tile
        g.pitch = g.tw + halo;
        g.th = (kTileCols - g.tw) / g.pitch + 1;          // (th - 1) * pitch + tw <= 128 MMA rows
        if (g.th > g.Ho) g.th = g.Ho;
        g.xrows = g.pitch * (g.th + halo);
        // a tap's view starts up to halo rows and halo pixels into its sub-tile and spans 128 pixel slots: views that
        // run past their sub-tile read the next one (or the tail) into output slots that are never stored
        const int reach = halo * g.pitch + halo + kTileCols;   // last row any tap's 128-row view touches, plus one
        g.xalloc = (g.xrows + 7) & ~7;                         // whole 1024-byte swizzle groups
        g.xtail = reach > g.xalloc ? ((reach - g.xalloc + 7) & ~7) : 0;
        // several sub-tiles (a strided convolution) of a wide, flat tile can outgrow a stage: narrower tiles are
        // taller, and the halo rows weigh less
        const long x_b = (long)nsplit * ((long)g.nph * g.xalloc + g.xtail) * 128;
        if (g.nph == 1 || x_b + (long)nsplit * taps * 16 * 128 <= 160 * 1024 || tw_cap <= 8) break;
        tw_cap /= 2;
    }
    g.tiles_w = (g.Wo + g.tw - 1) / g.tw;
    g.tiles_w_c = (g.Wo_c + g.tw - 1) / g.tw;
    g.tiles_h = (g.Ho + g.th - 1) / g.th;
    const int rows_c = twin ? p : 2 * p;                // rows of a complex problem
    g.bn_real = round_up16(p) > 256 ? 256 : round_up16(p);
    g.bn_cplx = round_up16(rows_c) > 256 ? 256 : round_up16(rows_c);
    {
        // all taps' weight tiles of one K block share a stage with the input tile: narrow the row
        // tile until a stage fits half of the shared memory (two stages), or all of it at worst
        const long x_b = (long)nsplit * ((long)g.nph * g.xalloc + g.xtail) * 128;
        long room = 96 * 1024 - x_b;
        if (room < (long)nsplit * taps * 16 * 128) room = 198 * 1024 - x_b;
        int cap = (int)(room / ((long)nsplit * taps * 128)) & ~15;
        if (cap < 16) cap = 16;
        if (g.bn_real > cap) g.bn_real = cap;
        if (g.bn_cplx > cap) g.bn_cplx = cap;
    }
    g.cols_out = (long)g.V * g.Ho * g.Wo;
    const int sp_tiles = g.V * g.tiles_h * g.tiles_w, sp_tiles_c = g.V * g.tiles_h * g.tiles_w_c;
    long ctas = 0;
    for (;;) {
        g.nt_real = (p + g.bn_real - 1) / g.bn_real;
        g.nt_cplx = (rows_c + g.bn_cplx - 1) / g.bn_cplx;
        g.ctas_real = 2 * g.nt_real * sp_tiles;
        ctas = (long)g.ctas_real + (long)(k / 2 - 1) * g.nt_cplx * sp_tiles_c;
        // a grid that leaves most of the 148 SMs idle is split into narrower row tiles
        // ... and so is a grid of fewer than 200 long float32 tiles (16 K blocks or more): with at most one tile per thread
        // block the longest tile sets the time; half-height tiles take 0.67 of it and most thread blocks then take a short
        // real tile on top (4096 x 4096, k = 4, batch 1024: 57.4 -> 49.4 us; short tiles, where latency rules, lose by it)
        const bool long_tiles = nsplit == 2 && (2 * q + kKBlock - 1) / kKBlock >= 16 && g.bn_cplx > 128;
        if (ctas >= (long_tiles ? 200 : 100) || g.bn_cplx <= 32) break;
        g.bn_cplx = round_up16(g.bn_cplx / 2);
        if (g.bn_real > 32) g.bn_real = round_up16(g.bn_real / 2);
    }

    // tensor maps.  A: [problem][row][hi|lo][tap][Kq]; one box = (K block, bn rows, all taps of the parts in use)
    CUtensorMap ma_r, ma_c, mxh_r, mxl_r, mxh_c, mxl_c;
    const size_t a_real_elems = (size_t)p * taps * 2 * q;  // one real problem of A (hi and lo)
    const cuuint32_t a_parts = (cuuint32_t)(nsplit * taps);
    int rc;
    {
        cuuint64_t dims[4] = {(cuuint64_t)q, (cuuint64_t)p, (cuuint64_t)taps * 2, 2};
        cuuint64_t str[3] = {(cuuint64_t)taps * 2 * q * 2, (cuuint64_t)q * 2, (cuuint64_t)a_real_elems * 2};
        cuuint32_t box[4] = {kKBlock, (cuuint32_t)g.bn_real, a_parts, 1};
        if ((rc = encode(&ma_r, const_cast<__nv_bfloat16*>(a_op), 4, dims, str, box)) != CIRC_OK) return rc;
    }
    {
        const int nc = k / 2 - 1 > 0 ? k / 2 - 1 : 1;
        // embedded: 2p rows per problem; twin: p rows of (Wr, Wi) pairs
        cuuint64_t dims[4] = {(cuuint64_t)2 * q, (cuuint64_t)rows_c, (cuuint64_t)taps * 2, (cuuint64_t)nc};
        cuuint64_t str[3] = {(cuuint64_t)taps * 2 * 2 * q * 2, (cuuint64_t)2 * q * 2, (cuuint64_t)(twin ? 2 : 4) * a_real_elems * 2};
        cuuint32_t box[4] = {kKBlock, (cuuint32_t)g.bn_cplx, a_parts, 1};
        if ((rc = encode(&ma_c, const_cast<__nv_bfloat16*>(a_op) + 2 * a_real_elems, 4, dims, str, box)) != CIRC_OK) return rc;
    }
    // X: [problem][v][h][w][part][Kq]; a strided convolution fetches every stride-th pixel of a phase (a box extent of
    // N x stride brings N pixels)
    const cuuint32_t xstr[5] = {1, (cuuint32_t)g.stride, (cuuint32_t)g.stride, 1, 1};
    const size_t cols_in = (size_t)g.V * g.H * g.W;
    const size_t x_real_elems = cols_in * nsplit * q;
    {
        cuuint64_t dims[5] = {(cuuint64_t)q, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.V, 2};
        cuuint64_t str[4] = {(cuuint64_t)nsplit * q * 2, (cuuint64_t)g.W * nsplit * q * 2,
                             (cuuint64_t)g.H * g.W * nsplit * q * 2, (cuuint64_t)x_real_elems * 2};
        cuuint32_t box[5] = {kKBlock, (cuuint32_t)(g.pitch * g.stride), (cuuint32_t)((g.th + halo) * g.stride), 1, 1};
        __nv_bfloat16* base = const_cast<__nv_bfloat16*>(xb);
        if ((rc = encode(&mxh_r, base, 5, dims, str, box, xstr)) != CIRC_OK) return rc;
        if ((rc = encode(&mxl_r, base + (nsplit == 2 ? q : 0), 5, dims, str, box, xstr)) != CIRC_OK) return rc;
    }
    {
        const int nc = k / 2 - 1 > 0 ? k / 2 - 1 : 1;
        const cuuint64_t wc = (cuuint64_t)(twin ? 2 * g.W : g.W);      // twin: (Zr, -Zi) columns, then (Zi, Zr) columns
        cuuint64_t dims[5] = {(cuuint64_t)2 * q, wc, (cuuint64_t)g.H, (cuuint64_t)g.V, (cuuint64_t)nc};
        cuuint64_t str[4] = {(cuuint64_t)nsplit * 2 * q * 2, wc * nsplit * 2 * q * 2,
                             (cuuint64_t)g.H * wc * nsplit * 2 * q * 2, (cuuint64_t)(twin ? 4 : 2) * x_real_elems * 2};
        cuuint32_t box[5] = {kKBlock, (cuuint32_t)(g.pitch * g.stride), (cuuint32_t)((g.th + halo) * g.stride), 1, 1};
        __nv_bfloat16* base = const_cast<__nv_bfloat16*>(xb) + 2 * x_real_elems;
        if ((rc = encode(&mxh_c, base, 5, dims, str, box, xstr)) != CIRC_OK) return rc;
        if ((rc = encode(&mxl_c, base + (nsplit == 2 ? 2 * q : 0), 5, dims, str, box, xstr)) != CIRC_OK) return rc;
    }

    const CUtensorMap maps[6] = {ma_r, ma_c, mxh_r, mxl_r, mxh_c, mxl_c};
    return launch_planned(g, maps, nsplit, taps, 2 * q, ctas, stream);
}


// One kind (real or complex problems) of a generic per-problem product  Y[prob][xrow][arow] = sum_c X[prob][xrow][c] * A[prob][arow][c]
// with both operands stored as split bfloat16 [prob][row][hi | lo][cols_padded].  The backward pass uses it for the
// batch sum of the weight gradient, where the contraction index is the batch column.
static int launch_tc_one_kind(bool real, const __nv_bfloat16* xt, int x_rows, const __nv_bfloat16* at, int a_rows, int cols,
                              int cols_padded, int nprob, float* y, int* status, cudaStream_t stream) {
    if (nprob <= 0) return CIRC_OK;
    TcArgs g;
    g.status = status;
    g.taps = 1; g.r = 1; g.pad = 0;
    g.nsplit = 2;
    g.npass = 3;
    g.spin_limit = kSpinLimit;
    g.no_copy = 0;
    g.stride = 1;
    g.sp = 1;
    g.nph = 1;
    g.W = g.Wo = x_rows; g.H = g.Ho = 1; g.V = 1;
    g.tw = x_rows < kTileCols ? x_rows : kTileCols;
    g.pitch = g.tw;
    g.th = 1;
    g.xrows = g.tw;
    g.xalloc = kTileCols;
    g.xtail = 0;
    g.tiles_w = g.tiles_w_c = (x_rows + g.tw - 1) / g.tw;
    g.tiles_h = 1;
    g.twin = 0;
    g.Wo_c = x_rows;
    g.cols_out = x_rows;
    int bn = round_up16(a_rows) > 256 ? 256 : round_up16(a_rows);
    const int nt = (a_rows + bn - 1) / bn;
    g.bn_real = g.bn_cplx = bn;
    const int sp_tiles = g.tiles_w;
    long ctas;
    if (real) {                      // the kernel's real group always has two problems
        g.p = a_rows; g.q = cols; g.k = 2;
        g.nt_real = nt; g.nt_cplx = 1;
        g.ctas_real = 2 * nt * sp_tiles;
        ctas = g.ctas_real;
        g.yop = y;
    } else {
        g.p = a_rows / 2; g.q = cols / 2; g.k = 2 * (nprob + 1);
        g.nt_real = 0; g.nt_cplx = nt;
        g.ctas_real = 0;
        ctas = (long)nprob * nt * sp_tiles;
        g.yop = y - 2 * (size_t)x_rows * (a_rows / 2);   // the kernel skips two real-sized problems before the complex ones
    }
    CUtensorMap ma, mxh, mxl;
    int rc;
    {
        cuuint64_t dims[4] = {(cuuint64_t)cols, (cuuint64_t)a_rows, 2, (cuuint64_t)nprob};
        cuuint64_t str[3] = {(cuuint64_t)2 * cols_padded * 2, (cuuint64_t)cols_padded * 2, (cuuint64_t)a_rows * 2 * cols_padded * 2};
        cuuint32_t box[4] = {kKBlock, (cuuint32_t)bn, 2, 1};
        if ((rc = encode(&ma, const_cast<__nv_bfloat16*>(at), 4, dims, str, box)) != CIRC_OK) return rc;
    }
    {
        const cuuint64_t row = (cuuint64_t)2 * cols_padded * 2, img = (cuuint64_t)x_rows * row;
        cuuint64_t dims[5] = {(cuuint64_t)cols, (cuuint64_t)x_rows, 1, 1, (cuuint64_t)nprob};
        cuuint64_t str[4] = {row, img, img, img};
        cuuint32_t box[5] = {kKBlock, (cuuint32_t)g.pitch, 1, 1, 1};
        __nv_bfloat16* base = const_cast<__nv_bfloat16*>(xt);
        if ((rc = encode(&mxh, base, 5, dims, str, box)) != CIRC_OK) return rc;
        if ((rc = encode(&mxl, base + cols_padded, 5, dims, str, box)) != CIRC_OK) return rc;
    }
    const CUtensorMap maps[6] = {ma, ma, mxh, mxl, mxh, mxl};
    return launch_planned(g, maps, 2, 1, cols, ctas, stream);
}

bool tensor_batch_product_supported(int cols) { return cols >= 8 && (cols % 2) == 0 && encode_fn() != nullptr; }

int launch_tc_batch_product(const __nv_bfloat16* xt, int q, const __nv_bfloat16* at, int p, int k, int cols, int cols_padded,
                            float* y_real, float* y_cplx, int* status, cudaStream_t stream) {
    const size_t x_real = (size_t)q * 2 * cols_padded, a_real = (size_t)p * 2 * cols_padded;   // elements of one real problem
    int rc = launch_tc_one_kind(true, xt, q, at, p, cols, cols_padded, 2, y_real, status, stream);
    if (rc != CIRC_OK) return rc;
    return launch_tc_one_kind(false, xt + 2 * x_real, 2 * q, at + 2 * a_real, 2 * p, cols, cols_padded, k / 2 - 1, y_cplx, status,
                              stream);
}

}  // namespace circ
