// S1 / C1 (input transforms) and S3 / C3 (inverse transforms + bias + activation) of the
// staged path.  Both kernels hold whole transforms in registers (circ_fft.cuh) and use shared
// memory only to turn the "one transform = contiguous k samples" view of x and y into the
// "one frequency = one matrix" view the per-frequency contraction needs (circ_common.cuh).
//
// The staging tile is bin-major: zs[bin][transform].  The side that holds transforms in
// registers touches (bin f2 + L*f1, transform gi); the side that talks to the operand in global
// memory walks along a row (consecutive transforms of one bin), which is also the direction in
// which the operand is contiguous, so those global accesses are full coalesced runs.
#include <type_traits>
#include <utility>
#include <vector>

#include "circ_common.cuh"
#include "circ_fft.cuh"
#include "circ_io.cuh"

namespace circ {


// Row length of the tile: TT transforms plus a pad that makes the register side conflict-free.
// A half warp there is (16 / L) consecutive transforms x L bins, so rows must be 16 / L float2
// apart modulo the 16 eight-byte banks.
template <int K, int EMAX>
struct Tile {
    static constexpr int L = FftShape<K, EMAX>::L;
    static constexpr int NT = K >= 1024 ? 128 : (K >= 128 && EMAX == 16) ? 256 : 128;   // threads per CTA: small CTAs fill the SMs more evenly
    static constexpr int TT = NT / L;
    static constexpr int PAD = L == 1 ? 0 : (L >= 16 ? 2 : 16 / L);  // even, so that rows stay 16-byte aligned
    static constexpr int ROW = TT + PAD;
    static constexpr size_t SMEM = sizeof(float2) * ((size_t)K + (size_t)K * ROW) + (size_t)TT * 16;   // twiddle table + staging tile + per-transform output offsets (dynamic shared memory)
};

// Position of a transform: T = c * rows + i (c: sample pair, i: block).  A CTA's transforms are consecutive, so the
// one 64-bit division is done for the CTA's first transform and the others follow by small-integer arithmetic
// (the kernels are bound by instruction issue; a 64-bit division per work item was a third of their instructions).
struct Split {
    int c0, i0;
};
__device__ __forceinline__ Split split_base(long base, int rows) {
    const long c = base / rows;
    return Split{(int)c, (int)(base - c * rows)};
}
template <int TT>
__device__ __forceinline__ void split_at(Split s, int d, int rows, int& c, int& i) {
    i = s.i0 + d;
    c = s.c0;
    if (i >= rows) {
        if (rows >= TT) {          // at most one wrap
            i -= rows;
            ++c;
        } else {                   // few rows: small 32-bit division
            const int a = i / rows;
            i -= a * rows;
            c += a;
        }
    }
}

// Operand Y -> tile (the first half of S3): fills zs[bin][transform] for the CTA's TT transforms.
// TWIN: Y of a complex problem holds the real parts of all 2 Bho columns, then the imaginary parts (p rows each),
// instead of 2p interleaved rows.
// Y may come as several copies, `copy_stride` floats apart (copies_r of every real problem, copies_c of every complex
// one), that are added here in a fixed order (the row-streaming contraction cuts its contraction range into pieces).
__device__ __forceinline__ float4 add4(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }
template <int K, int EMAX, bool VEC, bool TWIN = false>
__device__ __forceinline__ void gather_operand(float2 (*zs)[Tile<K, EMAX>::ROW], const float* __restrict__ yop, int p, int Bho,
                                               long total, Split sp, int copies_r = 1, int copies_c = 1, size_t copy_stride = 0) {
    constexpr int TT = Tile<K, EMAX>::TT, kThreads = Tile<K, EMAX>::NT;
    const size_t cols = 2 * (size_t)Bho;
    const size_t real_sz = cols * p, cplx_sz = 2 * real_sz;
    if constexpr (VEC) {
        // all loads of the tile are issued before the first one is used
        constexpr int GROUPS = TT / 4;
        constexpr int ITERS = GROUPS * K / kThreads;
        static_assert(GROUPS * K % kThreads == 0, "tile must divide evenly among the threads");
        float4 r0[ITERS], r1[ITERS];
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int item = threadIdx.x + it * kThreads;
            const int grp = item % GROUPS, f = item / GROUPS;
            const long T0 = (long)blockIdx.x * TT + grp * 4;
            r0[it] = r1[it] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (T0 >= total) continue;
            int c, i;
            split_at<TT>(sp, grp * 4, p, c, i);
            if (f == 0 || f == K / 2) {
                const float* yg = yop + problem_offset(f == 0 ? 0 : 1, real_sz, cplx_sz);
                for (int s = 0; s < copies_r; ++s, yg += copy_stride) {
                    r0[it] = add4(r0[it], __ldg(reinterpret_cast<const float4*>(yg + (size_t)c * p + i)));
                    r1[it] = add4(r1[it], __ldg(reinterpret_cast<const float4*>(yg + ((size_t)Bho + c) * p + i)));
                }
            } else {
                const bool mirror = f > K / 2;
                const int g = mirror ? K - f : f;
                if constexpr (TWIN) {
                    const float* r = yop + problem_offset(g + 1, real_sz, cplx_sz) + ((size_t)(mirror ? Bho : 0) + c) * p + i;
                    for (int s = 0; s < copies_c; ++s, r += copy_stride) {
                        r0[it] = add4(r0[it], __ldg(reinterpret_cast<const float4*>(r)));                        // four real parts
                        r1[it] = add4(r1[it], __ldg(reinterpret_cast<const float4*>(r + (size_t)2 * Bho * p)));  // their imaginary parts
                    }
                } else {
                    const float* r = yop + problem_offset(g + 1, real_sz, cplx_sz) + ((size_t)(mirror ? Bho : 0) + c) * 2 * p + 2 * i;
                    for (int s = 0; s < copies_c; ++s, r += copy_stride) {
                        r0[it] = add4(r0[it], __ldg(reinterpret_cast<const float4*>(r)));
                        r1[it] = add4(r1[it], __ldg(reinterpret_cast<const float4*>(r) + 1));
                    }
                }
            }
        }
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int item = threadIdx.x + it * kThreads;
            const int grp = item % GROUPS, f = item / GROUPS;
            float4 za, zb;
            if (f == 0 || f == K / 2) {
                za = make_float4(r0[it].x, r1[it].x, r0[it].y, r1[it].y);
                zb = make_float4(r0[it].z, r1[it].z, r0[it].w, r1[it].w);
            } else if constexpr (TWIN) {
                const float sgn = f > K / 2 ? -1.f : 1.f;
                za = make_float4(r0[it].x, sgn * r1[it].x, r0[it].y, sgn * r1[it].y);
                zb = make_float4(r0[it].z, sgn * r1[it].z, r0[it].w, sgn * r1[it].w);
            } else {
                const float sgn = f > K / 2 ? -1.f : 1.f;
                za = r0[it];
                zb = r1[it];
                za.y *= sgn; za.w *= sgn; zb.y *= sgn; zb.w *= sgn;
            }
            *reinterpret_cast<float4*>(&zs[f][grp * 4]) = za;
            *reinterpret_cast<float4*>(&zs[f][grp * 4 + 2]) = zb;
        }
    } else {
        for (int item = threadIdx.x; item < TT * K; item += kThreads) {
            const int tl = item % TT, f = item / TT;
            const long T2 = (long)blockIdx.x * TT + tl;
            if (T2 >= total) continue;
            int c, i;
            split_at<TT>(sp, tl, p, c, i);
            float2 z = make_float2(0.f, 0.f);
            if (f == 0 || f == K / 2) {
                const float* yg = yop + problem_offset(f == 0 ? 0 : 1, real_sz, cplx_sz);
                for (int s = 0; s < copies_r; ++s, yg += copy_stride) {
                    z.x += __ldg(yg + (size_t)c * p + i);
                    z.y += __ldg(yg + ((size_t)Bho + c) * p + i);
                }
            } else if constexpr (TWIN) {
                const bool mirror = f > K / 2;
                const float* yg = yop + problem_offset((mirror ? K - f : f) + 1, real_sz, cplx_sz) + ((size_t)(mirror ? Bho : 0) + c) * p + i;
                for (int s = 0; s < copies_c; ++s, yg += copy_stride) {
                    z.x += __ldg(yg);
                    z.y += __ldg(yg + (size_t)2 * Bho * p);
                }
                if (mirror) z.y = -z.y;
            } else {
                const bool mirror = f > K / 2;
                const float* yg = yop + problem_offset((mirror ? K - f : f) + 1, real_sz, cplx_sz) + ((size_t)(mirror ? Bho : 0) + c) * 2 * p + 2 * i;
                for (int s = 0; s < copies_c; ++s, yg += copy_stride) {
                    const float2 t = __ldg(reinterpret_cast<const float2*>(yg));
                    z.x += t.x;
                    z.y += t.y;
                }
                if (mirror) z.y = -z.y;
            }
            zs[f][tl] = z;
        }
    }
}

// Tile -> operand X (the second half of S1): zs[bin][transform] holds the spectra of the CTA's TT transforms.
// TWIN (bfloat16 modes): a complex problem gets two column groups, (Zr, -Zi) for the 2 Bh columns and then (Zi, Zr)
// for them again; multiplied by weights stored once as (Wr, Wi) pairs they give the real and the imaginary parts.
template <int K, int EMAX, int XMODE, bool TWIN = false>
__device__ __forceinline__ void scatter_operand(const float2 (*zs)[Tile<K, EMAX>::ROW], void* __restrict__ xop, int q, int Bh,
                                                long total, Split sp) {
    constexpr int TT = Tile<K, EMAX>::TT, kThreads = Tile<K, EMAX>::NT;
    const size_t cols = 2 * (size_t)Bh;
    constexpr int NPART = XMODE == 1 ? 2 : 1;
    const size_t real_sz = cols * q * NPART, cplx_sz = (TWIN ? 4 : 2) * real_sz;

    if constexpr (XMODE == 0) {
        // scalar scatter (any q): one work item = (bin, transform), consecutive threads = consecutive transforms
        float* xf = static_cast<float*>(xop);
        for (int item = threadIdx.x; item < TT * K; item += kThreads) {
            const int tl = item % TT, f = item / TT;
            const long T2 = (long)blockIdx.x * TT + tl;
            if (T2 >= total) continue;
            int c, j;
            split_at<TT>(sp, tl, q, c, j);
            const float2 z = zs[f][tl];
            if (f == 0 || f == K / 2) {
                float* xg = xf + problem_offset(f == 0 ? 0 : 1, real_sz, cplx_sz);
                xg[(size_t)c * q + j] = z.x;
                xg[((size_t)Bh + c) * q + j] = z.y;
            } else if (f < K / 2) {
                float* xg = xf + problem_offset(f + 1, real_sz, cplx_sz) + (size_t)c * 2 * q + 2 * j;
                *reinterpret_cast<float2*>(xg) = z;
            } else {
                float* xg = xf + problem_offset(K - f + 1, real_sz, cplx_sz) + ((size_t)Bh + c) * 2 * q + 2 * j;
                *reinterpret_cast<float2*>(xg) = make_float2(z.x, -z.y);
            }
        }
    } else {
        // vector scatter: one work item = (bin, 4 consecutive transforms) = 16 bytes of (Re, Im) bfloat16
        // pairs per part; consecutive lanes = consecutive groups = consecutive memory.
        // (q is a multiple of 4; runs are padded_q(q) entries long and the group that ends a run also zeroes its padding)
        __nv_bfloat16* xb = static_cast<__nv_bfloat16*>(xop);
        constexpr int GROUPS = TT / 4;
        const int qs = padded_q(q);
        const size_t real_sz = cols * qs * NPART, cplx_sz = (TWIN ? 4 : 2) * real_sz;
        const uint2 zero2 = make_uint2(0u, 0u);
        const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
        for (int item = threadIdx.x; item < GROUPS * K; item += kThreads) {
            const int grp = item % GROUPS, f = item / GROUPS;
            const long T0 = (long)blockIdx.x * TT + grp * 4;
            if (T0 >= total) continue;                 // total is a multiple of 4
            int c, j;
            split_at<TT>(sp, grp * 4, q, c, j);
            const bool pad = qs != q && j + 4 == q;    // this group ends its column's run
            const float4 za = *reinterpret_cast<const float4*>(&zs[f][grp * 4]);
            const float4 zb = *reinterpret_cast<const float4*>(&zs[f][grp * 4 + 2]);
            if (f == 0 || f == K / 2) {
                __nv_bfloat16* xg = xb + problem_offset(f == 0 ? 0 : 1, real_sz, cplx_sz);
                __nv_bfloat16* d0 = xg + (size_t)c * (NPART * qs) + j;
                __nv_bfloat16* d1 = xg + ((size_t)Bh + c) * (NPART * qs) + j;
                uint32_t l0, l1, l2, l3;
                const uint32_t h0 = bf16_split_pair(za.x, za.z, l0), h1 = bf16_split_pair(zb.x, zb.z, l1);
                const uint32_t h2 = bf16_split_pair(za.y, za.w, l2), h3 = bf16_split_pair(zb.y, zb.w, l3);
                *reinterpret_cast<uint2*>(d0) = make_uint2(h0, h1);
                *reinterpret_cast<uint2*>(d1) = make_uint2(h2, h3);
                if constexpr (XMODE == 1) {
                    *reinterpret_cast<uint2*>(d0 + qs) = make_uint2(l0, l1);
                    *reinterpret_cast<uint2*>(d1 + qs) = make_uint2(l2, l3);
                }
                if (pad) {
                    *reinterpret_cast<uint2*>(d0 + 4) = zero2;
                    *reinterpret_cast<uint2*>(d1 + 4) = zero2;
                    if constexpr (XMODE == 1) {
                        *reinterpret_cast<uint2*>(d0 + qs + 4) = zero2;
                        *reinterpret_cast<uint2*>(d1 + qs + 4) = zero2;
                    }
                }
            } else {
                const bool mirror = f > K / 2;
                const int g = mirror ? K - f : f;
                const float sgn = mirror ? -1.f : 1.f;
                __nv_bfloat16* d = xb + problem_offset(g + 1, real_sz, cplx_sz) +
                                   ((size_t)(mirror ? Bh : 0) + c) * (NPART * 2 * qs) + 2 * j;
                const float i0 = sgn * za.y, i1 = sgn * za.w, i2 = sgn * zb.y, i3 = sgn * zb.w;
                uint32_t l0, l1, l2, l3;
                const uint32_t h0 = bf16_split_pair(za.x, i0, l0), h1 = bf16_split_pair(za.z, i1, l1);
                const uint32_t h2 = bf16_split_pair(zb.x, i2, l2), h3 = bf16_split_pair(zb.z, i3, l3);
                if constexpr (TWIN) {
                    // a word holds (re | im << 16): negating im flips its sign bit, swapping re and im swaps the halves
                    constexpr uint32_t S = 0x80000000u;
                    auto swp = [](uint32_t v) { return __byte_perm(v, 0u, 0x1032); };
                    __nv_bfloat16* d2 = d + cols * (size_t)(NPART * 2 * qs);
                    *reinterpret_cast<uint4*>(d) = make_uint4(h0 ^ S, h1 ^ S, h2 ^ S, h3 ^ S);
                    *reinterpret_cast<uint4*>(d2) = make_uint4(swp(h0), swp(h1), swp(h2), swp(h3));
                    if constexpr (XMODE == 1) {
                        *reinterpret_cast<uint4*>(d + 2 * qs) = make_uint4(l0 ^ S, l1 ^ S, l2 ^ S, l3 ^ S);
                        *reinterpret_cast<uint4*>(d2 + 2 * qs) = make_uint4(swp(l0), swp(l1), swp(l2), swp(l3));
                    }
                } else {
                    *reinterpret_cast<uint4*>(d) = make_uint4(h0, h1, h2, h3);
                    if constexpr (XMODE == 1) *reinterpret_cast<uint4*>(d + 2 * qs) = make_uint4(l0, l1, l2, l3);
                    if (pad) {                         // (twin columns are only used when there is no padding)
                        *reinterpret_cast<uint4*>(d + 8) = zero4;
                        if constexpr (XMODE == 1) *reinterpret_cast<uint4*>(d + 2 * qs + 8) = zero4;
                    }
                }
            }
        }
    }
}

// ---- S1: x -> operand X ------------------------------------------------------------------------
// One transform = (pair c, column block j).  A CTA takes TT = 256 / L consecutive transforms.
// XMODE 0: float32 operand [problem][col][Kq]                      (FMA contraction, any q)
// XMODE 1: bfloat16 operand [problem][col][hi | lo][Kq]            (tensor cores, float32 input split in two)
// XMODE 2: bfloat16 operand [problem][col][Kq]                     (tensor cores, bfloat16 input)
// Complex problems interleave (Re, Im): contraction index 2j, 2j+1.  XMODE 1 / 2 need q % 8 == 0.
template <int K, int EMAX, typename TIN, int XMODE, bool TWIN = false>
__global__ void __launch_bounds__(Tile<K, EMAX>::NT)
input_fft_kernel(const TIN* __restrict__ x, void* __restrict__ xop, int n, int q,
                 int B, int Bh, long total, int ku, int pdl_late) {
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L, TT = Tile<K, EMAX>::TT, ROW = Tile<K, EMAX>::ROW;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2* tw = reinterpret_cast<float2*>(smem_raw);
    float2 (*zs)[ROW] = reinterpret_cast<float2 (*)[ROW]>(tw + K);
    load_twiddles<K>(tw);
    if (!pdl_late) pdl_trigger();
    pdl_wait();     // x may come from the kernel before; the operand buffer may still be read by it

    const int gi = threadIdx.x / L, l = threadIdx.x % L;
    const long T = (long)blockIdx.x * TT + gi;
    const Split sp = split_base((long)blockIdx.x * TT, q);
    float2 v[E];
    {
        float re[E], im[E];
#pragma unroll
        for (int r = 0; r < E; ++r) re[r] = im[r] = 0.f;
        if (T < total) {
            int c, j;
            split_at<TT>(sp, gi, q, c, j);
            if (ku == K) {
                load_run<E>(x + (size_t)c * n + (size_t)j * K + E * l, re);
                if (c + Bh < B) load_run<E>(x + (size_t)(c + Bh) * n + (size_t)j * K + E * l, im);
            } else {
                // embedded block size: the block has ku samples (any alignment), the rest of the transform is zero
                const TIN* x0 = x + (size_t)c * n + (size_t)j * ku;
                const TIN* x1 = x + (size_t)(c + Bh) * n + (size_t)j * ku;
                const bool second = c + Bh < B;
                if ((ku & 3) == 0) {
                    // rows and blocks start on multiples of four elements: whole groups of four are inside or outside
#pragma unroll
                    for (int g4 = 0; g4 < E; g4 += 4) {
                        const int t = E * l + g4;
                        if (t < ku) {
                            float t0[4], t1[4] = {0.f, 0.f, 0.f, 0.f};
                            load_run<4>(x0 + t, t0);
                            if (second) load_run<4>(x1 + t, t1);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                re[g4 + e] = t0[e];
                                im[g4 + e] = t1[e];
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int r = 0; r < E; ++r) {
                        const int t = E * l + r;
                        if (t < ku) {
                            re[r] = to_float(x0[t]);
                            if (second) im[r] = to_float(x1[t]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < E; ++r) v[r] = make_float2(re[r], im[r]);
    }
    __syncthreads();  // twiddles ready
    fft_forward<K, EMAX>(v, l, tw);
    const int f2 = lane_residue<K, EMAX>(l);
#pragma unroll
    for (int f1 = 0; f1 < E; ++f1) zs[f2 + L * f1][gi] = v[f1];
    __syncthreads();

    if (pdl_late) pdl_trigger();
    scatter_operand<K, EMAX, XMODE, TWIN>(zs, xop, q, Bh, total, sp);
}

// Bias, activation and stores of one inverse-transformed tile (block size = transform size).  `tile` is the staging
// tile the bins came from (reused for the hand-over), `offs` / `both` are TT entries of scratch behind it.
template <int K, int EMAX, typename TOUT>
__device__ __forceinline__ void store_outputs(const float2 (&v)[FftShape<K, EMAX>::E], const float (&bv)[FftShape<K, EMAX>::E],
                                              float2 (*zs)[Tile<K, EMAX>::ROW], long long* offs, int* both, int gi, int l, bool live,
                                              int c, int i, TOUT* __restrict__ y, int relu, int m, int Bo, int Bho) {
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L, TT = Tile<K, EMAX>::TT;
    if constexpr (E < 16 || !std::is_same<TOUT, float>::value) {
        // a lane's outputs are at most 32 bytes: direct stores are already (nearly) whole lines per instruction
        if (!live) return;
        const int col = i * K + E * l;
        float re[E], im[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            re[r] = v[r].x + bv[r];
            im[r] = v[r].y + bv[r];
            if (relu) {
                re[r] = fmaxf(re[r], 0.f);
                im[r] = fmaxf(im[r], 0.f);
            }
        }
        store_run<E>(y + (size_t)c * m + col, re);
        if (c + Bho < Bo) store_run<E>(y + (size_t)(c + Bho) * m + col, im);
        return;
    } else {
    // A lane holds E consecutive outputs (64 bytes at E = 16), so storing them directly makes every store
    // instruction write 16-byte pieces 64 bytes apart.  The outputs are instead handed over through the tile
    // (free once every thread has taken its bins) in 16-byte pieces, and stored with consecutive lanes on
    // consecutive pieces: whole lines per instruction.  A lane's pieces are permuted (slot = r xor f(thread)) so
    // that both the writes and the reads of the hand-over are free of bank conflicts.
    constexpr int PPL = E / 4;                                  // pieces per lane and sample
    constexpr int NT = Tile<K, EMAX>::NT;
    float4* ot = reinterpret_cast<float4*>(&zs[0][0]);          // [sample][thread][PPL] pieces; K * ROW * 8 >= 2 * NT * E * 4 bytes
    auto slot = [](int t, int r) { return PPL == 4 ? (r ^ ((t >> 1) & 3)) : PPL == 8 ? (r ^ (t & 7)) : r; };
    __syncthreads();   // every thread has taken its bins out of the tile
#pragma unroll
    for (int r = 0; r < PPL; ++r) {
        float o[2][4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            o[0][e] = v[4 * r + e].x + bv[4 * r + e];
            o[1][e] = v[4 * r + e].y + bv[4 * r + e];
            if (relu) {
                o[0][e] = fmaxf(o[0][e], 0.f);
                o[1][e] = fmaxf(o[1][e], 0.f);
            }
        }
        const int sl = slot((int)threadIdx.x, r);
        ot[(size_t)threadIdx.x * PPL + sl] = make_float4(o[0][0], o[0][1], o[0][2], o[0][3]);
        ot[(size_t)(NT + threadIdx.x) * PPL + sl] = make_float4(o[1][0], o[1][1], o[1][2], o[1][3]);
    }
    if (l == 0) {
        offs[gi] = live ? (long long)c * m + (long long)i * K : -1;
        both[gi] = live && c + Bho < Bo;
    }
    __syncthreads();
    constexpr int PPT = K / 4;                                  // pieces per transform
#pragma unroll
    for (int it = 0; it < 2 * PPL; ++it) {
        const int w = it * NT + (int)threadIdx.x;               // (sample, transform, piece), piece fastest
        const int pi = w % PPT, g2 = (w / PPT) % TT, smp = w / (PPT * TT);
        const long long off = offs[g2];
        if (off < 0 || (smp == 1 && !both[g2])) continue;
        const int t = g2 * L + pi / PPL;                        // the thread that produced the piece
        const float4 o = ot[(size_t)(smp * NT + t) * PPL + slot(t, pi % PPL)];
        const float r4[4] = {o.x, o.y, o.z, o.w};
        store_run<4>(y + (size_t)off + (smp ? (size_t)Bho * m : 0) + 4 * pi, r4);
    }
    }
}

// ---- S3: operand Y -> y --------------------------------------------------------------------------
// One transform = (pair c, row block i).  Y[problem][col][row], complex problems with rows 2i, 2i+1 = (Re, Im).
// VEC (p % 4 == 0): 32-byte reads of four consecutive row blocks; otherwise element by element.
template <int K, int EMAX, typename TOUT, bool VEC, bool TWIN = false>
__global__ void __launch_bounds__(Tile<K, EMAX>::NT)
output_ifft_kernel(const float* __restrict__ yop, TOUT* __restrict__ y, 
                   const float* __restrict__ bias, int relu, int m, int p, int Bo, int Bho, long total, int ku, int corr, int pdl_late,
                   int copies_r, int copies_c, size_t copy_stride) {
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L, TT = Tile<K, EMAX>::TT, ROW = Tile<K, EMAX>::ROW;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2* tw = reinterpret_cast<float2*>(smem_raw);
    float2 (*zs)[ROW] = reinterpret_cast<float2 (*)[ROW]>(tw + K);
    load_twiddles<K>(tw);
    if (!pdl_late) pdl_trigger();
    pdl_wait();     // Y is written by the contraction kernel before this one

    const int gi = threadIdx.x / L, l = threadIdx.x % L;
    const long T = (long)blockIdx.x * TT + gi;
    const bool live = T < total;
    const Split sp = split_base((long)blockIdx.x * TT, p);
    int c, i;                     // this thread's transform: sample pair c, row block i
    split_at<TT>(sp, gi, p, c, i);

    // the bias of this thread's outputs is fetched now, long before the epilogue needs it
    float bv[E];
#pragma unroll
    for (int r = 0; r < E; ++r) bv[r] = 0.f;
    if (bias && live && ku == K) load_run<E>(bias + i * K + E * l, bv);

    gather_operand<K, EMAX, VEC, TWIN>(zs, yop, p, Bho, total, sp, copies_r, copies_c, copy_stride);
    __syncthreads();

    const int f2 = lane_residue<K, EMAX>(l);
    float2 v[E];
#pragma unroll
    for (int f1 = 0; f1 < E; ++f1) v[f1] = live ? zs[f2 + L * f1][gi] : make_float2(0.f, 0.f);
    fft_inverse<K, EMAX>(v, l, tw);
    if (pdl_late) pdl_trigger();
    if (ku != K) {
        // embedded block size: v is the linear convolution (2 ku - 1 points) of the zero-padded blocks; the
        // circular one folds it, a[t] = c[t] + c[t + ku].  (corr: v is a linear correlation with lags -ku < s < ku,
        // the negative ones at K + s, and the fold is a[t] = c[t] + c[t - ku].)  The fold crosses lanes, so it goes
        // through the tile.
        __syncthreads();   // every thread has taken its bins out of the tile
        // time-major hand-over, one row of K points per transform; a lane's E points are rotated by the thread's
        // index so that lanes (whose rows of E points are 8 E bytes apart) fall on different banks
        float2* ft = &zs[0][0] + (size_t)gi * K;      // TT * K points fit: ROW >= TT
        const int rot = l + gi * L;
#pragma unroll
        for (int r = 0; r < E; ++r) ft[E * l + ((r + rot) & (E - 1))] = v[r];
        __syncthreads();
        if (!live) return;
        const bool second = c + Bho < Bo;
        float re[E], im[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int t = E * l + r;
            float2 a = v[r];                          // the low part is the lane's own
            const int hi = corr ? K - ku + t : t + ku;
            if (t < ku && (corr ? t > 0 : hi < K)) {
                const int lh = hi / E;
                const float2 b2 = ft[E * lh + (((hi & (E - 1)) + lh + gi * L) & (E - 1))];
                a.x += b2.x;
                a.y += b2.y;
            }
            re[r] = a.x;
            im[r] = a.y;
        }
        TOUT* y0 = y + (size_t)c * m + (size_t)i * ku;
        TOUT* y1 = y + (size_t)(c + Bho) * m + (size_t)i * ku;
        if ((ku & 3) == 0) {
            // rows and blocks start on multiples of four elements: vector loads of the bias, vector stores
#pragma unroll
            for (int g4 = 0; g4 < E; g4 += 4) {
                const int t = E * l + g4;
                if (t >= ku) continue;
                float bb[4] = {0.f, 0.f, 0.f, 0.f};
                if (bias) load_run<4>(bias + i * ku + t, bb);
                float o0[4], o1[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    o0[e] = re[g4 + e] + bb[e];
                    o1[e] = im[g4 + e] + bb[e];
                    if (relu) {
                        o0[e] = fmaxf(o0[e], 0.f);
                        o1[e] = fmaxf(o1[e], 0.f);
                    }
                }
                store_run<4>(y0 + t, o0);
                if (second) store_run<4>(y1 + t, o1);
            }
        } else {
#pragma unroll
            for (int r = 0; r < E; ++r) {
                const int t = E * l + r;
                if (t >= ku) continue;
                const float bb = bias ? __ldg(bias + i * ku + t) : 0.f;
                float o0 = re[r] + bb, o1 = im[r] + bb;
                if (relu) {
                    o0 = fmaxf(o0, 0.f);
                    o1 = fmaxf(o1, 0.f);
                }
                store_one(y0 + t, o0);
                if (second) store_one(y1 + t, o1);
            }
        }
        return;
    }
    long long* offs = reinterpret_cast<long long*>(&zs[0][0] + (size_t)K * ROW);   // [TT] first output element, or -1
    int* both = reinterpret_cast<int*>(offs + TT);                                  // [TT] does the pair's second sample exist
    store_outputs<K, EMAX, TOUT>(v, bv, zs, offs, both, gi, l, live, c, i, y, relu, m, Bo, Bho);
}

// ---- S3 with bulk-copied tiles ------------------------------------------------------------------------
// In the complex problems of Y the (Re, Im) pairs of consecutive transforms are consecutive in memory, so a bin's
// row of the staging tile is one contiguous run of the operand: the tile is fetched by bulk asynchronous copies
// (cp.async.bulk, one per bin, completion counted on an mbarrier) instead of by loads, address arithmetic and
// shared-memory stores of every thread.  CTAs are persistent and the tile is double-buffered: while a tile is
// transformed and stored, the copies of the CTA's next tile are in flight, which keeps enough bytes outstanding to
// run the memory system at its rate.  Mirror bins (f > K/2) arrive un-negated and are conjugated when read; the two
// real bins interleave two runs and are fetched with ordinary loads.  Needs 16-byte aligned runs: Bho * p even.
constexpr uint32_t kBulkSpinLimit = 1u << 22;   // bounded wait: polls before giving up

__device__ __forceinline__ uint32_t bulk_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool bulk_wait(uint64_t* bar, uint32_t parity, uint32_t limit = kBulkSpinLimit) {
    for (uint32_t it = 0; it < limit; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bulk_smem_u32(bar)), "r"(parity) : "memory");
        if (ok) return true;
        if (it > 64) __nanosleep(64);
    }
    return false;
}

template <int K, typename TOUT>
__global__ void __launch_bounds__(Tile<K, 16>::NT, 768 / Tile<K, 16>::NT)
output_ifft_bulk_kernel(const float* __restrict__ yop, TOUT* __restrict__ y, const float* __restrict__ bias, int relu, int m, int p,
                        int Bo, int Bho, long total, int ntiles, int* status, int no_copy, int pdl_late) {
    constexpr int EMAX = 16;
    const uint32_t spin_limit = no_copy ? (1u << 12) : kBulkSpinLimit;   // no_copy: fault injection (tests only)
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L, TT = Tile<K, EMAX>::TT, ROW = Tile<K, EMAX>::ROW;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2* tw = reinterpret_cast<float2*>(smem_raw);
    float2 (*z0)[ROW] = reinterpret_cast<float2 (*)[ROW]>(tw + K);
    auto zbuf = [&](int b) { return z0 + (size_t)b * K; };      // buffer b: K rows further
    long long* offs = reinterpret_cast<long long*>(tw + K + (size_t)2 * K * ROW);
    int* both = reinterpret_cast<int*>(offs + TT);
    uint64_t* full = reinterpret_cast<uint64_t*>(both + TT + (TT & 1));   // 8-byte aligned
    load_twiddles<K>(tw);
    if (threadIdx.x == 0) {
        for (int b = 0; b < 2; ++b)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bulk_smem_u32(&full[b])), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!pdl_late) pdl_trigger();
    pdl_wait();     // Y is written by the contraction kernel before this one

    const size_t cols = 2 * (size_t)Bho;
    const size_t real_sz = cols * p, cplx_sz = 2 * real_sz;
    const int gi = threadIdx.x / L, l = threadIdx.x % L;
    const int f2 = lane_residue<K, EMAX>(l);

    // bytes of one bin's run in a tile, and the two steps of fetching a tile: thread 0 announces the bytes, then (after a
    // CTA barrier) thread f issues the copy of bin f
    auto run_bytes = [&](int tile) {
        const long left = total - (long)tile * TT;
        return (uint32_t)((left < TT ? left : TT) * 8);
    };
    auto announce = [&](int tile, int b) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bulk_smem_u32(&full[b])),
                     "r"((uint32_t)(K - 2) * run_bytes(tile)) : "memory");
    };
    auto fetch = [&](int tile, int b) {
        if (no_copy) return;               // the bytes were announced, nothing is in flight: the wait below runs out
        for (int f = threadIdx.x; f < K; f += Tile<K, EMAX>::NT) {
            if (f == 0 || f == K / 2) continue;
            const bool mirror = f > K / 2;
            const int g = mirror ? K - f : f;
            const float* src = yop + problem_offset(g + 1, real_sz, cplx_sz) + (mirror ? (size_t)Bho * 2 * p : 0) + 2 * (size_t)tile * TT;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(bulk_smem_u32(&zbuf(b)[f][0])), "l"(src), "r"(run_bytes(tile)), "r"(bulk_smem_u32(&full[b])) : "memory");
        }
    };

    int tile = blockIdx.x;
    if (tile < ntiles && threadIdx.x == 0) announce(tile, 0);
    __syncthreads();   // barriers initialised, twiddles ready, bytes announced
    if (tile < ntiles) fetch(tile, 0);

    bool ok = true;
    int it = 0;
    for (; tile < ntiles; tile += gridDim.x, ++it) {
        const int b = it & 1;
        const int next = tile + (int)gridDim.x;
        if (next < ntiles && threadIdx.x == 0) announce(next, b ^ 1);

        const long T = (long)tile * TT + gi;
        const bool live = T < total;
        const Split sp = split_base((long)tile * TT, p);
        int c, i;
        split_at<TT>(sp, gi, p, c, i);
        float bv[E];
#pragma unroll
        for (int r = 0; r < E; ++r) bv[r] = 0.f;
        if (bias && live) load_run<E>(bias + i * K + E * l, bv);

        // the two real bins: (column c, column Bho + c) of problems 0 and 1
        float4 rb = make_float4(0.f, 0.f, 0.f, 0.f);
        const long Tr = (long)tile * TT + threadIdx.x;
        if (threadIdx.x < TT && Tr < total) {
            const float* y0 = yop + Tr;                   // problem 0, first column group
            rb = make_float4(__ldg(y0), __ldg(y0 + (size_t)Bho * p), __ldg(y0 + real_sz), __ldg(y0 + real_sz + (size_t)Bho * p));
        }
        ok = bulk_wait(&full[b], (uint32_t)(it >> 1) & 1u, spin_limit);
        if (threadIdx.x < TT) {
            zbuf(b)[0][threadIdx.x] = make_float2(rb.x, rb.y);
            zbuf(b)[K / 2][threadIdx.x] = make_float2(rb.z, rb.w);
        }
        ok = __syncthreads_and(ok);   // real bins visible; the other buffer's readers finished an iteration ago
        if (!ok) break;
        if (next < ntiles) fetch(next, b ^ 1);

        float2 v[E];
#pragma unroll
        for (int f1 = 0; f1 < E; ++f1) {
            const int f = f2 + L * f1;
            float2 z = zbuf(b)[f][gi];
            if (f > K / 2) z.y = -z.y;
            v[f1] = live ? z : make_float2(0.f, 0.f);
        }
        fft_inverse<K, EMAX>(v, l, tw);
        store_outputs<K, EMAX, TOUT>(v, bv, zbuf(b), offs, both, gi, l, live, c, i, y, relu, m, Bo, Bho);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic accesses to this buffer before its next bulk copies
        __syncthreads();
    }
    if (pdl_late) pdl_trigger();
    if (!ok) {
        // a wait gave up: report it, and give the copies that are still in flight (this tile's; the next tile's
        // have not been issued) one more bounded wait to land before the CTA's shared memory goes away
        if (threadIdx.x == 0) atomicExch(status, 1);
        if (!no_copy) bulk_wait(&full[it & 1], (uint32_t)(it >> 1) & 1u, spin_limit);
    }
}

// ---- relay: operand Y of one layer -> operand X of the next -----------------------------------------
// Between two stacked fully-connected layers with the same block size, the activation y = psi(a + theta) is only
// ever transformed again: this kernel is S3 of the first layer and S1 of the second in one launch, with the
// activation kept in registers (inverse transform, bias, activation, forward transform); y never reaches memory.
// One transform = (pair c, block i); the first layer's row blocks are the second layer's column blocks.
template <int K, int EMAX, int XMODE, bool VEC>
__global__ void __launch_bounds__(Tile<K, EMAX>::NT)
relay_kernel(const float* __restrict__ yop, void* __restrict__ xop, const float* __restrict__ bias, int relu, int p, int B, int Bh,
             long total, int pdl_late) {
    constexpr int E = FftShape<K, EMAX>::E, L = FftShape<K, EMAX>::L, TT = Tile<K, EMAX>::TT, ROW = Tile<K, EMAX>::ROW;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2* tw = reinterpret_cast<float2*>(smem_raw);
    float2 (*zs)[ROW] = reinterpret_cast<float2 (*)[ROW]>(tw + K);
    load_twiddles<K>(tw);
    if (!pdl_late) pdl_trigger();
    pdl_wait();
    const int gi = threadIdx.x / L, l = threadIdx.x % L;
    const long T = (long)blockIdx.x * TT + gi;
    const bool live = T < total;
    const Split sp = split_base((long)blockIdx.x * TT, p);
    int c, i;
    split_at<TT>(sp, gi, p, c, i);
    float bv[E];
#pragma unroll
    for (int r = 0; r < E; ++r) bv[r] = 0.f;
    if (bias && live) load_run<E>(bias + i * K + E * l, bv);

    gather_operand<K, EMAX, VEC>(zs, yop, p, Bh, total, sp);
    __syncthreads();
    const int f2 = lane_residue<K, EMAX>(l);
    float2 v[E];
#pragma unroll
    for (int f1 = 0; f1 < E; ++f1) v[f1] = live ? zs[f2 + L * f1][gi] : make_float2(0.f, 0.f);
    fft_inverse<K, EMAX>(v, l, tw);
    {
        // the second sample of the last pair does not exist when the batch is odd: it must enter the next layer as zero
        const bool second = live && c + Bh < B;
#pragma unroll
        for (int r = 0; r < E; ++r) {
            float re = v[r].x + bv[r], im = v[r].y + bv[r];
            if (relu) {
                re = fmaxf(re, 0.f);
                im = fmaxf(im, 0.f);
            }
            v[r] = make_float2(live ? re : 0.f, second ? im : 0.f);
        }
    }
    fft_forward<K, EMAX>(v, l, tw);
    __syncthreads();  // every thread has taken its bins out of the tile
#pragma unroll
    for (int f1 = 0; f1 < E; ++f1) zs[f2 + L * f1][gi] = v[f1];
    __syncthreads();
    if (pdl_late) pdl_trigger();
    scatter_operand<K, EMAX, XMODE>(zs, xop, p, Bh, total, sp);
}

// ---- launchers -------------------------------------------------------------------------------------
// Kernels whose tile exceeds the default 48 KB of dynamic shared memory (k = 1024) opt in once per device.
template <typename Kern>
static void allow_smem(Kern kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return;
    // remembered per (kernel, device); kernels of different block sizes share one function type, so the key is the pointer
    static thread_local std::vector<std::pair<const void*, int>> configured;
    int dev = 0;
    cudaGetDevice(&dev);
    const std::pair<const void*, int> key(reinterpret_cast<const void*>(kernel), dev);
    for (const auto& c : configured)
        if (c == key) return;
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    configured.push_back(key);
}

template <typename F>
static int dispatch_k(int k, F&& f) {
    switch (k) {
        case 4: return f(std::integral_constant<int, 4>{});
        case 8: return f(std::integral_constant<int, 8>{});
        case 16: return f(std::integral_constant<int, 16>{});
        case 32: return f(std::integral_constant<int, 32>{});
        case 64: return f(std::integral_constant<int, 64>{});
        case 128: return f(std::integral_constant<int, 128>{});
        case 256: return f(std::integral_constant<int, 256>{});
        case 512: return f(std::integral_constant<int, 512>{});
        case 1024: return f(std::integral_constant<int, 1024>{});
    }
    set_error(CIRC_ERR_SHAPE, "block size %d not supported", k);
    return CIRC_ERR_SHAPE;
}

// Points per lane for a launch: 16 (fewest shuffles) when the transforms fill the machine, otherwise 4
// (8 for k = 256), which quarters every thread's dependent chain for problems that are latency-bound.
template <int K>
struct SmallShape {
    static constexpr int EMAX = (K <= 8 || K >= 512) ? 16 : (K <= 128 ? 4 : 8);   // k = 4, 8 already sit in one lane; k >= 512 fills a warp anyway
};
static bool latency_bound(long transforms, int k) {
    const long warps_at_16 = transforms * (k < 16 ? 1 : k / 16) / 32;
    return k >= 16 && warps_at_16 < 148L * 8;
}

int launch_input_fft(const Layer* L, const void* x, void* xop, int xmode, const Extent& ext, cudaStream_t stream, bool twin) {
    const int q = L->geo.q, n = L->n;
    const long total = (long)ext.Bh * q;
    if (xmode != 0 && (q % 4) != 0) {
        set_error(CIRC_ERR_UNSUPPORTED, "bfloat16 operands need q %% 4 == 0 (q=%d)", q);
        return CIRC_ERR_UNSUPPORTED;
    }
    if (twin && (xmode == 0 || embedded(L->geo))) {
        set_error(CIRC_ERR_UNSUPPORTED, "twin columns need a bfloat16 operand and a block size that is its transform size");
        return CIRC_ERR_UNSUPPORTED;
    }
    const bool small = latency_bound(total, L->geo.k);
    // large forwards of power-of-two blocks from 16 to 256: tiles staged by bulk copies, exchange through shared memory
    if (!small && !L->no_bulk_input && input_fft_bulk_supported(L, x, total)) return launch_input_fft_bulk(L, x, xop, xmode, twin, ext, stream);
    auto go = [&](auto kc) -> int {
        constexpr int K = decltype(kc)::value;
        auto with_shape = [&](auto ec) {
            constexpr int EMAX = decltype(ec)::value;
            constexpr int TT = Tile<K, EMAX>::TT;
            const unsigned blocks = (unsigned)((total + TT - 1) / TT);
            auto launch = [&](auto tin, auto mode) {
                using TIN = decltype(tin);
                constexpr int XMODE = decltype(mode)::value;
                auto run = [&](auto kernel) {
                    allow_smem(kernel, Tile<K, EMAX>::SMEM);
                    launch_kernel(dependent_launches(), kernel, dim3(blocks), dim3(Tile<K, EMAX>::NT), Tile<K, EMAX>::SMEM, stream,
                                  static_cast<const TIN*>(x), xop, n, q, ext.B, ext.Bh, total, L->geo.ku, (int)(dependent_launches() == PDL_LATE));
                };
                if constexpr (XMODE != 0) {
                    if (twin) {
                        run(input_fft_kernel<K, EMAX, TIN, XMODE, true>);
                        return;
                    }
                }
                run(input_fft_kernel<K, EMAX, TIN, XMODE, false>);
            };
            const bool bf = L->x_dtype == CIRC_BF16;
            if (xmode == 0) {
                if (bf) launch(__nv_bfloat16{}, std::integral_constant<int, 0>{}); else launch(float{}, std::integral_constant<int, 0>{});
            } else if (xmode == 1) {
                if (bf) launch(__nv_bfloat16{}, std::integral_constant<int, 1>{}); else launch(float{}, std::integral_constant<int, 1>{});
            } else {
                if (bf) launch(__nv_bfloat16{}, std::integral_constant<int, 2>{}); else launch(float{}, std::integral_constant<int, 2>{});
            }
        };
        if (small) with_shape(std::integral_constant<int, SmallShape<K>::EMAX>{});
        else with_shape(std::integral_constant<int, 16>{});
        return CIRC_OK;
    };
    const int rc = dispatch_k(L->geo.k, go);
    if (rc != CIRC_OK) return rc;
    L->last_kernels[0] = KERNEL_S1_LOADS;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

// Resident CTAs per SM of a kernel at a given launch shape, remembered per (kernel, device).
template <typename Kern>
static int blocks_per_sm(Kern kernel, int threads, size_t smem) {
    static thread_local std::vector<std::pair<std::pair<const void*, int>, int>> known;
    int dev = 0;
    cudaGetDevice(&dev);
    const std::pair<const void*, int> key(reinterpret_cast<const void*>(kernel), dev);
    for (const auto& e : known)
        if (e.first == key) return e.second;
    int n = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = 1;
    }
    known.push_back(std::make_pair(key, n));
    return n;
}

template <int K>
static constexpr size_t bulk_smem() {
    return sizeof(float2) * ((size_t)K + (size_t)2 * K * Tile<K, 16>::ROW) + (size_t)Tile<K, 16>::TT * 12 + 32;
}

int launch_output_ifft(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream, bool correlation, bool twin, RowsPieces pieces) {
    const int p = L->geo.p, m = L->m;
    const long total = (long)ext.Bho * p;
    const bool small = latency_bound(total, L->geo.k);
    // large forwards of power-of-two blocks up to 256: tiles fetched by bulk copies, persistent CTAs (needs 16-byte aligned runs)
    // (measured at 16384 x 16384, batch 1024: k = 16: 40.7 -> 35.2 us, k = 64: 33.7 -> 32.5, k = 256: no change; k = 4, whose
    // tile has two bulk rows only, is slower this way and keeps the load-based kernel)
    if (twin && (embedded(L->geo) || correlation)) {
        set_error(CIRC_ERR_UNSUPPORTED, "twin columns need a block size that is its transform size");
        return CIRC_ERR_UNSUPPORTED;
    }
    const size_t copy_stride = (size_t)2 * ext.Bho * p * L->geo.k;     // all problems of Y
    // large forwards of power-of-two blocks: tiles loaded and written by TMA (32 .. 256: one exchange through shared memory;
    // 4 .. 16: one thread per transform).  16384 x 16384, batch 1024, float32: k = 4: 28.7 -> 19.1 us, k = 16: 37 -> 19.1 us.
    if (!small && !correlation && !twin && pieces.real == 0 && !L->no_tma_output && output_ifft_tma_supported(L, y, ext))
        return launch_output_ifft_tma(L, yop, y, ext, stream);
    const bool bulk = !twin && pieces.real == 0 && !small && !embedded(L->geo) && L->geo.k >= 16 && L->geo.k <= 256 && (total & 1) == 0 && total >= 148L * 256 &&
                      (reinterpret_cast<uintptr_t>(yop) & 15u) == 0 && L->dev_status != nullptr;
    if (bulk) {
        auto go = [&](auto kc) -> int {
            constexpr int K = decltype(kc)::value;
            if constexpr (K >= 16 && K <= 256) {
                constexpr int TT = Tile<K, 16>::TT, NT = Tile<K, 16>::NT;
                const long ntiles = (total + TT - 1) / TT;
                if (ntiles >= (1L << 31)) return CIRC_ERR_SHAPE;
                auto launch = [&](auto tout) {
                    using TOUT = decltype(tout);
                    allow_smem(output_ifft_bulk_kernel<K, TOUT>, bulk_smem<K>());
                    int sms = 148;
                    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, L->device);
                    const long resident = (long)sms * blocks_per_sm(output_ifft_bulk_kernel<K, TOUT>, NT, bulk_smem<K>());
                    const unsigned blocks = (unsigned)(ntiles < resident ? ntiles : resident);
                    launch_kernel(dependent_launches(), output_ifft_bulk_kernel<K, TOUT>, dim3(blocks), dim3(NT), bulk_smem<K>(), stream, yop,
                                  static_cast<TOUT*>(y), static_cast<const float*>(L->bias_dev), L->relu, m, p, ext.Bo, ext.Bho, total,
                                  (int)ntiles, L->dev_status, (int)(L->inject == INJECT_BULK_NO_COPY), (int)(dependent_launches() == PDL_LATE));
                };
                if (L->y_dtype == CIRC_BF16) launch(__nv_bfloat16{}); else launch(float{});
            }
            return CIRC_OK;
        };
        const int rc = dispatch_k(L->geo.k, go);
        if (rc != CIRC_OK) return rc;
        L->last_kernels[2] = KERNEL_S3_BULK;
        count_launches(1);
        CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
        return CIRC_OK;
    }
    auto go = [&](auto kc) -> int {
        constexpr int K = decltype(kc)::value;
        auto with_shape = [&](auto ec) {
            constexpr int EMAX = decltype(ec)::value;
            constexpr int TT = Tile<K, EMAX>::TT;
            const unsigned blocks = (unsigned)((total + TT - 1) / TT);
            auto launch = [&](auto tout, auto vec) {
                using TOUT = decltype(tout);
                constexpr bool VEC = decltype(vec)::value;
                auto run = [&](auto kernel) {
                    allow_smem(kernel, Tile<K, EMAX>::SMEM);
                    launch_kernel(dependent_launches(), kernel, dim3(blocks), dim3(Tile<K, EMAX>::NT), Tile<K, EMAX>::SMEM, stream, yop,
                                  static_cast<TOUT*>(y), static_cast<const float*>(L->bias_dev), L->relu, m, p, ext.Bo, ext.Bho, total, L->geo.ku,
                                  (int)correlation, (int)(dependent_launches() == PDL_LATE), pieces.real > 0 ? pieces.real : 1,
                                  pieces.cplx > 0 ? pieces.cplx : 1, copy_stride);
                };
                if (twin) run(output_ifft_kernel<K, EMAX, TOUT, VEC, true>);
                else run(output_ifft_kernel<K, EMAX, TOUT, VEC, false>);
            };
            const bool vec = (p % 4) == 0;
            if (L->y_dtype == CIRC_BF16) {
                if (vec) launch(__nv_bfloat16{}, std::true_type{}); else launch(__nv_bfloat16{}, std::false_type{});
            } else {
                if (vec) launch(float{}, std::true_type{}); else launch(float{}, std::false_type{});
            }
        };
        if (small) with_shape(std::integral_constant<int, SmallShape<K>::EMAX>{});
        else with_shape(std::integral_constant<int, 16>{});
        return CIRC_OK;
    };
    const int rc = dispatch_k(L->geo.k, go);
    if (rc != CIRC_OK) return rc;
    L->last_kernels[2] = KERNEL_S3_LOADS;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int launch_relay(const Layer* L, const float* yop, void* xop_next, int xmode, const Extent& ext, cudaStream_t stream) {
    const int p = L->geo.p;
    const long total = (long)ext.Bho * p;
    if (xmode != 0 && xmode != 1) {
        set_error(CIRC_ERR_ARG, "relay operand mode %d", xmode);
        return CIRC_ERR_ARG;
    }
    if (xmode == 1 && (p % 4) != 0) {
        set_error(CIRC_ERR_UNSUPPORTED, "bfloat16 operands need p %% 4 == 0 (p=%d)", p);
        return CIRC_ERR_UNSUPPORTED;
    }
    const bool small = latency_bound(total, L->geo.k);
    auto go = [&](auto kc) -> int {
        constexpr int K = decltype(kc)::value;
        auto with_shape = [&](auto ec) {
            constexpr int EMAX = decltype(ec)::value;
            constexpr int TT = Tile<K, EMAX>::TT;
            const unsigned blocks = (unsigned)((total + TT - 1) / TT);
            auto launch = [&](auto mode, auto vec) {
                constexpr int XMODE = decltype(mode)::value;
                constexpr bool VEC = decltype(vec)::value;
                allow_smem(relay_kernel<K, EMAX, XMODE, VEC>, Tile<K, EMAX>::SMEM);
                launch_kernel(dependent_launches(), relay_kernel<K, EMAX, XMODE, VEC>, dim3(blocks), dim3(Tile<K, EMAX>::NT), Tile<K, EMAX>::SMEM, stream, yop, xop_next,
                              static_cast<const float*>(L->bias_dev), L->relu, p, ext.Bo, ext.Bho, total, (int)(dependent_launches() == PDL_LATE));
            };
            if (xmode == 1) launch(std::integral_constant<int, 1>{}, std::true_type{});
            else if ((p % 4) == 0) launch(std::integral_constant<int, 0>{}, std::true_type{});
            else launch(std::integral_constant<int, 0>{}, std::false_type{});
        };
        if (small) with_shape(std::integral_constant<int, SmallShape<K>::EMAX>{});
        else with_shape(std::integral_constant<int, 16>{});
        return CIRC_OK;
    };
    const int rc = dispatch_k(L->geo.k, go);
    if (rc != CIRC_OK) return rc;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
