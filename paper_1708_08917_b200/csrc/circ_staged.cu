// S1 / C1 (input transforms) and S3 / C3 (inverse transforms + bias + activation) of the
// staged path.  Both kernels hold whole transforms in registers (circ_fft.cuh) and use shared
// memory only to turn the "one transform = contiguous k samples" view of x and y into the
// "one frequency = one matrix" view the per-frequency contraction needs (circ_common.cuh).
#include <type_traits>

#include "circ_common.cuh"
#include "circ_fft.cuh"
#include "circ_io.cuh"

namespace circ {

constexpr int kThreads = 256;

// ---- S1: x -> operand X ------------------------------------------------------------------------
// One transform = (pair c, column block j).  A CTA takes TT = 256 / L consecutive transforms.
template <int K, typename TIN, int XMODE>
__global__ void __launch_bounds__(kThreads)
input_fft_kernel(const TIN* __restrict__ x, void* __restrict__ xop, const float2* __restrict__ tw256, int n, int q,
                 int B, int Bh, long total) {
    constexpr int E = FftShape<K>::E, L = FftShape<K>::L, TT = kThreads / L;
    __shared__ float2 tw[K];
    __shared__ float2 zs[TT][K + 1];
    load_twiddles<K>(tw, tw256);
    __syncthreads();

    const int gi = threadIdx.x / L, l = threadIdx.x % L;
    const long T = (long)blockIdx.x * TT + gi;
    float2 v[E];
    if (T < total) {
        const int c = (int)(T / q), j = (int)(T % q);
        float re[E], im[E];
        load_run<E>(x + (size_t)c * n + (size_t)j * K + E * l, re);
        if (c + Bh < B) {
            load_run<E>(x + (size_t)(c + Bh) * n + (size_t)j * K + E * l, im);
        } else {
#pragma unroll
            for (int r = 0; r < E; ++r) im[r] = 0.f;
        }
#pragma unroll
        for (int r = 0; r < E; ++r) v[r] = make_float2(re[r], im[r]);
    } else {
#pragma unroll
        for (int r = 0; r < E; ++r) v[r] = make_float2(0.f, 0.f);
    }
    fft_forward<K>(v, l, tw);
    const int f2 = lane_residue<K>(l);
#pragma unroll
    for (int f1 = 0; f1 < E; ++f1) zs[gi][f2 + L * f1] = v[f1];
    __syncthreads();

    // Scatter: this thread now serves transform tl for the bins f0, f0 + L, ...
    const int tl = threadIdx.x % TT, f0 = threadIdx.x / TT;
    const long T2 = (long)blockIdx.x * TT + tl;
    if (T2 >= total) return;
    const int c = (int)(T2 / q), j = (int)(T2 % q);
    const size_t cols = 2 * (size_t)Bh;
    // XMODE 0: float32 operand [problem][col][Kq]; 1 / 2: bfloat16 operand [problem][col][part][Kq]
    // with parts (hi, lo) / (hi) for the tensor-core contraction.
    constexpr int NPART = XMODE == 1 ? 2 : 1;
    const size_t real_sz = cols * q * NPART, cplx_sz = 2 * real_sz;
    auto put = [&](int prob, size_t col, int kq, int kk, float val) {
        const size_t at = problem_offset(prob, real_sz, cplx_sz) + col * (size_t)(NPART * kq) + kk;
        if constexpr (XMODE == 0) {
            static_cast<float*>(xop)[at] = val;
        } else {
            __nv_bfloat16* xb = static_cast<__nv_bfloat16*>(xop);
            const __nv_bfloat16 hi = __float2bfloat16_rn(val);
            xb[at] = hi;
            if constexpr (XMODE == 1) xb[at + kq] = __float2bfloat16_rn(val - __bfloat162float(hi));
        }
    };
#pragma unroll
    for (int it = 0; it < E; ++it) {
        const int f = f0 + L * it;
        const float2 z = zs[tl][f];
        if (f == 0 || f == K / 2) {
            const int prob = f == 0 ? 0 : 1;
            put(prob, (size_t)c, q, j, z.x);
            put(prob, (size_t)Bh + c, q, j, z.y);
        } else if (f < K / 2) {
            put(f + 1, (size_t)c, 2 * q, j, z.x);
            put(f + 1, (size_t)c, 2 * q, q + j, z.y);
        } else {
            put(K - f + 1, (size_t)Bh + c, 2 * q, j, z.x);
            put(K - f + 1, (size_t)Bh + c, 2 * q, q + j, -z.y);
        }
    }
}

// ---- S3: operand Y -> y --------------------------------------------------------------------------
// One transform = (pair c, row block i).
template <int K, typename TOUT>
__global__ void __launch_bounds__(kThreads)
output_ifft_kernel(const float* __restrict__ yop, TOUT* __restrict__ y, const float2* __restrict__ tw256,
                   const float* __restrict__ bias, int relu, int m, int p, int Bo, int Bho, long total) {
    constexpr int E = FftShape<K>::E, L = FftShape<K>::L, TT = kThreads / L;
    __shared__ float2 tw[K];
    __shared__ float2 zs[TT][K + 1];
    load_twiddles<K>(tw, tw256);

    {
        const int tl = threadIdx.x % TT, f0 = threadIdx.x / TT;
        const long T2 = (long)blockIdx.x * TT + tl;
        if (T2 < total) {
            const int c = (int)(T2 / p), i = (int)(T2 % p);
            const size_t cols = 2 * (size_t)Bho;
            const size_t real_sz = cols * p, cplx_sz = 2 * real_sz;
#pragma unroll
            for (int it = 0; it < E; ++it) {
                const int f = f0 + L * it;
                float2 z;
                if (f == 0 || f == K / 2) {
                    const float* yg = yop + problem_offset(f == 0 ? 0 : 1, real_sz, cplx_sz);
                    z.x = yg[(size_t)c * p + i];
                    z.y = yg[((size_t)Bho + c) * p + i];
                } else if (f < K / 2) {
                    const float* yg = yop + problem_offset(f + 1, real_sz, cplx_sz) + (size_t)c * 2 * p;
                    z.x = yg[i];
                    z.y = yg[p + i];
                } else {
                    const float* yg = yop + problem_offset(K - f + 1, real_sz, cplx_sz) + ((size_t)Bho + c) * 2 * p;
                    z.x = yg[i];
                    z.y = -yg[p + i];
                }
                zs[tl][f] = z;
            }
        }
    }
    __syncthreads();

    const int gi = threadIdx.x / L, l = threadIdx.x % L;
    const long T = (long)blockIdx.x * TT + gi;
    const bool live = T < total;
    const int f2 = lane_residue<K>(l);
    float2 v[E];
#pragma unroll
    for (int f1 = 0; f1 < E; ++f1) v[f1] = live ? zs[gi][f2 + L * f1] : make_float2(0.f, 0.f);
    fft_inverse<K>(v, l, tw);
    if (!live) return;
    const int c = (int)(T / p), i = (int)(T % p);
    const int col = i * K + E * l;
    float re[E], im[E];
#pragma unroll
    for (int r = 0; r < E; ++r) {
        const float b = bias ? __ldg(bias + col + r) : 0.f;
        re[r] = v[r].x + b;
        im[r] = v[r].y + b;
        if (relu) {
            re[r] = fmaxf(re[r], 0.f);
            im[r] = fmaxf(im[r], 0.f);
        }
    }
    store_run<E>(y + (size_t)c * m + col, re);
    if (c + Bho < Bo) store_run<E>(y + (size_t)(c + Bho) * m + col, im);
}

// ---- launchers -------------------------------------------------------------------------------------
template <typename T, typename F>
static int dispatch_k(int k, F&& f) {
    switch (k) {
        case 4: return f(std::integral_constant<int, 4>{});
        case 8: return f(std::integral_constant<int, 8>{});
        case 16: return f(std::integral_constant<int, 16>{});
        case 32: return f(std::integral_constant<int, 32>{});
        case 64: return f(std::integral_constant<int, 64>{});
        case 128: return f(std::integral_constant<int, 128>{});
        case 256: return f(std::integral_constant<int, 256>{});
    }
    set_error(CIRC_ERR_SHAPE, "block size %d not supported", k);
    return CIRC_ERR_SHAPE;
}

int launch_input_fft(const Layer* L, const void* x, void* xop, int xmode, const Extent& ext, cudaStream_t stream) {
    const int q = L->geo.q, n = L->n;
    const long total = (long)ext.Bh * q;
    auto go = [&](auto kc) -> int {
        constexpr int K = decltype(kc)::value;
        constexpr int TT = kThreads / FftShape<K>::L;
        const unsigned blocks = (unsigned)((total + TT - 1) / TT);
        auto launch = [&](auto tin, auto mode) {
            using TIN = decltype(tin);
            constexpr int XMODE = decltype(mode)::value;
            input_fft_kernel<K, TIN, XMODE><<<blocks, kThreads, 0, stream>>>(static_cast<const TIN*>(x), xop, L->tw256, n, q,
                                                                            ext.B, ext.Bh, total);
        };
        const bool bf = L->x_dtype == CIRC_BF16;
        if (xmode == 0) {
            if (bf) launch(__nv_bfloat16{}, std::integral_constant<int, 0>{}); else launch(float{}, std::integral_constant<int, 0>{});
        } else if (xmode == 1) {
            if (bf) launch(__nv_bfloat16{}, std::integral_constant<int, 1>{}); else launch(float{}, std::integral_constant<int, 1>{});
        } else {
            if (bf) launch(__nv_bfloat16{}, std::integral_constant<int, 2>{}); else launch(float{}, std::integral_constant<int, 2>{});
        }
        return CIRC_OK;
    };
    const int rc = dispatch_k<void>(L->geo.k, go);
    if (rc != CIRC_OK) return rc;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int launch_output_ifft(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream) {
    const int p = L->geo.p, m = L->m;
    const long total = (long)ext.Bho * p;
    auto go = [&](auto kc) -> int {
        constexpr int K = decltype(kc)::value;
        constexpr int TT = kThreads / FftShape<K>::L;
        const unsigned blocks = (unsigned)((total + TT - 1) / TT);
        if (L->y_dtype == CIRC_BF16)
            output_ifft_kernel<K, __nv_bfloat16><<<blocks, kThreads, 0, stream>>>(
                yop, static_cast<__nv_bfloat16*>(y), L->tw256, L->bias_dev, L->relu, m, p, ext.Bo, ext.Bho, total);
        else
            output_ifft_kernel<K, float><<<blocks, kThreads, 0, stream>>>(yop, static_cast<float*>(y), L->tw256,
                                                                          L->bias_dev, L->relu, m, p, ext.Bo, ext.Bho, total);
        return CIRC_OK;
    };
    const int rc = dispatch_k<void>(L->geo.k, go);
    if (rc != CIRC_OK) return rc;
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

}  // namespace circ
