// Test and measurement aids (include/circ_debug.h): separate entry points, nothing here is reached from
// circ_fc_forward / circ_conv_forward.
#include "../../include/circ_debug.h"
#include "circ_common.cuh"

namespace circ {

static_assert((int)CIRC_KERNEL_S1_LOADS == (int)KERNEL_S1_LOADS && (int)CIRC_KERNEL_S1_BULK == (int)KERNEL_S1_BULK &&
                  (int)CIRC_KERNEL_S2_FMA == (int)KERNEL_S2_FMA && (int)CIRC_KERNEL_S2_TENSOR == (int)KERNEL_S2_TENSOR &&
                  (int)CIRC_KERNEL_S2_TENSOR_TWIN == (int)KERNEL_S2_TENSOR_TWIN && (int)CIRC_KERNEL_S2_ROWS == (int)KERNEL_S2_ROWS &&
                  (int)CIRC_KERNEL_S2_ROWS_TWIN == (int)KERNEL_S2_ROWS_TWIN &&
                  (int)CIRC_KERNEL_S3_LOADS == (int)KERNEL_S3_LOADS && (int)CIRC_KERNEL_S3_BULK == (int)KERNEL_S3_BULK &&
                  (int)CIRC_KERNEL_S4_FUSED == (int)KERNEL_S4_FUSED && (int)CIRC_KERNEL_S3_TMA == (int)KERNEL_S3_TMA,
              "public and internal kernel ids must agree");
static_assert((int)CIRC_INJECT_TENSOR_NO_COPY == (int)INJECT_TENSOR_NO_COPY && (int)CIRC_INJECT_BULK_NO_COPY == (int)INJECT_BULK_NO_COPY,
              "public and internal injection kinds must agree");

// Eight independent dependent chains per thread keep the FMA pipe full whatever its latency.
__global__ void __launch_bounds__(256) fma_burn_kernel(float* sink, int iters) {
    float a[8];
    const float m = 1.0f + 1e-7f * (float)threadIdx.x, c = 1e-9f * (float)blockIdx.x;
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = (float)(i + 1);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = fmaf(a[i], m, c);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += a[i];
    sink[(size_t)blockIdx.x * 256 + threadIdx.x] = s;
}

__global__ void empty_kernel() {}

}  // namespace circ

using namespace circ;

extern "C" {

int circ_debug_forward_repeat(circ_handle h, const void* x, void* y, int N, int H, int W, int stage, int times, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || !x || !y || x == y || stage < 0 || stage > 3 || times < 1 || times > 64 || N < 1) {
        set_error(CIRC_ERR_ARG, "bad handle / pointers, stage %d not in [0,3], times %d not in [1,64] or N < 1", stage, times);
        return CIRC_ERR_ARG;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int variant;
    Extent e;
    if (L->kind == 0) {
        variant = plan_fc_variant(L, N);
        e = fc_extent(N);
    } else {
        if (H < 1 || W < 1 || H + 2 * L->geo.pad < L->geo.r || W + 2 * L->geo.pad < L->geo.r) {
            set_error(CIRC_ERR_SHAPE, "bad image extent");
            return CIRC_ERR_SHAPE;
        }
        variant = L->variant == CIRC_VARIANT_AUTO ? (tensor_supported(L) ? CIRC_VARIANT_TENSOR : CIRC_VARIANT_STAGED) : L->variant;
        e = conv_extent(L, N, H, W);
    }
    int rc = CIRC_OK;
    if (variant == CIRC_VARIANT_FUSED) {
        if (L->kind != 0 || !fused_fc_supported(L, N)) {
            set_error(CIRC_ERR_UNSUPPORTED, "the fused kernel does not serve this call");
            return CIRC_ERR_UNSUPPORTED;
        }
        const int reps = stage == CIRC_STAGE_FUSED ? times : 1;
        for (int rep = 0; rep < reps && rc == CIRC_OK; ++rep) rc = launch_fused_fc(L, x, y, N, s);
        if (rc == CIRC_OK) L->last_variant = CIRC_VARIANT_FUSED;
        return rc;
    }
    const bool tensor = variant == CIRC_VARIANT_TENSOR;
    if (tensor && !tensor_supported(L)) {
        set_error(CIRC_ERR_UNSUPPORTED, "the tensor-core contraction cannot serve this layer");
        return CIRC_ERR_UNSUPPORTED;
    }
    float *xop = nullptr, *yop = nullptr;
    if ((rc = staged_operands(L, e, s, &xop, &yop)) != CIRC_OK) return rc;
    if ((rc = prepare_staged(L, e, s, tensor)) != CIRC_OK) return rc;
    struct DependentGuard {
        DependentGuard(int mode) { dependent_launches() = mode; }
        ~DependentGuard() { dependent_launches() = PDL_OFF; }
    } guard(staged_dependent_launches(L, e));
    for (int rep = 0; rep < (stage == CIRC_STAGE_INPUT_FFT ? times : 1); ++rep)
        if ((rc = stage_input(L, x, xop, e, s, tensor)) != CIRC_OK) return rc;
    for (int rep = 0; rep < (stage == CIRC_STAGE_CONTRACTION ? times : 1); ++rep)
        if ((rc = stage_contract(L, xop, yop, e, s, tensor)) != CIRC_OK) return rc;
    for (int rep = 0; rep < (stage == CIRC_STAGE_OUTPUT_IFFT ? times : 1); ++rep)
        if ((rc = stage_output(L, yop, y, e, s, tensor)) != CIRC_OK) return rc;
    L->last_variant = variant;
    return CIRC_OK;
}

int circ_debug_last_kernels(circ_handle h, int* ids) {
    const Layer* L = reinterpret_cast<const Layer*>(h);
    if (!L || !ids) {
        set_error(CIRC_ERR_ARG, "handle or output pointer is NULL");
        return CIRC_ERR_ARG;
    }
    for (int i = 0; i < 3; ++i) ids[i] = L->last_kernels[i];
    return CIRC_OK;
}

long circ_debug_launch_count(void) { return launches_so_far(); }

int circ_debug_fma_burn(float* sink, int blocks, int iters, double* flops, void* stream) {
    if (!sink || blocks < 1 || iters < 1) {
        set_error(CIRC_ERR_ARG, "sink is NULL, or blocks / iters < 1");
        return CIRC_ERR_ARG;
    }
    fma_burn_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(sink, iters);
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    if (flops) *flops = 2.0 * 8.0 * 256.0 * (double)blocks * (double)iters;
    return CIRC_OK;
}

int circ_debug_empty_kernel(void* stream) {
    empty_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>();
    count_launches(1);
    CIRC_CUDA_TRY(cudaGetLastError(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int circ_debug_inject(circ_handle h, int kind) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || kind < CIRC_INJECT_NONE || kind > CIRC_INJECT_BULK_NO_COPY) {
        set_error(CIRC_ERR_ARG, "bad handle or injection kind %d", kind);
        return CIRC_ERR_ARG;
    }
    L->inject = kind;
    return CIRC_OK;
}

int circ_debug_set_fused_split(circ_handle h, int slices) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || (slices != 0 && slices != 1 && slices != 2 && slices != 4 && slices != 8) || (slices > 0 && L->geo.q % slices)) {
        set_error(CIRC_ERR_ARG, "bad handle, or slices=%d is not 0, 1, 2, 4 or 8 or does not divide q", slices);
        return CIRC_ERR_ARG;
    }
    L->fused_split = slices;
    return CIRC_OK;
}

int circ_debug_set_contraction(circ_handle h, int allow_twin, int allow_rows) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || (allow_twin != 0 && allow_twin != 1) || (allow_rows != 0 && allow_rows != 1)) {
        set_error(CIRC_ERR_ARG, "bad handle or flags %d, %d", allow_twin, allow_rows);
        return CIRC_ERR_ARG;
    }
    L->no_twin = !allow_twin;
    L->no_rows_kernel = !allow_rows;
    return CIRC_OK;
}

int circ_debug_set_transforms(circ_handle h, int allow_tma_input, int allow_tma_output) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || (allow_tma_input != 0 && allow_tma_input != 1) || (allow_tma_output != 0 && allow_tma_output != 1)) {
        set_error(CIRC_ERR_ARG, "bad handle or flags %d, %d", allow_tma_input, allow_tma_output);
        return CIRC_ERR_ARG;
    }
    L->no_bulk_input = !allow_tma_input;
    L->no_tma_output = !allow_tma_output;
    return CIRC_OK;
}

int circ_debug_fail_alloc_after(long n) {
    fail_alloc_after(n);
    return CIRC_OK;
}

}  // extern "C"
