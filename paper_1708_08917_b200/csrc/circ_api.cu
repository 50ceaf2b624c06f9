// The C ABI (include/circ.h): argument checking, the layer object, workspace, variant choice.
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "circ_common.cuh"

namespace circ {

static thread_local char g_err[512] = "";
static thread_local int g_code = CIRC_OK;
static std::atomic<long> g_launches{0};

// CIRC_LOG in the environment (read once): one line on stderr per error, per created layer and per forward.
bool log_enabled() {
    static const bool on = getenv("CIRC_LOG") != nullptr;
    return on;
}
void set_error(int code, const char* fmt, ...) {
    g_code = code;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    if (log_enabled()) fprintf(stderr, "[circ] error %d: %s\n", code, g_err);
}
void log_line(const char* fmt, ...) {
    char buf[384];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    fprintf(stderr, "[circ] %s\n", buf);
}
void count_launches(long n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

// Device allocation with a test hook: fail_alloc_after(n) makes the n-th allocation from now report
// cudaErrorMemoryAllocation without calling the runtime (n = 1: the next one; n <= 0: never).
static std::atomic<long> g_alloc_countdown{0};
void fail_alloc_after(long n) { g_alloc_countdown.store(n > 0 ? n : 0, std::memory_order_relaxed); }
cudaError_t dev_alloc(void** ptr, size_t bytes) {
    long c = g_alloc_countdown.load(std::memory_order_relaxed);
    while (c > 0 && !g_alloc_countdown.compare_exchange_weak(c, c - 1, std::memory_order_relaxed)) {}
    if (c == 1) {
        *ptr = nullptr;
        return cudaErrorMemoryAllocation;
    }
    return cudaMalloc(ptr, bytes);
}

static bool pow2_in_range(int k) { return k >= 4 && k <= 1024 && (k & (k - 1)) == 0; }

// Copy `count` floats from a host or device pointer into fresh device memory.
static int to_device(const float* src, size_t count, float** out) {
    float* d = nullptr;
    if (dev_alloc(&d, count * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        set_error(CIRC_ERR_ALLOC, "cudaMalloc of %zu bytes failed", count * sizeof(float));
        return CIRC_ERR_ALLOC;
    }
    // cudaMemcpyDefault resolves host / device / managed sources under unified addressing.
    cudaError_t e = cudaMemcpy(d, src, count * sizeof(float), cudaMemcpyDefault);
    if (e != cudaSuccess) {
        cudaFree(d);
        set_error(CIRC_ERR_CUDA, "copy of %zu floats failed: %s", count, cudaGetErrorString(e));
        return CIRC_ERR_CUDA;
    }
    *out = d;
    return CIRC_OK;
}

void free_layer(Layer* L) {
    if (!L) return;
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != L->device) cudaSetDevice(L->device);
    cudaFree(L->w_dev);
    cudaFree(L->bias_dev);
    cudaFree(L->w_stream);
    cudaFree(L->w_stream_bf16);
    cudaFree(L->a_f32);
    cudaFree(L->a_bf16);
    cudaFree(L->a_twin);
    cudaFree(L->ws);
    cudaFree(L->dev_status);
    cudaFree(L->x_stage);
    cudaFree(L->y_stage);
    if (L->transposed) free_layer(L->transposed);
    if (prev != L->device && prev >= 0) cudaSetDevice(prev);
    delete L;
}

Layer* make_layer(int kind, int m, int n, int k, int taps, int r, int pad, const float* w) {
    if (!w) {
        set_error(CIRC_ERR_ARG, "w is NULL");
        return nullptr;
    }
    // transform size: k itself for powers of two in [4, 1024]; otherwise the smallest power of two that holds the
    // linear convolution of two length-k vectors (2k - 1 points), which the inverse-transform kernel folds back
    int kt = k;
    if (k >= 1 && !pow2_in_range(k)) {
        kt = 4;
        while (kt < 2 * k - 1 && kt <= 1024) kt <<= 1;
    }
    if (k < 1 || kt > 1024) {
        set_error(CIRC_ERR_SHAPE, "block size k=%d is not supported: powers of two up to 1024, any other size up to 512", k);
        return nullptr;
    }
    if (m <= 0 || n <= 0 || m % k || n % k) {
        set_error(CIRC_ERR_SHAPE, "k=%d must divide m=%d and n=%d (pad on the caller's side)", k, m, n);
        return nullptr;
    }
    Layer* L = new (std::nothrow) Layer();
    if (!L) {
        set_error(CIRC_ERR_ALLOC, "host allocation failed");
        return nullptr;
    }
    memset(L, 0, sizeof(*L));
    L->kind = kind;
    L->m = m;
    L->n = n;
    L->geo = Geometry{m / k, n / k, kt, taps, r, pad, k, 1};
    L->x_dtype = L->y_dtype = (kind == 1 ? CIRC_BF16 : CIRC_F32);
    L->variant = CIRC_VARIANT_AUTO;
    if (cudaGetDevice(&L->device) != cudaSuccess) {
        set_error(CIRC_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
        delete L;
        return nullptr;
    }
    const size_t wcount = (size_t)taps * (m / k) * (n / k) * kt;   // spectra are stored at the transform size
    if (to_device(w, (size_t)taps * (m / k) * (n / k) * k, &L->w_dev) != CIRC_OK) {
        free_layer(L);
        return nullptr;
    }
    const size_t a_real = (size_t)taps * (m / k) * (n / k);
    L->a_elems = 2 * a_real + (size_t)(kt / 2 - 1) * 4 * a_real;
    // Only the packed spectra are made now (the paper's storage figure, m n / k values); the operand layouts of the
    // staged contractions are re-arrangements of them, built when a forward first takes that path.
    bool ok = dev_alloc(&L->w_stream, wcount * sizeof(float)) == cudaSuccess && dev_alloc(&L->dev_status, sizeof(int)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        set_error(CIRC_ERR_ALLOC, "device allocation of the weight spectra failed");
        free_layer(L);
        return nullptr;
    }
    if (cudaMemset(L->dev_status, 0, sizeof(int)) != cudaSuccess || launch_precompute(L, 0) != CIRC_OK ||
        cudaDeviceSynchronize() != cudaSuccess) {
        set_error(CIRC_ERR_CUDA, "spectrum precompute failed: %s", cudaGetErrorString(cudaGetLastError()));
        free_layer(L);
        return nullptr;
    }
    if (!embedded(L->geo)) {   // a power-of-two block's defining vectors can be recovered from its spectra
        cudaFree(L->w_dev);
        L->w_dev = nullptr;
    }
    if (log_enabled())
        log_line("create %s m=%d n=%d k=%d (transform size %d) p=%d q=%d taps=%d spectra=%zu bytes", kind ? "conv" : "fc", m, n, L->geo.ku,
                 L->geo.k, L->geo.p, L->geo.q, taps, (size_t)taps * L->geo.p * L->geo.q * L->geo.k * sizeof(float));
    return L;
}

int ensure_forms(Layer* L, unsigned forms, cudaStream_t stream) {
    const bool need_f32 = (forms & FORM_A_F32) && !L->a_f32, need_bf16 = (forms & FORM_A_BF16) && !L->a_bf16,
               need_twin = (forms & FORM_A_TWIN) && !L->a_twin;
    if (!need_f32 && !need_bf16 && !need_twin) return CIRC_OK;
    if (stream_is_capturing(stream)) {
        set_error(CIRC_ERR_UNSUPPORTED, "this forward needs a stored form of the spectra that has not been built yet, and the stream "
                  "is being captured: call circ_reserve (or run one forward of this size) before the capture");
        return CIRC_ERR_UNSUPPORTED;
    }
    float* a_f32 = nullptr;
    __nv_bfloat16 *a_bf16 = nullptr, *a_twin = nullptr;
    bool ok = true;
    if (need_f32) ok = ok && dev_alloc(&a_f32, L->a_elems * sizeof(float)) == cudaSuccess;
    if (need_bf16) ok = ok && dev_alloc(&a_bf16, bf16_form_elems(L) * sizeof(__nv_bfloat16) + 256) == cudaSuccess;
    if (need_twin) ok = ok && dev_alloc(&a_twin, twin_elems(L) * sizeof(__nv_bfloat16) + 256) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cudaFree(a_f32);
        cudaFree(a_bf16);
        cudaFree(a_twin);
        set_error(CIRC_ERR_ALLOC, "device allocation of a stored form of the spectra failed");
        return CIRC_ERR_ALLOC;
    }
    // on the caller's stream: ordered before the forward that is about to read the new layout
    const int rc = launch_spectrum_forms(L, a_f32, a_bf16, a_twin, stream);
    if (a_f32) {
        L->a_f32 = a_f32;
        if (L->kind == 0) noalloc_warm();   // the allocation-free forward reads this form: have its scratch array resident too
    }
    if (a_bf16) L->a_bf16 = a_bf16;
    if (a_twin) L->a_twin = a_twin;
    return rc;
}

static size_t x_operand_floats(const Layer* L, const Extent& e) {
    const size_t xin = (size_t)2 * e.Bh * padded_q(L->geo.q) * L->geo.k;   // all problems of X (bfloat16 runs may be padded)
    return (use_twin(L, e) ? 2 * xin : xin);                     // twin columns: the complex problems twice
}

// Copies of Y: the row-streaming contraction writes one per piece of its contraction range.
static size_t y_copies(const Layer* L, const Extent& e) {
    const ContractionPlan pl = plan_contraction(L, e);
    return pl.rows ? (size_t)rows_pieces(L, e, pl.twin).cplx : 1;
}

static size_t workspace_need(const Layer* L, const Extent& e) {
    const size_t xin = x_operand_floats(L, e);                   // floats: all problems of X
    const size_t yout = (size_t)2 * e.Bho * L->geo.p * L->geo.k * y_copies(L, e); // floats: all problems of Y (and its copies)
    return (xin + yout) * sizeof(float) + 512;
}

int ensure_workspace(Layer* L, size_t need) {
    if (L->ws_bytes >= need) return CIRC_OK;
    if (L->ws) cudaFree(L->ws);  // implicit synchronisation: earlier forwards have finished with it
    L->ws = nullptr;
    L->ws_bytes = 0;
    if (dev_alloc(&L->ws, need) != cudaSuccess) {
        cudaGetLastError();
        set_error(CIRC_ERR_ALLOC, "workspace allocation of %zu bytes failed", need);
        return CIRC_ERR_ALLOC;
    }
    L->ws_bytes = need;
    return CIRC_OK;
}

Extent fc_extent(int batch) {
    Extent e;
    e.B = e.Bo = batch;
    e.Bh = e.Bho = (batch + 1) / 2;
    e.H = e.Ho = 1;
    e.W = e.Wo = batch;
    e.Nh = e.Bh;
    return e;
}

Extent conv_extent(const Layer* L, int N, int H, int W) {
    Extent e;
    e.H = H;
    e.W = W;
    e.Ho = (H + 2 * L->geo.pad - L->geo.r) / L->geo.stride + 1;
    e.Wo = (W + 2 * L->geo.pad - L->geo.r) / L->geo.stride + 1;
    e.Nh = (N + 1) / 2;
    e.B = N * H * W;
    e.Bh = e.Nh * H * W;
    e.Bo = N * e.Ho * e.Wo;
    e.Bho = e.Nh * e.Ho * e.Wo;
    return e;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_io(const Layer* L, const void* x, const void* y) {
    if (!L) {
        set_error(CIRC_ERR_ARG, "handle is NULL");
        return CIRC_ERR_ARG;
    }
    if (!x || !y || x == y) {
        set_error(CIRC_ERR_ARG, "x and y must be distinct non-NULL device pointers");
        return CIRC_ERR_ARG;
    }
    if (!aligned16(x) || !aligned16(y)) {
        set_error(CIRC_ERR_ARG, "x and y must be 16-byte aligned");
        return CIRC_ERR_ARG;
    }
    return CIRC_OK;
}

// Workspace of a staged forward: operand X, then operand Y.
bool stream_is_capturing(cudaStream_t stream) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &st) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return st != cudaStreamCaptureStatusNone;
}

int staged_operands(Layer* L, const Extent& e, cudaStream_t stream, float** xop, float** yop) {
    const size_t need = workspace_need(L, e);
    if (L->ws_bytes < need && stream_is_capturing(stream)) {
        // growing frees and allocates, which a capturing stream cannot record: say so before anything is enqueued
        set_error(CIRC_ERR_UNSUPPORTED, "the workspace (%zu bytes) is too small for this forward (%zu bytes) and the stream is "
                  "being captured: call circ_reserve before the capture", L->ws_bytes, need);
        return CIRC_ERR_UNSUPPORTED;
    }
    const int rc = ensure_workspace(L, need);
    if (rc != CIRC_OK) return rc;
    *xop = static_cast<float*>(L->ws);
    *yop = *xop + ((x_operand_floats(L, e) + 63) & ~(size_t)63);
    return CIRC_OK;
}

// Small forwards (none of the three kernels fills the machine) overlap each kernel's launch and set-up with its
// predecessor (programmatic dependent launch).
int staged_dependent_launches(const Layer* L, const Extent& e) {
    return (long)e.Bh * (L->geo.p > L->geo.q ? L->geo.p : L->geo.q) * L->geo.k <= 32768 ? PDL_EARLY : PDL_LATE;
}

int prepare_staged(Layer* L, const Extent& e, cudaStream_t stream, bool tensor) {
    return ensure_forms(L, !tensor ? FORM_A_F32 : use_twin(L, e) ? FORM_A_TWIN : FORM_A_BF16, stream);
}

int stage_input(Layer* L, const void* x, float* xop, const Extent& e, cudaStream_t stream, bool tensor) {
    // tensor path: bfloat16 operands, split hi/lo unless the input itself is bfloat16
    const int xmode = !tensor ? 0 : (L->x_dtype == CIRC_BF16 ? 2 : 1);
    return launch_input_fft(L, x, xop, xmode, e, stream, tensor && use_twin(L, e));
}

int stage_contract(Layer* L, const float* xop, float* yop, const Extent& e, cudaStream_t stream, bool tensor) {
    if (tensor) {
        const ContractionPlan pl = plan_contraction(L, e);
        const int nsplit = L->x_dtype == CIRC_BF16 ? 1 : 2;
        if (pl.rows) {
            L->last_kernels[1] = pl.twin ? KERNEL_S2_ROWS_TWIN : KERNEL_S2_ROWS;
            return launch_contract_rows(L, reinterpret_cast<const __nv_bfloat16*>(xop), yop, e, nsplit, stream, pl.twin);
        }
        L->last_kernels[1] = pl.twin ? KERNEL_S2_TENSOR_TWIN : KERNEL_S2_TENSOR;
        return launch_contract_tc(L, reinterpret_cast<const __nv_bfloat16*>(xop), yop, e, nsplit, stream, pl.twin);
    }
    L->last_kernels[1] = KERNEL_S2_FMA;
    return launch_contract_fma(L, xop, yop, e, stream);
}

int stage_output(Layer* L, const float* yop, void* y, const Extent& e, cudaStream_t stream, bool tensor) {
    const ContractionPlan pl = tensor ? plan_contraction(L, e) : ContractionPlan{false, false};
    return launch_output_ifft(L, yop, y, e, stream, false, pl.twin, pl.rows ? rows_pieces(L, e, pl.twin) : RowsPieces{0, 0});
}

static int run_staged(Layer* L, const void* x, void* y, const Extent& e, cudaStream_t stream, bool tensor) {
    float *xop = nullptr, *yop = nullptr;
    int rc = staged_operands(L, e, stream, &xop, &yop);
    if (rc != CIRC_OK) return rc;
    if ((rc = prepare_staged(L, e, stream, tensor)) != CIRC_OK) return rc;
    struct DependentGuard {   // reset on every exit path
        DependentGuard(int mode) { dependent_launches() = mode; }
        ~DependentGuard() { dependent_launches() = PDL_OFF; }
    } guard(staged_dependent_launches(L, e));
    if ((rc = stage_input(L, x, xop, e, stream, tensor)) != CIRC_OK) return rc;
    if ((rc = stage_contract(L, xop, yop, e, stream, tensor)) != CIRC_OK) return rc;
    if ((rc = stage_output(L, yop, y, e, stream, tensor)) != CIRC_OK) return rc;
    L->last_variant = tensor ? CIRC_VARIANT_TENSOR : CIRC_VARIANT_STAGED;
    if (log_enabled())
        log_line("forward %s variant=%s kernels=%d/%d/%d columns=%ld workspace=%zu bytes stored forms=%zu bytes", L->kind ? "conv" : "fc",
                 tensor ? "tensor" : "staged", L->last_kernels[0], L->last_kernels[1], L->last_kernels[2],
                 L->kind ? 2L * e.Nh * e.Ho * e.Wo : 2L * e.Bh, L->ws_bytes, (size_t)circ_weight_bytes(reinterpret_cast<circ_handle>(L)));
    return CIRC_OK;
}

int plan_fc_variant(const Layer* L, int batch) {
    if (L->variant != CIRC_VARIANT_AUTO) return L->variant;
    return fused_fc_preferred(L, batch, tensor_supported(L)) ? CIRC_VARIANT_FUSED
           : tensor_supported(L)                            ? CIRC_VARIANT_TENSOR
                                                            : CIRC_VARIANT_STAGED;
}

}  // namespace circ

using namespace circ;

extern "C" {

circ_handle circ_fc_create(int m, int n, int k, const float* w) {
    return reinterpret_cast<circ_handle>(make_layer(0, m, n, k, 1, 1, 0, w));
}

circ_handle circ_conv_create(int c_out, int c_in, int r, int pad, int k, const float* w) {
    if (r < 1 || r > 7 || pad < 0 || pad >= (r > 1 ? r : 2)) {
        set_error(CIRC_ERR_SHAPE, "filter size r=%d must be in [1,7] and pad=%d in [0,r-1]", r, pad);
        return nullptr;
    }
    return reinterpret_cast<circ_handle>(make_layer(1, c_out, c_in, k, r * r, r, pad, w));
}

void circ_destroy(circ_handle h) { free_layer(reinterpret_cast<Layer*>(h)); }

int circ_fc_forward(circ_handle h, const void* x, void* y, int batch, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    int rc = check_io(L, x, y);
    if (rc != CIRC_OK) return rc;
    if (L->kind != 0) {
        set_error(CIRC_ERR_ARG, "circ_fc_forward called on a convolution handle");
        return CIRC_ERR_ARG;
    }
    if (batch < 1) {
        set_error(CIRC_ERR_SHAPE, "batch=%d must be >= 1", batch);
        return CIRC_ERR_SHAPE;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int variant = plan_fc_variant(L, batch);
    if (variant == CIRC_VARIANT_FUSED) {
        if (!fused_fc_supported(L, batch)) {
            set_error(CIRC_ERR_UNSUPPORTED, "the fused kernel does not serve batch=%d for this layer", batch);
            return CIRC_ERR_UNSUPPORTED;
        }
        rc = launch_fused_fc(L, x, y, batch, s);
        if (rc == CIRC_OK) L->last_variant = CIRC_VARIANT_FUSED;
        if (rc == CIRC_OK && log_enabled())
            log_line("forward fc variant=fused batch=%d column slices=%d row blocks per thread block=%d spectra=%zu bytes", batch,
                     L->last_kernels[1], L->last_kernels[2], (size_t)L->geo.p * L->geo.q * L->geo.k * (L->w_dtype == CIRC_BF16 ? 2 : 4));
        return rc;
    }
    if (variant == CIRC_VARIANT_TENSOR && !tensor_supported(L)) {
        set_error(CIRC_ERR_UNSUPPORTED, "the tensor-core contraction needs q = n/k to be a multiple of 4 (q=%d)", L->geo.q);
        return CIRC_ERR_UNSUPPORTED;
    }
    return run_staged(L, x, y, fc_extent(batch), s, variant == CIRC_VARIANT_TENSOR);
}

int circ_conv_forward(circ_handle h, const void* x, void* y, int N, int H, int W, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    int rc = check_io(L, x, y);
    if (rc != CIRC_OK) return rc;
    if (L->kind != 1) {
        set_error(CIRC_ERR_ARG, "circ_conv_forward called on a fully-connected handle");
        return CIRC_ERR_ARG;
    }
    if (N < 1 || H < 1 || W < 1 || H + 2 * L->geo.pad < L->geo.r || W + 2 * L->geo.pad < L->geo.r) {
        set_error(CIRC_ERR_SHAPE, "bad image extent N=%d H=%d W=%d for r=%d pad=%d", N, H, W, L->geo.r, L->geo.pad);
        return CIRC_ERR_SHAPE;
    }
    if ((long)N * H * W > (1L << 30)) {
        set_error(CIRC_ERR_SHAPE, "N*H*W too large");
        return CIRC_ERR_SHAPE;
    }
    if (L->variant == CIRC_VARIANT_FUSED || (L->variant == CIRC_VARIANT_TENSOR && !tensor_supported(L))) {
        set_error(CIRC_ERR_UNSUPPORTED, "variant %d not available for this convolution", L->variant);
        return CIRC_ERR_UNSUPPORTED;
    }
    const bool tensor = L->variant == CIRC_VARIANT_TENSOR || (L->variant == CIRC_VARIANT_AUTO && tensor_supported(L));
    if (L->geo.stride > 1 && !tensor) {
        set_error(CIRC_ERR_UNSUPPORTED, "a strided convolution runs on the tensor-core contraction only (needs c_in / k to be a multiple of 4)");
        return CIRC_ERR_UNSUPPORTED;
    }
    return run_staged(L, x, y, conv_extent(L, N, H, W), static_cast<cudaStream_t>(stream), tensor);
}

// Grow the device staging buffers of the host-pointer entry points.
static int ensure_stage(Layer* L, size_t xbytes, size_t ybytes) {
    if (L->x_stage_bytes < xbytes) {
        cudaFree(L->x_stage);
        L->x_stage = nullptr;
        L->x_stage_bytes = 0;
        if (dev_alloc(&L->x_stage, xbytes) != cudaSuccess) {
            cudaGetLastError();
            set_error(CIRC_ERR_ALLOC, "staging allocation of %zu bytes failed", xbytes);
            return CIRC_ERR_ALLOC;
        }
        L->x_stage_bytes = xbytes;
    }
    if (L->y_stage_bytes < ybytes) {
        cudaFree(L->y_stage);
        L->y_stage = nullptr;
        L->y_stage_bytes = 0;
        if (dev_alloc(&L->y_stage, ybytes) != cudaSuccess) {
            cudaGetLastError();
            set_error(CIRC_ERR_ALLOC, "staging allocation of %zu bytes failed", ybytes);
            return CIRC_ERR_ALLOC;
        }
        L->y_stage_bytes = ybytes;
    }
    return CIRC_OK;
}

int circ_fc_forward_host(circ_handle h, const void* x_host, void* y_host, int batch, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || !x_host || !y_host || L->kind != 0 || batch < 1) {
        set_error(CIRC_ERR_ARG, "bad handle, NULL host pointer or batch < 1");
        return CIRC_ERR_ARG;
    }
    const size_t xb = (size_t)batch * L->n * (L->x_dtype == CIRC_BF16 ? 2 : 4);
    const size_t yb = (size_t)batch * L->m * (L->y_dtype == CIRC_BF16 ? 2 : 4);
    int rc = ensure_stage(L, xb, yb);
    if (rc != CIRC_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CIRC_CUDA_TRY(cudaMemcpyAsync(L->x_stage, x_host, xb, cudaMemcpyHostToDevice, s), CIRC_ERR_CUDA);
    if ((rc = circ_fc_forward(h, L->x_stage, L->y_stage, batch, stream)) != CIRC_OK) return rc;
    CIRC_CUDA_TRY(cudaMemcpyAsync(y_host, L->y_stage, yb, cudaMemcpyDeviceToHost, s), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int circ_conv_forward_host(circ_handle h, const void* x_host, void* y_host, int N, int H, int W, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || !x_host || !y_host || L->kind != 1 || N < 1 || H < 1 || W < 1) {
        set_error(CIRC_ERR_ARG, "bad handle, NULL host pointer or empty image");
        return CIRC_ERR_ARG;
    }
    const int Ho = (H + 2 * L->geo.pad - L->geo.r) / L->geo.stride + 1, Wo = (W + 2 * L->geo.pad - L->geo.r) / L->geo.stride + 1;
    if (Ho < 1 || Wo < 1) {
        set_error(CIRC_ERR_SHAPE, "image smaller than the filter");
        return CIRC_ERR_SHAPE;
    }
    const size_t xb = (size_t)N * H * W * L->n * (L->x_dtype == CIRC_BF16 ? 2 : 4);
    const size_t yb = (size_t)N * Ho * Wo * L->m * (L->y_dtype == CIRC_BF16 ? 2 : 4);
    int rc = ensure_stage(L, xb, yb);
    if (rc != CIRC_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CIRC_CUDA_TRY(cudaMemcpyAsync(L->x_stage, x_host, xb, cudaMemcpyHostToDevice, s), CIRC_ERR_CUDA);
    if ((rc = circ_conv_forward(h, L->x_stage, L->y_stage, N, H, W, stream)) != CIRC_OK) return rc;
    CIRC_CUDA_TRY(cudaMemcpyAsync(y_host, L->y_stage, yb, cudaMemcpyDeviceToHost, s), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int circ_device_status(circ_handle h) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L) {
        set_error(CIRC_ERR_ARG, "handle is NULL");
        return CIRC_ERR_ARG;
    }
    int word = 0;
    CIRC_CUDA_TRY(cudaMemcpy(&word, L->dev_status, sizeof(int), cudaMemcpyDeviceToHost), CIRC_ERR_CUDA);
    if (word != 0) {
        cudaMemset(L->dev_status, 0, sizeof(int));
        set_error(CIRC_ERR_DEVICE_TIMEOUT, "a bounded device-side wait expired (code %d); the output of that forward is invalid", word);
        return CIRC_ERR_DEVICE_TIMEOUT;
    }
    return CIRC_OK;
}

int circ_set_bias(circ_handle h, const float* bias) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L) {
        set_error(CIRC_ERR_ARG, "handle is NULL");
        return CIRC_ERR_ARG;
    }
    CIRC_CUDA_TRY(cudaDeviceSynchronize(), CIRC_ERR_CUDA);
    cudaFree(L->bias_dev);
    L->bias_dev = nullptr;
    if (!bias) return CIRC_OK;
    return to_device(bias, (size_t)L->m, &L->bias_dev);
}

int circ_set_activation(circ_handle h, int relu) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || (relu != 0 && relu != 1)) {
        set_error(CIRC_ERR_ARG, "bad handle or activation code %d", relu);
        return CIRC_ERR_ARG;
    }
    L->relu = relu;
    return CIRC_OK;
}

int circ_conv_set_stride(circ_handle h, int stride) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || L->kind != 1) {
        set_error(CIRC_ERR_ARG, "circ_conv_set_stride needs a convolution handle");
        return CIRC_ERR_ARG;
    }
    if (stride < 1 || stride > 4) {
        set_error(CIRC_ERR_SHAPE, "stride=%d must be in [1, 4]", stride);
        return CIRC_ERR_SHAPE;
    }
    L->geo.stride = stride;
    return CIRC_OK;
}

int circ_set_io_dtype(circ_handle h, int x_dtype, int y_dtype) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || (x_dtype != CIRC_F32 && x_dtype != CIRC_BF16) || (y_dtype != CIRC_F32 && y_dtype != CIRC_BF16)) {
        set_error(CIRC_ERR_ARG, "bad handle or dtype codes (%d, %d)", x_dtype, y_dtype);
        return CIRC_ERR_ARG;
    }
    L->x_dtype = x_dtype;
    L->y_dtype = y_dtype;
    return CIRC_OK;
}

int circ_set_convention(circ_handle h, int convention) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || (convention != 0 && convention != 1)) {
        set_error(CIRC_ERR_ARG, "bad handle or convention %d", convention);
        return CIRC_ERR_ARG;
    }
    if (convention == L->convention) return CIRC_OK;
    CIRC_CUDA_TRY(cudaDeviceSynchronize(), CIRC_ERR_CUDA);
    L->convention = convention;
    if (L->transposed) {
        free_layer(L->transposed);   // rebuilt on the next backward call
        L->transposed = nullptr;
    }
    // a power-of-two block changes convention by conjugating its spectra; an embedded one is recomputed from its vectors
    int rc = embedded(L->geo) ? launch_precompute(L, 0) : launch_conjugate_stream(L, 0);
    if (rc == CIRC_OK && !embedded(L->geo)) rc = launch_spectrum_forms(L, L->a_f32, L->a_bf16, L->a_twin, 0);
    if (rc != CIRC_OK) return rc;
    CIRC_CUDA_TRY(cudaDeviceSynchronize(), CIRC_ERR_CUDA);
    return CIRC_OK;
}

int circ_set_spectrum_dtype(circ_handle h, int dtype) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || (dtype != CIRC_F32 && dtype != CIRC_BF16)) {
        set_error(CIRC_ERR_ARG, "bad handle or spectrum dtype %d", dtype);
        return CIRC_ERR_ARG;
    }
    if (dtype == CIRC_BF16 && !L->w_stream_bf16) {
        const size_t count = (size_t)L->geo.taps * L->geo.p * L->geo.q * L->geo.k;
        CIRC_CUDA_TRY(cudaDeviceSynchronize(), CIRC_ERR_CUDA);
        if (dev_alloc(&L->w_stream_bf16, count * sizeof(__nv_bfloat16)) != cudaSuccess) {
            cudaGetLastError();
            L->w_stream_bf16 = nullptr;
            set_error(CIRC_ERR_ALLOC, "allocation of the bfloat16 spectra (%zu bytes) failed", count * sizeof(__nv_bfloat16));
            return CIRC_ERR_ALLOC;
        }
        int rc = launch_round_stream(L, 0);
        if (rc != CIRC_OK) return rc;
        CIRC_CUDA_TRY(cudaDeviceSynchronize(), CIRC_ERR_CUDA);
    }
    L->w_dtype = dtype;
    return CIRC_OK;
}

int circ_set_variant(circ_handle h, int variant) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || variant < CIRC_VARIANT_AUTO || variant > CIRC_VARIANT_TENSOR) {
        set_error(CIRC_ERR_ARG, "bad handle or variant %d", variant);
        return CIRC_ERR_ARG;
    }
    L->variant = variant;
    return CIRC_OK;
}

int circ_reserve(circ_handle h, long max_batch) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || max_batch < 1 || max_batch > (1L << 30)) {
        set_error(CIRC_ERR_ARG, "bad handle or max_batch %ld", max_batch);
        return CIRC_ERR_ARG;
    }
    // Bound for both layer kinds: pairs <= ceil(max_batch / 2) + one image's worth of slack is
    // covered by sizing for max_batch pairs on each side.
    Extent e;
    e.Bh = e.Bho = (int)max_batch;
    const size_t plain = ((size_t)2 * e.Bh * L->geo.q * L->geo.k + (size_t)2 * e.Bho * L->geo.p * L->geo.k) * sizeof(float) + 512;
    size_t need = plain;
    if (L->kind == 0 && max_batch <= (1L << 30) / 2) {       // what a forward of exactly this size takes (twin columns, copies of Y)
        const size_t exact = workspace_need(L, fc_extent((int)max_batch));
        if (exact > need) need = exact;
    }
    int rc = ensure_workspace(L, need);
    if (rc != CIRC_OK) return rc;
    // the stored form that a forward of exactly this size reads (other sizes may take another path and build theirs then)
    if (max_batch > (1L << 30) / 2) return CIRC_OK;
    int variant;
    Extent ef;
    if (L->kind == 0) {
        variant = plan_fc_variant(L, (int)max_batch);
        ef = fc_extent((int)max_batch);
    } else {
        variant = L->variant == CIRC_VARIANT_AUTO ? (tensor_supported(L) ? CIRC_VARIANT_TENSOR : CIRC_VARIANT_STAGED) : L->variant;
        ef = e;
    }
    if (variant == CIRC_VARIANT_FUSED) return CIRC_OK;
    if (variant == CIRC_VARIANT_TENSOR && !tensor_supported(L)) return CIRC_OK;   // the forward itself reports it
    return prepare_staged(L, ef, 0, variant == CIRC_VARIANT_TENSOR);
}

long circ_workspace_bytes(circ_handle h) {
    Layer* L = reinterpret_cast<Layer*>(h);
    return L ? (long)L->ws_bytes : 0;
}

long circ_weight_bytes(circ_handle h) {
    const Layer* L = reinterpret_cast<const Layer*>(h);
    if (!L) return 0;
    const size_t blocks = (size_t)L->geo.taps * L->geo.p * L->geo.q;
    size_t b = 0;
    if (L->w_dev) b += blocks * L->geo.ku * sizeof(float);
    if (L->w_stream) b += blocks * L->geo.k * sizeof(float);
    if (L->w_stream_bf16) b += blocks * L->geo.k * sizeof(__nv_bfloat16);
    if (L->a_f32) b += L->a_elems * sizeof(float);
    if (L->a_bf16) b += bf16_form_elems(L) * sizeof(__nv_bfloat16) + 256;
    if (L->a_twin) b += twin_elems(L) * sizeof(__nv_bfloat16) + 256;
    if (L->transposed) b += (size_t)circ_weight_bytes(reinterpret_cast<circ_handle>(L->transposed));
    return (long)b;
}

int circ_last_variant(circ_handle h) {
    Layer* L = reinterpret_cast<Layer*>(h);
    return L ? L->last_variant : 0;
}

const char* circ_last_error(void) { return g_err; }
int circ_last_code(void) { return g_code; }

}  // extern "C"
