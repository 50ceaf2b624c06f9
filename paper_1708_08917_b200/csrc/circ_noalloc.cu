// circ_fc_forward_noalloc -- a forward pass for callers that are not allowed to allocate.
//
// Who needs this: code that runs where device allocation is off limits -- a real-time inference
// loop whose latency budget cannot absorb a cudaMalloc (it may synchronise the whole device), a
// host thread sharing the GPU with a framework whose caching allocator owns all free memory, or
// a plug-in that was handed fixed input / output buffers and nothing else.  The regular
// circ_fc_forward may grow the handle's workspace with cudaMalloc; this entry point never does.
//
// It runs the staged fully-connected path (input transforms -> per-frequency FMA contraction ->
// inverse transforms with bias / ReLU) with the frequency-domain operands X and Y placed in the
// fixed device array below instead of an allocated workspace.
#include <atomic>

#include "circ_common.cuh"

namespace circ {

// The scratch area: reserved in every GPU context that loads this library, for its lifetime.
constexpr size_t kNoAllocScratchBytes = (size_t)CIRC_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address.  The
// address is looked up once per device (with that device current) and cached here.
constexpr int kMaxDevices = 64;
static std::atomic<void*> g_scratch_addr[kMaxDevices];

static int scratch_for_current_device(void** out) {
    int dev = -1;
    CIRC_CUDA_TRY(cudaGetDevice(&dev), CIRC_ERR_CUDA);
    if (dev < 0 || dev >= kMaxDevices) {
        set_error(CIRC_ERR_UNSUPPORTED, "device ordinal %d is beyond the %d devices this entry point tracks", dev, kMaxDevices);
        return CIRC_ERR_UNSUPPORTED;
    }
    void* ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        // first use on this device: the runtime loads the module that holds the array (this is when its 32 MiB are
        // taken from the device) and gives its address; concurrent first calls all get the same answer
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) {
            set_error(CIRC_ERR_CUDA, "cudaGetSymbolAddress(scratch) failed: %s", cudaGetErrorString(e));
            return CIRC_ERR_CUDA;
        }
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return CIRC_OK;
}

// Called where the library is allowed to allocate anyway (when the stored form that the allocation-free path reads
// is built): the array's module is loaded and its address known before the first allocation-free forward.
int noalloc_warm() {
    void* p = nullptr;
    return scratch_for_current_device(&p);
}

}  // namespace circ

using namespace circ;

extern "C" {

long circ_noalloc_max_bytes(void) { return (long)kNoAllocScratchBytes; }

int circ_fc_forward_noalloc(circ_handle h, const void* x, void* y, int batch, void* stream) {
    Layer* L = reinterpret_cast<Layer*>(h);
    if (!L || L->kind != 0) {
        set_error(CIRC_ERR_ARG, "circ_fc_forward_noalloc needs a fully-connected handle");
        return CIRC_ERR_ARG;
    }
    if (!x || !y || x == y || (reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(y) & 15u)) {
        set_error(CIRC_ERR_ARG, "x and y must be distinct, non-NULL, 16-byte aligned device pointers");
        return CIRC_ERR_ARG;
    }
    if (batch < 1) {
        set_error(CIRC_ERR_SHAPE, "batch=%d must be >= 1", batch);
        return CIRC_ERR_SHAPE;
    }
    int dev = -1;
    CIRC_CUDA_TRY(cudaGetDevice(&dev), CIRC_ERR_CUDA);
    if (dev != L->device) {
        set_error(CIRC_ERR_ARG, "the handle belongs to device %d but device %d is current", L->device, dev);
        return CIRC_ERR_ARG;
    }
    Extent e;
    e.B = e.Bo = batch;
    e.Bh = e.Bho = (batch + 1) / 2;
    e.H = e.Ho = 1;
    e.W = e.Wo = batch;
    e.Nh = e.Bh;
    // operand X: 2*Bh columns x n floats; operand Y: 2*Bh columns x m floats (all frequencies together)
    const size_t x_floats = ((size_t)2 * e.Bh * L->geo.q * L->geo.k + 63) & ~(size_t)63;
    const size_t y_floats = (size_t)2 * e.Bh * L->geo.p * L->geo.k;
    const size_t need = (x_floats + y_floats) * sizeof(float);
    if (need > kNoAllocScratchBytes) {
        set_error(CIRC_ERR_SHAPE,
                  "batch=%d with m=%d, n=%d needs %zu bytes of scratch; circ_fc_forward_noalloc is limited to %zu bytes "
                  "(use circ_fc_forward, or a smaller batch)",
                  batch, L->m, L->n, need, kNoAllocScratchBytes);
        return CIRC_ERR_SHAPE;
    }
    if (!L->a_f32) {
        // the float32 operand of the staged path is built (allocated) on first use; this call may not allocate
        set_error(CIRC_ERR_UNSUPPORTED,
                  "the stored form the staged path reads has not been built yet: while allocation is still allowed, call "
                  "circ_set_variant(h, CIRC_VARIANT_STAGED) and circ_reserve(h, batch), or run one circ_fc_forward on that path");
        return CIRC_ERR_UNSUPPORTED;
    }
    void* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != CIRC_OK) return rc;
    float* xop = static_cast<float*>(scratch);
    float* yop = xop + x_floats;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Every element of X and Y that a later stage reads is written by the stage before it, so the
    // previous call's contents never need clearing.
    if ((rc = launch_input_fft(L, x, xop, 0, e, s)) != CIRC_OK) return rc;
    if ((rc = launch_contract_fma(L, xop, yop, e, s)) != CIRC_OK) return rc;
    if ((rc = launch_output_ifft(L, yop, y, e, s)) != CIRC_OK) return rc;
    return CIRC_OK;
}

}  // extern "C"
