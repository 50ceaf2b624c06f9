// Shared declarations of the block-circulant layer library: the layer object, the
// layouts of the stored spectra and of the frequency-domain operands, and error plumbing.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/circ.h"

namespace circ {

// ---------------------------------------------------------------------------------------------
// Frequency-domain layouts.
//
// Two real signals share one complex transform (see circ_fft.cuh).  Sample (or pixel) b < Bh is the
// real part of pair b, sample Bh + b its imaginary part (Bh = "half": number of pairs).  The size-K
// complex spectrum Z[f] of a pair is multiplied by the weight spectrum What[f], with
// What[K - f] = conj(What[f]) because w is real.  Bins f and K - f therefore share one weight
// matrix, and the per-frequency contraction  Yhat[f] (p x cols) = What[f] (p x q) . Z[f] (q x cols)
// is organised as K/2 + 1 real "problems":
//
//   problem 0 : bin 0          real    M = p,  Kd = q    column c      <- Re Z[0]  of pair c
//   problem 1 : bin K/2        real                      column Bh+c   <- Im Z[..] of pair c
//   problem g+1, 0 < g < K/2 : complex, embedded as a real product
//        [Yr]   [Wr -Wi] [Zr]      M = 2p, Kd = 2q       column c      <- ( Re Z[g],    Im Z[g]   )
//        [Yi] = [Wi  Wr] [Zi]                            column Bh+c   <- ( Re Z[K-g], -Im Z[K-g] )
//   (the second column group is the conjugate of bin K-g, so that it multiplies What[g] too).
//   Real and imaginary parts are interleaved: contraction index 2j / 2j+1 = Re / Im of column
//   block j, row 2i / 2i+1 = Re / Im of row block i, so that the transforms read and write
//   (Re, Im) pairs as one vector.
//
// Every problem has 2*Bh columns.  Operands are "K-major": X[col][kk], A[row][kk]; results are
// Y[col][row].  Convolutions concatenate the taps along the contraction index:
// kk = tap * Kd + (kk within tap), and the column of tap (di, dj) is the input pixel shifted by it.
// ---------------------------------------------------------------------------------------------

struct Geometry {
    int p, q, k;      // block grid and transform size (a power of two)
    int taps;         // 1 for FC, r*r for CONV
    int r, pad;       // CONV filter size and zero padding (r = 1, pad = 0 for FC)
    int ku;           // the caller's block size.  ku == k for powers of two in [4, 1024].  Any other block size is
                      // embedded: a circular convolution of length ku is the linear convolution of the zero-padded
                      // vectors folded back, y[t] = c[t] + c[t + ku], and the linear convolution is a circular one of
                      // any length k >= 2 ku - 1.  S0 and S1 zero-pad w_ij and x_j to k, S3 folds; everything in
                      // between works on k-point spectra and does not know.
    int stride;       // CONV: every stride-th output position of Eq. 6 is kept (1 unless circ_conv_set_stride)
};
__host__ __device__ inline bool embedded(const Geometry& g) { return g.ku != g.k; }

__host__ __device__ inline int problem_of_bin(int g, int k) { return g == 0 ? 0 : (g == k / 2 ? 1 : g + 1); }
__host__ __device__ inline int num_problems(int k) { return k / 2 + 1; }
__host__ __device__ inline bool problem_is_real(int prob) { return prob < 2; }

// Offset (in elements) of problem `prob` inside an operand whose real problems have `real_sz`
// elements each and whose complex problems have `cplx_sz` elements each.
__host__ __device__ inline size_t problem_offset(int prob, size_t real_sz, size_t cplx_sz) {
    return prob < 2 ? (size_t)prob * real_sz : 2 * real_sz + (size_t)(prob - 2) * cplx_sz;
}

// Spatial description of a forward call.  FC: images = 1, H = 1, W = batch (pixels = samples).
struct Extent {
    int B;        // real samples / pixels on the input side (N*H*W)
    int Bh;       // pairs on the input side
    int Bo;       // real samples / pixels on the output side
    int Bho;      // pairs on the output side
    int H, W;     // input image
    int Ho, Wo;   // output image
    int Nh;       // image pairs (CONV); FC: Bh
};

// ---------------------------------------------------------------------------------------------
// The layer object behind circ_handle.
// ---------------------------------------------------------------------------------------------
struct Layer {
    int kind;  // 0 = FC, 1 = CONV
    int device;
    int m, n;  // FC: output / input width; CONV: c_out / c_in
    Geometry geo;
    int convention;
    int relu;
    int x_dtype, y_dtype;
    int variant;
    int last_variant;

    float* w_dev;       // retained copy of the defining vectors [taps][p][q][ku]: embedded block sizes only (a power-of-two
                        // block's vectors can be recovered from its spectra), else nullptr
    float* bias_dev;    // [m] or nullptr
    float* w_stream;    // the canonical stored form, [taps][p][q][k] packed half spectra (m n / k floats); read by the
                        // one-launch kernel.  The operand layouts below are built from it on first use (ensure_forms).
    __nv_bfloat16* w_stream_bf16;  // the same rounded to bfloat16 (only after circ_set_spectrum_dtype), or nullptr
    int w_dtype;        // CIRC_F32 or CIRC_BF16: which stream the fused kernel reads
    float* a_f32;       // embedded float32 operand for the staged FMA contraction
    __nv_bfloat16* a_bf16;  // embedded bfloat16 operand (hi | lo split) for the tensor-core contraction
    __nv_bfloat16* a_twin;  // bfloat16 operand (hi | lo split) with every complex value once, for the twin-column contraction
    size_t a_elems;     // elements of a_f32 (a_bf16 has twice as many, a_twin as many)

    void* ws;           // workspace: frequency-domain operands X and Y
    size_t ws_bytes;
    int* dev_status;    // device error word (bounded waits report here)
    void* x_stage;      // device staging buffers of the host-pointer entry points
    void* y_stage;
    size_t x_stage_bytes, y_stage_bytes;
    mutable int last_kernels[3];  // which S1 / S2 / S3 kernel served the most recent staged forward (KERNEL_* ids below)
    int inject;           // test-only fault injection (circ_debug.h): 0 = none
    int no_bulk_input;    // 1: never use the TMA-staged input transforms (circ_debug_set_transforms)
    int no_tma_output;    // 1: never use the TMA-written inverse transforms (circ_debug_set_transforms)
    int no_rows_kernel;   // 1: never use the row-streaming tensor-core contraction (circ_debug_set_contraction)
    int no_twin;          // 1: never use the twin-column form of the tensor contraction (circ_debug_set_twin)
    int fused_split;      // column slices of the one-launch kernel forced by circ_debug_set_fused_split (0 = planner's choice)
    Layer* transposed;  // the n x m layer W^T (built on first use by the backward pass), or nullptr
};

// Copies of Y that the row-streaming contraction writes for a real / a complex problem ({0, 0}: Y is a single array).
struct RowsPieces {
    int real, cplx;
};

// Kernel ids recorded in Layer::last_kernels (read back through circ_debug_last_kernels).
enum {
    KERNEL_NONE = 0,
    KERNEL_S1_LOADS = 1,      // input transforms, per-thread vector loads
    KERNEL_S1_BULK = 2,       // input transforms, tiles staged by bulk asynchronous copies
    KERNEL_S2_FMA = 10,       // contraction on the float32 FMA pipes
    KERNEL_S2_TENSOR = 11,    // contraction on the tensor cores, embedded weights [Wr -Wi; Wi Wr]
    KERNEL_S2_TENSOR_TWIN = 12,  // contraction on the tensor cores, weights stored once, twin column groups of X
    KERNEL_S2_ROWS = 13,      // row-streaming tensor-core contraction (weight rows on the MMA's M side), embedded weights
    KERNEL_S2_ROWS_TWIN = 14, // the same with twin columns
    KERNEL_S3_LOADS = 20,     // inverse transforms, per-thread loads
    KERNEL_S3_BULK = 21,      // inverse transforms, tiles staged by bulk asynchronous copies
    KERNEL_S3_TMA = 22,       // inverse transforms, one exchange through shared memory, output tile written by TMA
    KERNEL_S4_FUSED = 30      // the one-launch kernel: last_kernels = {this id, column slices, row blocks per thread block}
};

// Test-only fault injection (circ_debug_inject): the named producer issues no copy and every bounded wait of that
// kernel gets a short limit, so that the consumer's wait runs out with nothing in flight.
enum { INJECT_NONE = 0, INJECT_TENSOR_NO_COPY = 1, INJECT_BULK_NO_COPY = 2 };

// Layer life cycle and workspace (circ_api.cu).
Layer* make_layer(int kind, int m, int n, int k, int taps, int r, int pad, const float* w);
void free_layer(Layer* L);
int ensure_workspace(Layer* L, size_t bytes);
// Every device allocation of the library goes through here (tests can make the n-th one fail: circ_debug.h).
cudaError_t dev_alloc(void** ptr, size_t bytes);
template <typename T>
inline cudaError_t dev_alloc(T** ptr, size_t bytes) { return dev_alloc(reinterpret_cast<void**>(ptr), bytes); }
void fail_alloc_after(long n);
long launches_so_far();

// The three stages of the staged forward, each exactly one kernel launch (circ_api.cu).
int staged_operands(Layer* L, const Extent& e, cudaStream_t stream, float** xop, float** yop);
bool stream_is_capturing(cudaStream_t stream);
int stage_input(Layer* L, const void* x, float* xop, const Extent& e, cudaStream_t stream, bool tensor);
int stage_contract(Layer* L, const float* xop, float* yop, const Extent& e, cudaStream_t stream, bool tensor);
int stage_output(Layer* L, const float* yop, void* y, const Extent& e, cudaStream_t stream, bool tensor);
int prepare_staged(Layer* L, const Extent& e, cudaStream_t stream, bool tensor);   // stored form of the path, before the first launch
int staged_dependent_launches(const Layer* L, const Extent& e);
Extent fc_extent(int batch);
Extent conv_extent(const Layer* L, int N, int H, int W);
int plan_fc_variant(const Layer* L, int batch);     // the planner's CIRC_VARIANT_* for a fully-connected forward

// Thread-local error record.
void set_error(int code, const char* fmt, ...);
void count_launches(long n);

#define CIRC_CUDA_TRY(expr, ret)                                                             \
    do {                                                                                     \
        cudaError_t e_ = (expr);                                                             \
        if (e_ != cudaSuccess) {                                                             \
            ::circ::set_error(CIRC_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
            return ret;                                                                      \
        }                                                                                    \
    } while (0)

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched with the "programmatic stream serialization"
// attribute may be scheduled while its predecessor in the stream still runs, so that its launch
// latency and set-up overlap the predecessor's work.  The contract every forward kernel keeps:
//   pdl_trigger()  lets the next kernel's thread blocks be scheduled once every block of this kernel has
//                  issued it (or exited).  Small forwards issue it first thing (PDL_EARLY): the next kernel's
//                  blocks become resident at once and their set-up (twiddle tables, barriers, tensor memory)
//                  overlaps this kernel's work.  Forwards whose kernels fill the machine issue it when a block
//                  has only its stores left (PDL_LATE): resident waiting blocks would take registers and shared
//                  memory away from this kernel's later waves, but the next launch still overlaps the tail.
//   pdl_wait()     before the first access to global memory: blocks until all earlier kernels have
//                  finished and their writes are visible.
// Both are no-ops when the kernel was launched without the attribute.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

enum { PDL_OFF = 0, PDL_EARLY = 1, PDL_LATE = 2 };
// How the staged kernels launched by this thread use programmatic dependent launch (set by the forward pass).
inline int& dependent_launches() {
    static thread_local int mode = PDL_OFF;
    return mode;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(int dependent, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent != PDL_OFF ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------------------------------------
// Kernel launchers (one translation unit each).  All return a CIRC_* code and only enqueue.
// ---------------------------------------------------------------------------------------------

// S0: spectra of the defining vectors (w_dev -> w_stream), then every operand layout the layer already holds.
int launch_precompute(Layer* L, cudaStream_t stream);
// w_stream -> the given operand layouts (null pointers are skipped), and the bfloat16 stream if the layer has one.
int launch_spectrum_forms(Layer* L, float* a_f32, __nv_bfloat16* a_bf16, __nv_bfloat16* a_twin, cudaStream_t stream);
// The other circulant convention of a power-of-two block: conjugate w_stream in place.
int launch_conjugate_stream(Layer* L, cudaStream_t stream);
// Defining vectors [taps][p][q][k] recovered from w_stream (power-of-two blocks).
int launch_defining_vectors(const Layer* L, float* w_out, cudaStream_t stream);
// Stored operand layouts, built on first use.  `forms` is a mask of FORM_*; fails with CIRC_ERR_UNSUPPORTED when a
// form is missing while `stream` is being captured (building allocates).
enum { FORM_A_F32 = 1, FORM_A_BF16 = 2, FORM_A_TWIN = 4 };
// The bfloat16 operands of the tensor-core contractions (X, a_bf16, a_twin) keep their contraction runs a multiple of 8
// entries long (16 bytes: what a TMA stride and the hi | lo part offset need): a layer with q = 4, 12, 20 ... column blocks
// stores them with 4 zero entries (8 for the (Re, Im) runs of complex problems) at the end of every run.
__host__ __device__ inline int padded_q(int q) { return (q + 7) & ~7; }
inline size_t bf16_form_elems(const Layer* L) { return 2 * L->a_elems / L->geo.q * padded_q(L->geo.q); }   // bfloat16 values of a_bf16 (hi and lo)
inline size_t twin_elems(const Layer* L) { return (L->a_elems + (size_t)2 * L->geo.taps * L->geo.p * L->geo.q) / L->geo.q * padded_q(L->geo.q); }   // bfloat16 values of a_twin
int ensure_forms(Layer* L, unsigned forms, cudaStream_t stream);
// How the tensor-core contraction of a forward runs (circ_tensor_rows.cu): `twin`: weights stored once, X twice;
// `rows`: the row-streaming kernel instead of the large-batch one.
struct ContractionPlan {
    bool twin, rows;
};
ContractionPlan plan_contraction(const Layer* L, const Extent& e);
inline bool use_twin(const Layer* L, const Extent& e) { return plan_contraction(L, e).twin; }
int launch_contract_rows(const Layer* L, const __nv_bfloat16* xb, float* yop, const Extent& ext, int nsplit, cudaStream_t stream, bool twin);
// Copies of Y that the row-streaming contraction writes for a real / a complex problem; the inverse-transform kernel
// adds them up.  {0, 0}: Y is a single array.
RowsPieces rows_pieces(const Layer* L, const Extent& e, bool twin);
// Loads the fixed scratch array of the allocation-free entry point and caches its address (circ_noalloc.cu).
int noalloc_warm();
// Rounds w_stream into w_stream_bf16 (which must be allocated).
int launch_round_stream(Layer* L, cudaStream_t stream);

// S1 / C1: forward transforms of the input -> operand X.  xmode 0: float32 [problem][col][Kq];
// 1: bfloat16 [problem][col][hi | lo][Kq] (split of float32 values); 2: bfloat16 [problem][col][Kq].
// `twin` (xmode 1 / 2, fully-connected): complex problems get two column groups, (Zr, -Zi) and (Zi, Zr).
int launch_input_fft(const Layer* L, const void* x, void* xop, int xmode, const Extent& ext, cudaStream_t stream, bool twin = false);

// S1 for large forwards (circ_input_bulk.cu): tiles staged by bulk copies, one exchange through shared memory.
bool input_fft_bulk_supported(const Layer* L, const void* x, long total);
int launch_input_fft_bulk(const Layer* L, const void* x, void* xop, int xmode, bool twin, const Extent& ext, cudaStream_t stream);

// S3 for large forwards (circ_output_bulk.cu): one exchange through shared memory, output tiles written by TMA.
bool output_ifft_tma_supported(const Layer* L, const void* y, const Extent& ext);
int launch_output_ifft_tma(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream);

// S2 / C2 on the float32 FMA pipes: Y = A . X per problem.
int launch_contract_fma(const Layer* L, const float* xop, float* yop, const Extent& ext, cudaStream_t stream);

// S2 / C2 on the tensor cores (bfloat16 operands from xmode 1 or 2, float32 accumulate).
// `twin`: the weights come from a_twin, complex problems have p rows and twice the columns (real parts, then imaginary parts).
int launch_contract_tc(const Layer* L, const __nv_bfloat16* xb, float* yop, const Extent& ext, int nsplit, cudaStream_t stream, bool twin = false);
bool tensor_supported(const Layer* L);

// Tensor-core batch product of the backward pass: for every frequency problem
//   Y[prob][xrow][arow] = sum_col X^T[prob][xrow][col] * A^T[prob][arow][col]
// with both operands as split bfloat16 [prob][row][hi | lo][cols_padded]; real problems have q / p rows,
// complex ones 2q / 2p.  y_real: [2][q][p], y_cplx: [k/2 - 1][2q][2p].
int launch_tc_batch_product(const __nv_bfloat16* xt, int q, const __nv_bfloat16* at, int p, int k, int cols, int cols_padded,
                            float* y_real, float* y_cplx, int* status, cudaStream_t stream);
bool tensor_batch_product_supported(int cols);

// S3 / C3: inverse transforms + bias + activation -> y.
// `correlation`: how an embedded block size folds.  false: a[t] = c[t] + c[t + ku] (the forward pass, a circular
// convolution); true: a[t] = c[t] + c[t - ku] (the weight gradient, a circular correlation whose negative lags sit at
// the top of the transform).  Ignored when the block size is the transform size.
// `twin`: Y of the complex problems is [real parts of all columns][imaginary parts of all columns] instead of interleaved rows.
// `pieces`: Y comes as that many copies per real / complex problem, to be added up ({0, 0}: a single array).
int launch_output_ifft(const Layer* L, const float* yop, void* y, const Extent& ext, cudaStream_t stream, bool correlation = false,
                       bool twin = false, RowsPieces pieces = RowsPieces{0, 0});

// S3 of layer L and S1 of the next layer (same k, its q = L's p) in one launch: Y operand -> X operand (xmode 0 or 1).
int launch_relay(const Layer* L, const float* yop, void* xop_next, int xmode, const Extent& ext, cudaStream_t stream);

// S4: the whole FC forward in one launch (small batch, weight-streaming).
int launch_fused_fc(const Layer* L, const void* x, void* y, int batch, cudaStream_t stream);
bool fused_fc_supported(const Layer* L, int batch);
// The planner's choice between the one-launch kernel and the tensor-core path (`tensor_ok`: that path can serve the layer).
bool fused_fc_preferred(const Layer* L, int batch, bool tensor_ok);

}  // namespace circ
