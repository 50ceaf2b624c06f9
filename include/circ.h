/*
 * circ.h -- C ABI of the block-circulant layer library (CUDA, sm_100a).
 *
 * A layer's m x n weight matrix is cut into p x q square blocks of size k
 * (p = m / k, q = n / k); every block is circulant and is stored as one
 * length-k defining vector w_ij (Sec. 3.1, Eq. 3).  The forward pass is
 *
 *     y_i = psi( IFFT( sum_j FFT(w_ij) o FFT(x_j) ) + theta_i )        (Algorithm 1 + Eq. 1)
 *
 * with the weight spectra computed once at create time, one forward transform
 * per input block, accumulation in the frequency domain, and one inverse
 * transform per output block with bias and ReLU fused.  Convolution layers use
 * the same structure along the channel pair at every filter tap (Sec. 3.2,
 * Eq. 6 and Eq. 7).
 *
 * General rules
 *   - All functions are extern "C"; no exception crosses the boundary.
 *   - Functions returning int return CIRC_OK (0) or a negative CIRC_ERR_* code;
 *     create functions return NULL on error.  circ_last_error() gives a
 *     thread-local message for the most recent failure.
 *   - There is no CPU fallback: every call that computes needs a CUDA device.
 *   - A handle belongs to the device that was current when it was created.
 *   - Calls on one handle must not run concurrently (the handle owns one
 *     workspace); different handles are independent.
 */
#ifndef CIRC_H_
#define CIRC_H_

/*
 * Environment: CIRC_LOG (any value, read once per process) makes the library print one line on stderr for every error,
 * every created layer (shape, block size, bytes of spectra) and every forward (variant, kernels, columns, workspace and
 * stored-form bytes).  Off by default; nothing else in the environment is read.
 */
#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define CIRC_API __attribute__((visibility("default")))
#else
#define CIRC_API
#endif

typedef struct circ_layer* circ_handle; /* opaque, owned by the library */

enum {
    CIRC_OK = 0,
    CIRC_ERR_ARG = -1,            /* NULL / misaligned pointer, bad enum value, wrong handle kind */
    CIRC_ERR_SHAPE = -2,          /* unsupported block size, k does not divide m or n, batch < 1 ... */
    CIRC_ERR_ALLOC = -3,          /* device or host allocation failed */
    CIRC_ERR_CUDA = -4,           /* a CUDA runtime call or a kernel launch failed */
    CIRC_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait gave up */
    CIRC_ERR_UNSUPPORTED = -6     /* valid request that this build cannot serve */
};

enum { CIRC_F32 = 0, CIRC_BF16 = 1 };

/* Kernel variants (circ_set_variant). */
enum {
    CIRC_VARIANT_AUTO = 0,   /* chosen from (p, q, k, batch) */
    CIRC_VARIANT_FUSED = 1,  /* one launch: transform x, stream the spectra, accumulate, inverse transform */
    CIRC_VARIANT_STAGED = 2, /* three launches: transforms, per-frequency contraction on fp32 FMA pipes */
    CIRC_VARIANT_TENSOR = 3  /* three launches, per-frequency contraction on the tensor cores */
};

/*
 * circ_fc_create -- build a fully-connected block-circulant layer (Sec. 3.1).
 *   m, n : output / input widths; k : block size; it must divide both (the paper
 *          defines p = m / k, q = n / k and has no remainder rule; pad on the
 *          caller's side).
 *          Powers of two in [4, 1024] run on a transform of exactly k points.
 *          Blocks above 256 are built from the same small transform with more
 *          butterfly levels (the recursive construction of Sec. 4.1); they run
 *          on the three-launch paths only.
 *          Any other k in [1, 512] (k = 1 is an ordinary dense layer) is embedded:
 *          the circular convolution of length k is the linear convolution of the
 *          zero-padded vectors folded back, a[t] = c[t] + c[t + k], computed on
 *          the next power-of-two transform with at least 2k - 1 points (zero
 *          padding in the input-transform kernel, the fold in the inverse one).
 *          Same results, about (transform size / k) times the work; three-launch
 *          paths only.  The backward calls serve such layers too (the weight
 *          gradient is a circular correlation: it folds as g[t] = c[t] + c[t - k]).
 *   w    : float32 defining vectors, layout [p][q][k]: w[(i*q + j)*k + t] is
 *          element t of w_ij.  HOST or DEVICE pointer (detected); read during
 *          the call, the caller keeps ownership.
 * Circulant convention 0 (default): W_ij[r][c] = w_ij[(r - c) mod k], i.e.
 * a_i = sum_j w_ij (*) x_j (circular convolution), which is what Algorithm 1's
 * FFT product computes.  See circ_set_convention for the other reading.
 * Computes the weight spectra FFT(w_ij) (the quantity the paper keeps in RAM,
 * Sec. 4.2) on the current device and synchronises before returning.
 * Defaults: no bias, identity activation, float32 x and y.
 * Returns NULL on error (CIRC_ERR_SHAPE / ARG / ALLOC / CUDA in circ_last_code()).
 */
CIRC_API circ_handle circ_fc_create(int m, int n, int k, const float* w);

/*
 * circ_fc_forward -- y = psi(W x + theta) for a batch (Eq. 1, Algorithm 1).
 *   x : DEVICE pointer, [batch][n] row-major contiguous, float32 or bfloat16 (circ_set_io_dtype)
 *   y : DEVICE pointer, [batch][m] row-major contiguous; must not alias x
 *   both 16-byte aligned, owned by the caller
 *   stream : a cudaStream_t passed as void* (NULL = legacy default stream)
 * Only enqueues work on `stream`; never synchronises.  After circ_reserve(h, B)
 * a forward with batch <= B allocates nothing; otherwise the workspace grows
 * (cudaMalloc) before the launch.
 */
CIRC_API int circ_fc_forward(circ_handle h, const void* x, void* y, int batch, void* stream);

/*
 * circ_conv_create -- build an r x r, stride-1 block-circulant convolution (Sec. 3.2).
 *   c_out, c_in : output / input channels (P and C of Eq. 6); k divides both
 *   r : filter size (1..7); pad : zero padding on each side (0..r-1)
 *   w : float32 [r][r][p][q][k], p = c_out / k, q = c_in / k: at every tap (i, j)
 *       the channel pair is a p x q grid of circulant blocks (Eq. 7), same
 *       convention as the FC layer.  HOST or DEVICE pointer.
 * Defaults: no bias, identity, bfloat16 x and y (change with circ_set_io_dtype).
 */
CIRC_API circ_handle circ_conv_create(int c_out, int c_in, int r, int pad, int k, const float* w);

/*
 * circ_conv_forward -- Eq. 6 with zero padding (cross-correlation, no filter flip):
 *   y[n][h][w][P] = psi( theta + sum_{i,j<r} sum_c F(i,j,c,P) x[n][h+i-pad][w+j-pad][c] ),  out-of-image x = 0
 *   x : DEVICE pointer, channel-last [N][H][W][c_in]
 *   y : DEVICE pointer, channel-last [N][H + 2 pad - r + 1][W + 2 pad - r + 1][c_out]
 * Same stream / allocation / alignment rules as circ_fc_forward.
 */
CIRC_API int circ_conv_forward(circ_handle h, const void* x, void* y, int N, int H, int W, void* stream);

/*
 * circ_fc_forward_host / circ_conv_forward_host -- the same layers for callers whose tensors live
 * in HOST memory (pinned memory makes the copies asynchronous).  Enqueues on `stream`: a
 * host-to-device copy of x into a staging buffer owned by the handle, the forward pass, and a
 * device-to-host copy of y.  y_host is valid after the stream has been synchronised.  The staging
 * buffers grow on demand (cudaMalloc) and are reused by later calls.
 */
CIRC_API int circ_fc_forward_host(circ_handle h, const void* x_host, void* y_host, int batch, void* stream);
CIRC_API int circ_conv_forward_host(circ_handle h, const void* x_host, void* y_host, int N, int H, int W, void* stream);

/*
 * circ_fc_forward_noalloc -- circ_fc_forward for callers that must not allocate device memory.
 * (The paper has no counterpart: this is a deployment aid of the library, not part of the method.)
 *
 * Meant for code that cannot call cudaMalloc at forward time: latency-critical loops where an
 * allocation could stall the device, processes whose free memory is owned by another allocator,
 * or plug-ins that only receive pre-made buffers.  This call never calls cudaMalloc, cudaFree or
 * any allocating routine.  Its scratch memory (the frequency-domain operands between the three
 * kernels of the staged path) is a fixed array of CIRC_NOALLOC_SCRATCH_BYTES compiled into the
 * library; every GPU context that loads the library holds that array until it exits.
 *
 *   h, x, y, batch, stream : exactly as circ_fc_forward (x, y DEVICE pointers owned by the caller).
 *   Preparation, while allocation is still allowed: the staged path reads a stored form of the spectra that a handle
 *          builds (allocates) the first time it is needed.  Call circ_set_variant(h, CIRC_VARIANT_STAGED) and
 *          circ_reserve(h, batch) once, or run one circ_fc_forward on that path; this also loads the scratch
 *          array (that is when its bytes are taken from the device) and looks up its address.  Without it this
 *          call fails with CIRC_ERR_UNSUPPORTED rather than allocate.
 *   Limit: 4 * (2 * ceil(batch / 2)) * (p + q) * kt bytes (+ alignment) must fit in the array, kt being the
 *          transform size: k itself for powers of two in [4, 1024], else the smallest power of two >= 2k - 1
 *          (so (p + q) * kt = n + m for power-of-two blocks).  Larger requests fail with CIRC_ERR_SHAPE and a
 *          message that names both numbers.  circ_noalloc_max_bytes() returns the array size.
 *   If no preparation ran on the device, the first call looks up the array's device address
 *   (cudaGetSymbolAddress); make that first call outside any stream capture.
 *   All calls, on all handles and streams, share the one array and leave their intermediate
 *   results in it: two calls whose kernels overlap on the GPU race and corrupt each other, so
 *   issue them on one stream or order them yourself.  Nothing in the array needs clearing between
 *   calls (each stage overwrites everything the next one reads).
 *   Always uses the three-launch float32 FMA path, whatever circ_set_variant says.
 */
#define CIRC_NOALLOC_SCRATCH_BYTES (32 * 1024 * 1024)
CIRC_API int circ_fc_forward_noalloc(circ_handle h, const void* x, void* y, int batch, void* stream);
CIRC_API long circ_noalloc_max_bytes(void);

/*
 * circ_fc_backward -- gradients through a = W x (Algorithm 2), float32 tensors only.
 *   x       : DEVICE pointer, [batch][n], the input of the forward pass (needed for grad_w only)
 *   grad_a  : DEVICE pointer, [batch][m], dL/da, the gradient with respect to the PRE-activation output
 *             (Algorithm 2's input; a caller that used the fused ReLU masks dL/dy with y > 0 first)
 *   grad_x  : DEVICE pointer, [batch][n], receives dL/dx = W^T grad_a; NULL to skip
 *   grad_w  : DEVICE pointer, float32 [p][q][k], receives dL/dw_ij = IFFT(sum_b FFT(grad_a_i) o conj(FFT(x_j)))
 *             (the paper's x' is x with reversed indices, whose transform is conj(FFT(x))); overwritten, not
 *             accumulated; NULL to skip.  The gradient with respect to the bias is the column sum of grad_a and is
 *             left to the caller.
 * Honours circ_set_convention.  The first call builds the transposed layer W^T inside the handle (allocates
 * and synchronises); later calls only enqueue on `stream`, growing the workspace when the batch grows.
 */
CIRC_API int circ_fc_backward(circ_handle h, const void* x, const void* grad_a, void* grad_x, float* grad_w, int batch,
                              void* stream);

/*
 * circ_conv_backward_input -- dL/dx of the convolution (the CONV counterpart of Algorithm 2's dL/dx line; Sec. 3.2):
 *   grad_x[n][h][w][c] = sum_{i,j<r} sum_P F(i,j,c,P) grad_y[n][h-i+pad][w-j+pad][P]      (terms outside grad_y are 0)
 *   grad_y : DEVICE pointer, channel-last [N][H + 2 pad - r + 1][W + 2 pad - r + 1][c_out], element type = the layer's y type
 *   grad_x : DEVICE pointer, channel-last [N][H][W][c_in], element type = the layer's x type
 *   N, H, W : the extent of the forward INPUT (as in circ_conv_forward)
 * It runs as a forward convolution of the transposed layer (taps flipped, channel blocks transposed, defining
 * vectors index-reversed, padding r - 1 - pad), built inside the handle on the first call (allocates, synchronises).
 */
CIRC_API int circ_conv_backward_input(circ_handle h, const void* grad_y, void* grad_x, int N, int H, int W, void* stream);

/*
 * circ_conv_backward_weight -- dL/dw of the convolution (the CONV counterpart of Algorithm 2's dL/dw line; Sec. 3.2):
 *   grad_w[i][j][P-block][C-block][t] = the sum, over the entries of the dense channel block of tap (i, j) that hold
 *   element t of its defining vector, of  sum_{n,ho,wo} grad_y[n][ho][wo][row] * x[n][ho+i-pad][wo+j-pad][column]
 * computed in the frequency domain as IFFT( sum_pixels FFT(grad_y block) o conj(FFT(x block at the tap's offset)) ).
 *   x      : DEVICE pointer, channel-last [N][H][W][c_in], the forward input, element type = the layer's x type
 *   grad_y : DEVICE pointer, channel-last [N][H + 2 pad - r + 1][W + 2 pad - r + 1][c_out], dL/d(pre-activation
 *            output), element type = the layer's y type
 *   grad_w : DEVICE pointer, float32 [r][r][p][q][k] (the layout of circ_conv_create's w); overwritten
 *   N, H, W : the extent of the forward INPUT
 * r <= 7 (CIRC_ERR_UNSUPPORTED otherwise).  The pixel sum is split over thread blocks and added up in a fixed
 * order, so results repeat bit for bit.  Honours circ_set_convention; the first backward call on a handle
 * allocates and synchronises (as circ_conv_backward_input).
 */
CIRC_API int circ_conv_backward_weight(circ_handle h, const void* x, const void* grad_y, float* grad_w, int N, int H, int W,
                                       void* stream);

/*
 * Layer stacks -- several fully-connected layers run as one call (the paper evaluates whole networks, e.g. the
 * FC layers of AlexNet in Sec. 5, and keeps activations on chip between layers).
 *
 * circ_stack_create  : layers[0..count) are fully-connected handles with layers[l].m == layers[l+1].n, on one
 *                      device; the stack BORROWS them (the caller keeps ownership, must keep them alive and destroys
 *                      them after the stack).  Each layer keeps its own bias / activation / variant / dtype settings.
 *                      Returns NULL on error (circ_last_error()).
 * circ_stack_forward : y[batch][m_last] = layer_{count-1}( ... layer_0(x) ... ); x, y DEVICE pointers, 16-byte
 *                      aligned, element types = the first layer's x type / the last layer's y type.  Enqueues on
 *                      `stream`.  Between two consecutive layers that both run on the staged (three-kernel) path
 *                      with the same block size and float32 activations, the inverse transforms of the first and
 *                      the input transforms of the second run as ONE relay kernel and the activation between them
 *                      is never written to memory: 2*count + 1 launches instead of 3*count.  Other boundaries
 *                      (batch <= 8 on the single-launch kernel, different k, bfloat16 in between) go through an
 *                      intermediate buffer owned by the stack.  Results equal those of calling circ_fc_forward
 *                      layer by layer up to float32 rounding.
 * circ_stack_reserve : allocate every workspace for batches up to max_batch now, so that later forwards only
 *                      enqueue (needed before stream capture).
 * circ_stack_relayed : number of layer boundaries the last circ_stack_forward relayed.
 * circ_stack_destroy : frees the stack (not the layers).  NULL is a no-op.
 */
typedef struct circ_stack* circ_stack_handle;
CIRC_API circ_stack_handle circ_stack_create(const circ_handle* layers, int count);
CIRC_API int circ_stack_forward(circ_stack_handle s, const void* x, void* y, int batch, void* stream);
CIRC_API int circ_stack_reserve(circ_stack_handle s, long max_batch);
CIRC_API int circ_stack_relayed(circ_stack_handle s);
CIRC_API void circ_stack_destroy(circ_stack_handle s);

/* circ_destroy -- free a handle and everything it owns.  NULL is a no-op. */
CIRC_API void circ_destroy(circ_handle h);

/* circ_set_bias -- theta of Eq. 1: float32, length m (c_out); HOST or DEVICE pointer, copied.
 * NULL removes the bias. */
CIRC_API int circ_set_bias(circ_handle h, const float* bias);

/* circ_set_activation -- psi of Eq. 1: 0 = identity, 1 = ReLU max(0, v). */
CIRC_API int circ_set_activation(circ_handle h, int relu);

/* circ_set_io_dtype -- element types of x and y in device memory (CIRC_F32 / CIRC_BF16).
 * Arithmetic is float32 inside; bfloat16 outputs are rounded to nearest even.  With bfloat16
 * inputs the tensor-core contraction takes single bfloat16 operands (float32 accumulate);
 * with float32 inputs it takes split (high + low) bfloat16 operands. */
CIRC_API int circ_set_io_dtype(circ_handle h, int x_dtype, int y_dtype);

/* circ_set_convention -- 0: W_ij[r][c] = w_ij[(r-c) mod k] (default, Algorithm 1);
 * 1: W_ij[r][c] = w_ij[(c-r) mod k] (w_ij read literally as the first row with a column
 * vector x).  Recomputes the spectra from the retained copy of w; synchronises. */
CIRC_API int circ_set_convention(circ_handle h, int convention);

/*
 * circ_set_spectrum_dtype -- storage type of the weight spectra that the small-batch streaming kernel reads
 * (Sec. 4.3 keeps FFT(w_ij) in 16-bit words; here the reduced type is bfloat16, round to nearest even).
 *   dtype : CIRC_F32 (default) or CIRC_BF16.
 * With CIRC_BF16 the fused kernel (batch <= 8), which is bound by reading the spectra once, reads half the bytes;
 * arithmetic stays float32.  The result is then the exact layer of the rounded spectra: expect the accuracy class
 * of the bfloat16-activation path (relative error to the output scale ~1e-3, bound 2e-2), not 1e-4.  The larger
 * batch paths are unaffected (the tensor path with bfloat16 activations uses bfloat16 spectra by itself).
 * The first switch to CIRC_BF16 allocates m*n/k*2 bytes and synchronises.
 */
CIRC_API int circ_set_spectrum_dtype(circ_handle h, int dtype);

/* circ_set_variant -- force a kernel variant (CIRC_VARIANT_*); AUTO restores the planner. */
CIRC_API int circ_set_variant(circ_handle h, int variant);

/* circ_reserve -- size the workspace for forwards up to `max_batch` samples (FC) or pixels
 * N*H*W (CONV), so that later forwards allocate nothing. */
CIRC_API int circ_reserve(circ_handle h, long max_batch);

/* circ_workspace_bytes -- bytes of device workspace currently held by the handle. */
CIRC_API long circ_workspace_bytes(circ_handle h);

/* circ_weight_bytes -- bytes of device memory the handle holds for the layer's weights, all stored forms
 * together (the paper's storage figure is m*n/k values, Sec. 3.1: compare against 4*m*n/k). */
CIRC_API long circ_weight_bytes(circ_handle h);

/* circ_last_variant -- the CIRC_VARIANT_* the most recent forward on this handle used. */
CIRC_API int circ_last_variant(circ_handle h);

/* circ_device_status -- waits for the device (blocking copy of the handle's error word) and
 * returns CIRC_ERR_DEVICE_TIMEOUT if a kernel of this handle gave up on a bounded wait (TMA /
 * tensor-core pipeline barriers) since the last call; the word is cleared.  CIRC_OK otherwise. */
CIRC_API int circ_device_status(circ_handle h);

/* circ_last_error / circ_last_code -- message and code of the calling thread's latest failure. */
CIRC_API const char* circ_last_error(void);
CIRC_API int circ_last_code(void);

/*
 * circ_conv_set_stride -- strided convolution: every stride-th output position of Eq. 6 is kept in both directions,
 * y(n, i, j, :) = [Eq. 6](n, stride i, stride j, :), Ho = (H + 2 pad - r) / stride + 1, Wo likewise (the subsampling
 * convolution of the networks the paper evaluates; Eq. 6 itself is stride 1, the default).  Only the positions that are
 * kept are computed: the input tile of the tensor-core contraction is fetched as one sub-tile per phase (row, column offset
 * modulo the stride) by strided TMA boxes, and a filter tap reads a shifted view of its phase's sub-tile.
 *   stride : 1 .. 4.  Strides above 1 need the tensor-core contraction (c_in / k a multiple of 4; circ_conv_forward
 *            returns CIRC_ERR_UNSUPPORTED otherwise) and are not served by the backward calls.
 * Errors: CIRC_ERR_ARG (not a convolution handle), CIRC_ERR_SHAPE (stride out of range).
 */
CIRC_API int circ_conv_set_stride(circ_handle h, int stride);

/* Pooling operations of circ_pool_forward. */
enum { CIRC_POOL_MAX = 0, CIRC_POOL_AVG = 1, CIRC_POOL_L2 = 2 };

/*
 * circ_pool_forward -- the pooling layer (Sec. 2.1: a subsampling of the extracted features by a max, average or
 * L2-norm calculation; Sec. 4.2: one of the operations of the peripheral computing block).  No handle: the layer has
 * no parameters.
 *   x : DEVICE pointer, [N][H][W][C] contiguous (the layout of circ_conv_forward's output), float32 or bfloat16 (dtype)
 *   y : DEVICE pointer, [N][Ho][Wo][C], same element type, Ho = (H - window) / stride + 1, Wo likewise: whole windows
 *       only, no padding; y(n, i, j, c) = op over a, b in [0, window) of x(n, stride i + a, stride j + b, c)
 *   mode : CIRC_POOL_MAX, CIRC_POOL_AVG (arithmetic mean) or CIRC_POOL_L2 (square root of the sum of squares)
 *   dtype : CIRC_F32 or CIRC_BF16 (arithmetic in float32; bfloat16 results rounded to nearest even)
 *   stream : a cudaStream_t passed as void*; the call only enqueues one kernel and allocates nothing
 * Both buffers stay the caller's.  Errors: CIRC_ERR_ARG (NULL or misaligned pointer, unknown mode or dtype),
 * CIRC_ERR_SHAPE (a dimension < 1, window > H or W or 64, stride < 1), CIRC_ERR_CUDA.
 */
CIRC_API int circ_pool_forward(const void* x, void* y, int N, int H, int W, int C, int window, int stride, int mode, int dtype,
                               void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CIRC_H_ */
