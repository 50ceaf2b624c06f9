/*
 * circ_debug.h -- test and measurement aids of the block-circulant layer library.
 *
 * None of these calls is part of the method (the paper has no counterpart) and none of them sits on the
 * path of circ_fc_forward / circ_conv_forward: they are separate entry points of the same shared library,
 * used by the benchmark to time single kernels and by the tests to look inside a forward pass and to
 * exercise error paths without faulting a device.  Same rules as circ.h: extern "C", CIRC_OK or a negative
 * CIRC_ERR_* code, circ_last_error() for the message.
 */
#ifndef CIRC_DEBUG_H_
#define CIRC_DEBUG_H_

#include "circ.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Stages of a forward pass, as numbered by circ_debug_forward_repeat and circ_debug_last_kernels. */
enum {
    CIRC_STAGE_INPUT_FFT = 0,   /* S1: forward transforms of the input blocks */
    CIRC_STAGE_CONTRACTION = 1, /* S2: per-frequency contraction */
    CIRC_STAGE_OUTPUT_IFFT = 2, /* S3: inverse transforms + bias + activation */
    CIRC_STAGE_FUSED = 3        /* S4: the one-launch small-batch kernel */
};

/* Kernel ids reported by circ_debug_last_kernels. */
enum {
    CIRC_KERNEL_NONE = 0,
    CIRC_KERNEL_S1_LOADS = 1,   /* input transforms fed by per-thread vector loads */
    CIRC_KERNEL_S1_BULK = 2,    /* input transforms fed by TMA copies into shared memory */
    CIRC_KERNEL_S2_FMA = 10,    /* contraction on the float32 FMA pipes */
    CIRC_KERNEL_S2_TENSOR = 11, /* contraction on the tensor cores, weights in the embedded real form [Wr -Wi; Wi Wr] */
    CIRC_KERNEL_S2_TENSOR_TWIN = 12, /* contraction on the tensor cores, every complex weight stored once (twin column groups of X) */
    CIRC_KERNEL_S2_ROWS = 13,   /* row-streaming tensor-core contraction (few columns, many row blocks), embedded weights */
    CIRC_KERNEL_S2_ROWS_TWIN = 14, /* row-streaming tensor-core contraction with twin columns */
    CIRC_KERNEL_S3_LOADS = 20,  /* inverse transforms fed by per-thread loads */
    CIRC_KERNEL_S3_BULK = 21,   /* inverse transforms fed by bulk asynchronous copies */
    CIRC_KERNEL_S3_TMA = 22,    /* inverse transforms with tiles loaded and written by TMA (one exchange through shared memory; short blocks: one thread per transform) */
    CIRC_KERNEL_S4_FUSED = 30   /* the one-launch small-batch kernel */
};

/* Fault injection kinds of circ_debug_inject. */
enum {
    CIRC_INJECT_NONE = 0,
    CIRC_INJECT_TENSOR_NO_COPY = 1, /* the tensor-core contraction's producer issues no copy */
    CIRC_INJECT_BULK_NO_COPY = 2    /* the bulk-fed inverse-transform kernel issues no copy */
};

/*
 * circ_debug_forward_repeat -- the same forward pass as circ_fc_forward (fully-connected handle: N = batch,
 * H and W ignored) or circ_conv_forward (convolution handle), except that the kernel of `stage` is launched
 * `times` times back to back (1 <= times <= 64).  Every kernel of the path overwrites its own output from
 * unchanged inputs, so y is the same; the time difference between times = 1 + R and times = 1, divided by R,
 * is that kernel's duration without any per-event overhead.  A stage the chosen variant does not run is
 * ignored.  Same pointer, stream and allocation rules as the forward it mirrors.
 */
CIRC_API int circ_debug_forward_repeat(circ_handle h, const void* x, void* y, int N, int H, int W, int stage, int times,
                                       void* stream);

/* circ_debug_last_kernels -- ids[0..2] = which S1 / S2 / S3 kernel (CIRC_KERNEL_*) the most recent staged
 * forward of this handle launched (HOST pointer to three ints).  After a one-launch forward:
 * ids = { CIRC_KERNEL_S4_FUSED, column slices (thread blocks per cluster), row blocks per thread block }. */
CIRC_API int circ_debug_last_kernels(circ_handle h, int* ids);

/* circ_debug_launch_count -- kernels this library has launched in this process so far. */
CIRC_API long circ_debug_launch_count(void);

/*
 * circ_debug_fma_burn -- enqueue a kernel of independent float32 fused multiply-add chains: `blocks` thread
 * blocks of 256 threads, 8 chains per thread, `iters` steps per chain.  Returns, through flops (HOST
 * pointer), the floating-point operations the launch performs (2 per fused multiply-add); timing it gives
 * the measured float32 FMA rate of the device, the arithmetic roofline of the kernels that run on the
 * ordinary pipes.  sink: DEVICE pointer to at least `blocks` * 256 floats (written, so that nothing is optimised away).
 */
CIRC_API int circ_debug_fma_burn(float* sink, int blocks, int iters, double* flops, void* stream);

/* circ_debug_empty_kernel -- enqueue a kernel of one thread that does nothing: the launch floor. */
CIRC_API int circ_debug_empty_kernel(void* stream);

/*
 * circ_debug_inject -- test-only fault injection on one handle.  With CIRC_INJECT_TENSOR_NO_COPY the next
 * tensor-core contractions of the handle run with a producer that announces its bytes but issues no copy,
 * and with a wait limit of a few thousand polls: the consumer's wait runs out, the thread block raises its
 * abort flag, frees its tensor memory and returns, and circ_device_status reports CIRC_ERR_DEVICE_TIMEOUT.
 * CIRC_INJECT_BULK_NO_COPY does the same to the inverse-transform kernel that stages its tiles by bulk
 * copies.  Nothing is in flight when the wait gives up, nothing faults and nothing waits without a bound.
 * The outputs of such a forward are invalid.  CIRC_INJECT_NONE restores normal operation.
 */
CIRC_API int circ_debug_inject(circ_handle h, int kind);

/* circ_debug_set_fused_split -- force the one-launch kernel to split the layer's columns over `slices` thread
 * blocks per cluster (1, 2, 4 or 8; must divide q); 0 restores the planner's choice.  For tests and tuning. */
CIRC_API int circ_debug_set_fused_split(circ_handle h, int slices);

/* circ_debug_set_contraction -- restrict the planner's choices for the tensor-core contraction of this handle, for
 * tests and tuning that compare the forms on one shape.  allow_twin = 0: never the twin-column form (every complex
 * weight stored once, X twice); allow_rows = 0: never the row-streaming kernel.  1 / 1 (default): the planner decides. */
CIRC_API int circ_debug_set_contraction(circ_handle h, int allow_twin, int allow_rows);

/* circ_debug_set_transforms -- allow_tma_input = 0: the input transforms of this handle never take the kernel that
 * stages its tiles by TMA (the load-based kernel serves every size); allow_tma_output = 0: likewise for the inverse
 * transforms that write their tiles by TMA.  1 / 1 (default): the planner decides. */
CIRC_API int circ_debug_set_transforms(circ_handle h, int allow_tma_input, int allow_tma_output);

/* circ_debug_fail_alloc_after -- the n-th device allocation the library makes from now on fails as if the
 * device were out of memory (n = 1: the next one); n <= 0 cancels.  Exercises the CIRC_ERR_ALLOC paths. */
CIRC_API int circ_debug_fail_alloc_after(long n);

#ifdef __cplusplus
}
#endif
#endif /* CIRC_DEBUG_H_ */
