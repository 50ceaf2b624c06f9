"""ctypes binding of ``libcirc.so``: the same names as ``include/circ.h``, argument marshalling only.

Every step of the forward pass runs inside the CUDA library; nothing here computes.  torch (or any
other owner of device memory) is used by callers for allocation and streams only: tensors are
passed as raw device pointers, streams as ``cudaStream_t`` integers.  If the library has not been
built, or cannot be loaded, importing a function from here raises -- there is no fallback path.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "libcirc.so"

CIRC_OK = 0
CIRC_ERR_ARG, CIRC_ERR_SHAPE, CIRC_ERR_ALLOC, CIRC_ERR_CUDA, CIRC_ERR_DEVICE_TIMEOUT, CIRC_ERR_UNSUPPORTED = -1, -2, -3, -4, -5, -6
CIRC_F32, CIRC_BF16 = 0, 1
CIRC_POOL_MAX, CIRC_POOL_AVG, CIRC_POOL_L2 = 0, 1, 2
CIRC_VARIANT_AUTO, CIRC_VARIANT_FUSED, CIRC_VARIANT_STAGED, CIRC_VARIANT_TENSOR = 0, 1, 2, 3
# include/circ_debug.h
CIRC_STAGE_INPUT_FFT, CIRC_STAGE_CONTRACTION, CIRC_STAGE_OUTPUT_IFFT, CIRC_STAGE_FUSED = 0, 1, 2, 3
CIRC_KERNEL_NONE, CIRC_KERNEL_S1_LOADS, CIRC_KERNEL_S1_BULK = 0, 1, 2
CIRC_KERNEL_S2_TENSOR_TWIN, CIRC_KERNEL_S2_ROWS, CIRC_KERNEL_S2_ROWS_TWIN = 12, 13, 14
CIRC_KERNEL_S2_FMA, CIRC_KERNEL_S2_TENSOR, CIRC_KERNEL_S3_LOADS, CIRC_KERNEL_S3_BULK, CIRC_KERNEL_S4_FUSED = 10, 11, 20, 21, 30
CIRC_KERNEL_S3_TMA = 22
CIRC_INJECT_NONE, CIRC_INJECT_TENSOR_NO_COPY, CIRC_INJECT_BULK_NO_COPY = 0, 1, 2

# name -> (restype, argtypes); mirrors include/circ.h one to one
_vp, _ci, _cl = ctypes.c_void_p, ctypes.c_int, ctypes.c_long
SIGNATURES = {
    "circ_fc_create": (_vp, [_ci, _ci, _ci, _vp]),
    "circ_fc_forward": (_ci, [_vp, _vp, _vp, _ci, _vp]),
    "circ_conv_create": (_vp, [_ci, _ci, _ci, _ci, _ci, _vp]),
    "circ_conv_forward": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _vp]),
    "circ_fc_forward_host": (_ci, [_vp, _vp, _vp, _ci, _vp]),
    "circ_conv_forward_host": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _vp]),
    "circ_fc_forward_noalloc": (_ci, [_vp, _vp, _vp, _ci, _vp]),
    "circ_noalloc_max_bytes": (_cl, []),
    "circ_fc_backward": (_ci, [_vp, _vp, _vp, _vp, _vp, _ci, _vp]),
    "circ_conv_backward_input": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _vp]),
    "circ_conv_backward_weight": (_ci, [_vp, _vp, _vp, _vp, _ci, _ci, _ci, _vp]),
    "circ_stack_create": (_vp, [_vp, _ci]),
    "circ_stack_forward": (_ci, [_vp, _vp, _vp, _ci, _vp]),
    "circ_stack_reserve": (_ci, [_vp, _cl]),
    "circ_stack_relayed": (_ci, [_vp]),
    "circ_stack_destroy": (None, [_vp]),
    "circ_device_status": (_ci, [_vp]),
    "circ_destroy": (None, [_vp]),
    "circ_set_bias": (_ci, [_vp, _vp]),
    "circ_set_activation": (_ci, [_vp, _ci]),
    "circ_set_io_dtype": (_ci, [_vp, _ci, _ci]),
    "circ_set_convention": (_ci, [_vp, _ci]),
    "circ_set_spectrum_dtype": (_ci, [_vp, _ci]),
    "circ_set_variant": (_ci, [_vp, _ci]),
    "circ_reserve": (_ci, [_vp, _cl]),
    "circ_workspace_bytes": (_cl, [_vp]),
    "circ_last_variant": (_ci, [_vp]),
    "circ_weight_bytes": (_cl, [_vp]),
    # include/circ_debug.h
    "circ_debug_forward_repeat": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _ci, _ci, _vp]),
    "circ_debug_last_kernels": (_ci, [_vp, _vp]),
    "circ_debug_launch_count": (_cl, []),
    "circ_debug_fma_burn": (_ci, [_vp, _ci, _ci, _vp, _vp]),
    "circ_debug_empty_kernel": (_ci, [_vp]),
    "circ_debug_inject": (_ci, [_vp, _ci]),
    "circ_debug_fail_alloc_after": (_ci, [_cl]),
    "circ_debug_set_fused_split": (_ci, [_vp, _ci]),
    "circ_debug_set_contraction": (_ci, [_vp, _ci, _ci]),
    "circ_debug_set_transforms": (_ci, [_vp, _ci, _ci]),
    "circ_conv_set_stride": (_ci, [_vp, _ci]),
    "circ_pool_forward": (_ci, [_vp, _vp, _ci, _ci, _ci, _ci, _ci, _ci, _ci, _ci, _vp]),
    "circ_last_error": (ctypes.c_char_p, []),
    "circ_last_code": (_ci, []),
}

_lib = None


class CircError(RuntimeError):
    """A libcirc call failed; ``code`` is the CIRC_ERR_* value."""

    def __init__(self, code: int, message: str):
        super().__init__(f"libcirc error {code}: {message}")
        self.code = code


def load() -> ctypes.CDLL:
    """Load ``libcirc.so`` (built by ``paper_1708_08917_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1708_08917_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _ptr(a) -> int | None:
    """Raw address of a torch tensor, a numpy array, an int, or None."""
    if a is None:
        return None
    if isinstance(a, int):
        return a
    if isinstance(a, np.ndarray):
        assert a.flags["C_CONTIGUOUS"]
        return a.ctypes.data
    assert a.is_contiguous()
    return a.data_ptr()


def _stream(stream) -> int | None:
    if stream is None or isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(rc: int) -> None:
    if rc != CIRC_OK:
        raise CircError(rc, circ_last_error())


def _weights(w):
    if isinstance(w, np.ndarray):
        w = np.ascontiguousarray(w, dtype=np.float32)
    return w


def circ_last_error() -> str:
    return load().circ_last_error().decode()


def circ_last_code() -> int:
    return load().circ_last_code()


def circ_fc_create(m: int, n: int, k: int, w) -> int:
    """``w``: float32 ``[p][q][k]`` defining vectors (numpy array on the host or a device tensor)."""
    w = _weights(w)
    h = load().circ_fc_create(m, n, k, _ptr(w))
    if not h:
        raise CircError(circ_last_code(), circ_last_error())
    return h


def circ_conv_create(c_out: int, c_in: int, r: int, pad: int, k: int, w) -> int:
    """``w``: float32 ``[r][r][p][q][k]``."""
    w = _weights(w)
    h = load().circ_conv_create(c_out, c_in, r, pad, k, _ptr(w))
    if not h:
        raise CircError(circ_last_code(), circ_last_error())
    return h


def circ_fc_forward(h: int, x, y, batch: int, stream=None) -> None:
    """Enqueue ``y[batch][m] = psi(W x + theta)``; ``x``, ``y`` are device tensors or raw device addresses."""
    _check(load().circ_fc_forward(h, _ptr(x), _ptr(y), batch, _stream(stream)))


def circ_conv_forward(h: int, x, y, N: int, H: int, W: int, stream=None) -> None:
    """Enqueue the channel-last convolution ``x[N][H][W][C] -> y[N][Ho][Wo][P]``."""
    _check(load().circ_conv_forward(h, _ptr(x), _ptr(y), N, H, W, _stream(stream)))


def circ_conv_set_stride(h: int, stride: int) -> None:
    _check(load().circ_conv_set_stride(h, int(stride)))


def circ_pool_forward(x, y, N: int, H: int, W: int, C: int, window: int, stride: int, mode: int, dtype: int, stream=None) -> None:
    """Enqueue the pooling layer ``x[N][H][W][C] -> y[N][Ho][Wo][C]`` (whole windows, no padding)."""
    _check(load().circ_pool_forward(_ptr(x), _ptr(y), N, H, W, C, window, stride, mode, dtype, _stream(stream)))


def circ_fc_forward_host(h: int, x_host, y_host, batch: int, stream=None) -> None:
    """Host-memory variant: ``x_host`` / ``y_host`` are (pinned) CPU tensors, numpy arrays or addresses."""
    _check(load().circ_fc_forward_host(h, _ptr(x_host), _ptr(y_host), batch, _stream(stream)))


def circ_conv_forward_host(h: int, x_host, y_host, N: int, H: int, W: int, stream=None) -> None:
    _check(load().circ_conv_forward_host(h, _ptr(x_host), _ptr(y_host), N, H, W, _stream(stream)))


def circ_fc_forward_noalloc(h: int, x, y, batch: int, stream=None) -> None:
    """``circ_fc_forward`` for callers that may not allocate: scratch lives in a fixed array inside the library.

    Use it from code that cannot afford (or is not permitted) a ``cudaMalloc`` at forward time.  The batch is
    limited by ``circ_noalloc_max_bytes()``; all calls share one scratch array, so do not overlap them on the GPU;
    make the first call on a device outside stream capture.
    """
    _check(load().circ_fc_forward_noalloc(h, _ptr(x), _ptr(y), batch, _stream(stream)))


def circ_noalloc_max_bytes() -> int:
    return load().circ_noalloc_max_bytes()


def circ_fc_backward(h: int, x, grad_a, grad_x, grad_w, batch: int, stream=None) -> None:
    """Enqueue ``grad_x = W^T grad_a`` and ``grad_w[p][q][k]`` (either may be None) from ``grad_a = dL/da``."""
    _check(load().circ_fc_backward(h, _ptr(x), _ptr(grad_a), _ptr(grad_x), _ptr(grad_w), batch, _stream(stream)))


def circ_conv_backward_input(h: int, grad_y, grad_x, N: int, H: int, W: int, stream=None) -> None:
    """Enqueue ``grad_x[N][H][W][C]`` from ``grad_y[N][Ho][Wo][P]``; ``N, H, W`` are the forward input's extent."""
    _check(load().circ_conv_backward_input(h, _ptr(grad_y), _ptr(grad_x), N, H, W, _stream(stream)))


def circ_conv_backward_weight(h: int, x, grad_y, grad_w, N: int, H: int, W: int, stream=None) -> None:
    """Enqueue ``grad_w[r][r][p][q][k]`` (float32) from the forward input ``x`` and ``grad_y``."""
    _check(load().circ_conv_backward_weight(h, _ptr(x), _ptr(grad_y), _ptr(grad_w), N, H, W, _stream(stream)))


def circ_stack_create(layers) -> int:
    """A stack over fully-connected layer handles (borrowed: destroy the stack first, then the layers)."""
    arr = (ctypes.c_void_p * len(layers))(*layers)
    s = load().circ_stack_create(ctypes.addressof(arr), len(layers))
    if not s:
        raise CircError(circ_last_code(), circ_last_error())
    return s


def circ_stack_forward(s: int, x, y, batch: int, stream=None) -> None:
    """Enqueue all layers; boundaries between staged layers of equal block size run as one relay kernel."""
    _check(load().circ_stack_forward(s, _ptr(x), _ptr(y), batch, _stream(stream)))


def circ_stack_reserve(s: int, max_batch: int) -> None:
    _check(load().circ_stack_reserve(s, max_batch))


def circ_stack_relayed(s: int) -> int:
    return load().circ_stack_relayed(s)


def circ_stack_destroy(s: int | None) -> None:
    load().circ_stack_destroy(s)


def circ_device_status(h: int) -> None:
    """Blocks until the device is idle; raises CircError(CIRC_ERR_DEVICE_TIMEOUT) if a bounded wait expired."""
    _check(load().circ_device_status(h))


def circ_destroy(h: int | None) -> None:
    load().circ_destroy(h)


def circ_set_bias(h: int, bias) -> None:
    if isinstance(bias, np.ndarray):
        bias = np.ascontiguousarray(bias, dtype=np.float32)
    _check(load().circ_set_bias(h, _ptr(bias)))


def circ_set_activation(h: int, relu: int) -> None:
    _check(load().circ_set_activation(h, int(relu)))


def circ_set_io_dtype(h: int, x_dtype: int, y_dtype: int) -> None:
    _check(load().circ_set_io_dtype(h, x_dtype, y_dtype))


def circ_set_convention(h: int, convention: int) -> None:
    _check(load().circ_set_convention(h, convention))


def circ_set_spectrum_dtype(h: int, dtype: int) -> None:
    """CIRC_BF16: the small-batch streaming kernel reads bfloat16 weight spectra (half the bytes)."""
    _check(load().circ_set_spectrum_dtype(h, dtype))


def circ_set_variant(h: int, variant: int) -> None:
    _check(load().circ_set_variant(h, variant))


def circ_reserve(h: int, max_batch: int) -> None:
    _check(load().circ_reserve(h, max_batch))


def circ_workspace_bytes(h: int) -> int:
    return load().circ_workspace_bytes(h)


def circ_last_variant(h: int) -> int:
    return load().circ_last_variant(h)


def circ_weight_bytes(h: int) -> int:
    """Bytes of device memory the handle holds for the layer's weights in all stored forms."""
    return load().circ_weight_bytes(h)


# ---- include/circ_debug.h: test and measurement aids ------------------------------------------------

def circ_debug_forward_repeat(h: int, x, y, N: int, H: int, W: int, stage: int, times: int, stream=None) -> None:
    """The forward pass with the kernel of ``stage`` launched ``times`` times (results unchanged): per-kernel timing."""
    _check(load().circ_debug_forward_repeat(h, _ptr(x), _ptr(y), N, H, W, stage, times, _stream(stream)))


def circ_debug_last_kernels(h: int) -> list[int]:
    """CIRC_KERNEL_* ids of the S1 / S2 / S3 kernels of the handle's most recent staged forward."""
    ids = (ctypes.c_int * 3)()
    _check(load().circ_debug_last_kernels(h, ctypes.addressof(ids)))
    return list(ids)


def circ_debug_launch_count() -> int:
    return load().circ_debug_launch_count()


def circ_debug_fma_burn(sink, blocks: int, iters: int, stream=None) -> float:
    """Enqueue the float32 FMA micro-benchmark kernel; returns the flops of the launch."""
    flops = ctypes.c_double(0.0)
    _check(load().circ_debug_fma_burn(_ptr(sink), blocks, iters, ctypes.addressof(flops), _stream(stream)))
    return flops.value


def circ_debug_empty_kernel(stream=None) -> None:
    _check(load().circ_debug_empty_kernel(_stream(stream)))


def circ_debug_inject(h: int, kind: int) -> None:
    _check(load().circ_debug_inject(h, kind))


def circ_debug_set_fused_split(h: int, slices: int) -> None:
    _check(load().circ_debug_set_fused_split(h, slices))


def circ_debug_set_contraction(h: int, allow_twin: int, allow_rows: int) -> None:
    _check(load().circ_debug_set_contraction(h, int(allow_twin), int(allow_rows)))


def circ_debug_set_transforms(h: int, allow_tma_input: int, allow_tma_output: int = 1) -> None:
    _check(load().circ_debug_set_transforms(h, int(allow_tma_input), int(allow_tma_output)))


def circ_debug_fail_alloc_after(n: int) -> None:
    _check(load().circ_debug_fail_alloc_after(n))
