"""ctypes front end of the CPU oracle (``circ_oracle.c``) -- TEST INFRASTRUCTURE.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / reference
legs of ``bench.py`` may import this package.  It knows nothing of the CUDA
library and imports nothing from it.  Arrays go in and come out as float64;
callers widen their float32 / bfloat16 device inputs exactly before calling.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "circ_oracle.c"
_LIB_PATH = _HERE / "libcirc_oracle.so"
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is missing or stale."""
    if force or not _LIB_PATH.exists() or _LIB_PATH.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB_PATH.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-fvisibility=hidden", "-o", str(tmp),
                        str(_SRC), "-lm"], check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.circ_oracle_threads.restype = ctypes.c_int
    return _lib


def _d(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(_dp)


def threads() -> int:
    """Number of OpenMP threads the layer functions use."""
    return int(_load().circ_oracle_threads())


def expand_block(wij, convention: int = 0) -> np.ndarray:
    """Dense k x k matrix of one circulant block (Eq. 3's W_ij)."""
    wij = _d(wij)
    k = wij.shape[0]
    out = np.empty((k, k), dtype=np.float64)
    _load().circ_oracle_expand_block(ctypes.c_int(k), ctypes.c_int(convention), _ptr(wij), _ptr(out))
    return out


def expand_matrix(w, convention: int = 0) -> np.ndarray:
    """Dense m x n matrix of a whole block-circulant weight ``w[p][q][k]`` (small cases)."""
    w = _d(w)
    p, q, k = w.shape
    out = np.empty((p * k, q * k), dtype=np.float64)
    _load().circ_oracle_expand_matrix(ctypes.c_int(p * k), ctypes.c_int(q * k), ctypes.c_int(k),
                                      ctypes.c_int(convention), _ptr(w), _ptr(out))
    return out


def fc(w, x, bias=None, relu: bool = False, convention: int = 0) -> np.ndarray:
    """``y[B][m] = psi(W x + theta)`` (Eq. 1) with ``w[p][q][k]``, ``x[B][n]``."""
    w = _d(w)
    x = _d(x)
    p, q, k = w.shape
    if x.ndim == 1:
        x = x[None, :]
    batch, n = x.shape
    assert n == q * k, (n, q, k)
    b = None if bias is None else _d(bias)
    y = np.empty((batch, p * k), dtype=np.float64)
    _load().circ_oracle_fc(ctypes.c_int(p * k), ctypes.c_int(n), ctypes.c_int(k), ctypes.c_int(convention),
                           _ptr(w), _ptr(x), _ptr(b), ctypes.c_int(int(relu)), ctypes.c_long(batch), _ptr(y))
    return y


def fc_backward(w, x, g, convention: int = 0, want_gx: bool = True, want_gw: bool = True):
    """Gradients of ``L`` through ``a = W x`` given ``g = dL/da`` (``[B][m]``): returns ``(dL/dx [B][n], dL/dw [p][q][k])``.

    This is what Algorithm 2 computes; here it is the chain rule on the dense expansion, in float64.
    """
    w = _d(w)
    x = _d(x)
    g = _d(g)
    p, q, k = w.shape
    batch, n = x.shape
    assert n == q * k and g.shape == (batch, p * k)
    gx = np.empty((batch, n), dtype=np.float64) if want_gx else None
    gw = np.empty((p, q, k), dtype=np.float64) if want_gw else None
    _load().circ_oracle_fc_backward(ctypes.c_int(p * k), ctypes.c_int(n), ctypes.c_int(k), ctypes.c_int(convention),
                                    _ptr(w), _ptr(x), _ptr(g), ctypes.c_long(batch), _ptr(gx), _ptr(gw))
    return gx, gw


def conv(w, x, pad: int, bias=None, relu: bool = False, convention: int = 0, stride: int = 1) -> np.ndarray:
    """Eq. 6 with zero padding: ``w[r][r][p][q][k]``, ``x[N][H][W][C]`` -> ``y[N][Ho][Wo][P]``; ``stride`` > 1 keeps
    every stride-th output position of it in both directions."""
    w = _d(w)
    x = _d(x)
    r, r2, p, q, k = w.shape
    assert r == r2
    N, H, W, C = x.shape
    assert C == q * k
    if stride != 1:
        assert stride >= 1
        Ho, Wo = (H + 2 * pad - r) // stride + 1, (W + 2 * pad - r) // stride + 1
        b = None if bias is None else _d(bias)
        y = np.empty((N, Ho, Wo, p * k), dtype=np.float64)
        _load().circ_oracle_conv_strided(ctypes.c_int(p * k), ctypes.c_int(C), ctypes.c_int(r), ctypes.c_int(pad), ctypes.c_int(stride),
                                         ctypes.c_int(k), ctypes.c_int(convention), _ptr(w), _ptr(x), _ptr(b),
                                         ctypes.c_int(int(relu)), ctypes.c_int(N), ctypes.c_int(H), ctypes.c_int(W), _ptr(y))
        return y
    Ho, Wo = H + 2 * pad - r + 1, W + 2 * pad - r + 1
    b = None if bias is None else _d(bias)
    y = np.empty((N, Ho, Wo, p * k), dtype=np.float64)
    _load().circ_oracle_conv(ctypes.c_int(p * k), ctypes.c_int(C), ctypes.c_int(r), ctypes.c_int(pad),
                             ctypes.c_int(k), ctypes.c_int(convention), _ptr(w), _ptr(x), _ptr(b),
                             ctypes.c_int(int(relu)), ctypes.c_int(N), ctypes.c_int(H), ctypes.c_int(W), _ptr(y))
    return y


def conv_backward_input(w, g, pad: int, H: int, W: int, convention: int = 0) -> np.ndarray:
    """dL/dx of Eq. 6 from ``g = dL/dy`` (``[N][Ho][Wo][P]``): returns ``[N][H][W][C]``."""
    w = _d(w)
    g = _d(g)
    r, _, p, q, k = w.shape
    N, Ho, Wo, P = g.shape
    assert P == p * k and Ho == H + 2 * pad - r + 1 and Wo == W + 2 * pad - r + 1
    gx = np.empty((N, H, W, q * k), dtype=np.float64)
    _load().circ_oracle_conv_backward_input(ctypes.c_int(P), ctypes.c_int(q * k), ctypes.c_int(r), ctypes.c_int(pad),
                                            ctypes.c_int(k), ctypes.c_int(convention), _ptr(w), _ptr(g), ctypes.c_int(N),
                                            ctypes.c_int(H), ctypes.c_int(W), _ptr(gx))
    return gx


def conv_backward_weight(x, g, r: int, pad: int, k: int, convention: int = 0) -> np.ndarray:
    """dL/dw of Eq. 6 from ``x`` (``[N][H][W][C]``) and ``g = dL/dy`` (``[N][Ho][Wo][P]``): returns ``[r][r][p][q][k]``."""
    x = _d(x)
    g = _d(g)
    N, H, W, C = x.shape
    _, Ho, Wo, P = g.shape
    assert g.shape[0] == N and Ho == H + 2 * pad - r + 1 and Wo == W + 2 * pad - r + 1 and C % k == 0 and P % k == 0
    gw = np.empty((r, r, P // k, C // k, k), dtype=np.float64)
    _load().circ_oracle_conv_backward_weight(ctypes.c_int(P), ctypes.c_int(C), ctypes.c_int(r), ctypes.c_int(pad),
                                             ctypes.c_int(k), ctypes.c_int(convention), _ptr(x), _ptr(g), ctypes.c_int(N),
                                             ctypes.c_int(H), ctypes.c_int(W), _ptr(gw))
    return gw


def conv_pixels(w, x, pad: int, pixels, bias=None, relu: bool = False, convention: int = 0) -> np.ndarray:
    """Eq. 6 at the listed output pixels only: ``pixels[t] = (n, ho, wo)`` -> ``y[t][P]``."""
    w = _d(w)
    x = _d(x)
    r, _, p, q, k = w.shape
    N, H, W, C = x.shape
    pix = np.ascontiguousarray(pixels, dtype=np.int32).reshape(-1, 3)
    b = None if bias is None else _d(bias)
    y = np.empty((pix.shape[0], p * k), dtype=np.float64)
    _load().circ_oracle_conv_pixels(ctypes.c_int(p * k), ctypes.c_int(C), ctypes.c_int(r), ctypes.c_int(pad),
                                    ctypes.c_int(k), ctypes.c_int(convention), _ptr(w), _ptr(x), _ptr(b),
                                    ctypes.c_int(int(relu)), ctypes.c_int(N), ctypes.c_int(H), ctypes.c_int(W),
                                    ctypes.c_long(pix.shape[0]), pix.ctypes.data_as(_ip), _ptr(y))
    return y


POOL_MAX, POOL_AVG, POOL_L2 = 0, 1, 2


def pool(x, window: int, stride: int, mode: int = POOL_MAX) -> np.ndarray:
    """Pooling layer (Sec. 2.1): ``x[N][H][W][C]`` -> ``y[N][Ho][Wo][C]``, whole windows only, no padding."""
    x = _d(x)
    N, H, W, C = x.shape
    assert 1 <= window <= min(H, W) and stride >= 1 and mode in (POOL_MAX, POOL_AVG, POOL_L2)
    Ho, Wo = (H - window) // stride + 1, (W - window) // stride + 1
    y = np.empty((N, Ho, Wo, C), dtype=np.float64)
    _load().circ_oracle_pool(ctypes.c_int(mode), ctypes.c_int(window), ctypes.c_int(stride), ctypes.c_int(N), ctypes.c_int(H),
                             ctypes.c_int(W), ctypes.c_int(C), _ptr(x), _ptr(y))
    return y


def dft(re, im=None, sign: int = -1):
    """Naive O(k^2) DFT (``sign=-1`` forward, ``+1`` inverse, both unnormalised) -> (re, im)."""
    re = _d(re)
    imv = None if im is None else _d(im)
    k = re.shape[0]
    out_re = np.empty(k)
    out_im = np.empty(k)
    _load().circ_oracle_dft(ctypes.c_int(k), ctypes.c_int(sign), _ptr(re), _ptr(imv), _ptr(out_re), _ptr(out_im))
    return out_re, out_im
