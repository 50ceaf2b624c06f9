"""Seeded synthetic inputs for block-circulant layers.

This module only draws numbers and rounds them to storage precision.  It holds
none of the layer arithmetic (no circulant expansion, no transforms), so both
the CUDA path and the CPU oracle can be fed from it without sharing any of the
method between them.

Generator: a counter-based stream.  Element ``i`` of stream ``s`` is
``splitmix64(base + s * GOLDEN + i)`` mapped to a uniform in (0, 1); normals
come from the Box-Muller formula evaluated in float64 on two such uniforms.
Every value is then rounded to float32 (and optionally to bfloat16, round to
nearest even) because that is what the device buffers hold; the oracle
receives exactly those rounded values widened to float64.

Distributions follow the workload table of the block-circulant benchmark
configurations: N(0, v) takes the *variance* as second argument.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 170808917
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """The splitmix64 output function applied elementwise to uint64 counters."""
    with np.errstate(over="ignore"):
        z = (z + _GOLDEN).astype(np.uint64)
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def stream_id(config: str, tensor: str) -> int:
    """Stable 32-bit id of a (configuration, tensor name) pair."""
    return zlib.crc32(f"{config}/{tensor}".encode()) & 0xFFFFFFFF


def _uniform01(count: int, stream: int, offset: int = 0, seed: int = BASE_SEED) -> np.ndarray:
    """``count`` float64 uniforms in the open interval (0, 1)."""
    with np.errstate(over="ignore"):
        base = np.uint64(seed) * np.uint64(0x100000001B3) + np.uint64(stream) * _GOLDEN
        ctr = base + np.arange(offset, offset + count, dtype=np.uint64)
    bits = _splitmix64(ctr) >> np.uint64(11)            # 53 random bits
    return (bits.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def uniform(shape, lo: float, hi: float, stream: int, seed: int = BASE_SEED) -> np.ndarray:
    """float32 array of U(lo, hi) draws."""
    count = int(np.prod(shape))
    u = _uniform01(count, stream, 0, seed)
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(shape, variance: float, stream: int, seed: int = BASE_SEED, absolute: bool = False) -> np.ndarray:
    """float32 array of N(0, variance) draws (|N| when ``absolute``)."""
    count = int(np.prod(shape))
    half = (count + 1) // 2
    u1 = _uniform01(half, stream, 0, seed)
    u2 = _uniform01(half, stream, half, seed)
    rad = np.sqrt(-2.0 * np.log(u1))
    z = np.concatenate([rad * np.cos(2.0 * np.pi * u2), rad * np.sin(2.0 * np.pi * u2)])[:count]
    z = z * np.sqrt(variance)
    if absolute:
        z = np.abs(z)
    return z.astype(np.float32).reshape(shape)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    with np.errstate(over="ignore"):
        rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """The uint16 storage pattern of float32 values that are already bfloat16-representable."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    return (bits >> np.uint32(16)).astype(np.uint16).reshape(a.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen uint16 bfloat16 patterns to float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(b.shape)


@dataclass
class FcCase:
    """One fully-connected block-circulant problem: weights ``w[p][q][k]``, inputs ``x[B][n]``."""
    name: str
    m: int
    n: int
    k: int
    batch: int
    w: np.ndarray
    x: np.ndarray
    bias: np.ndarray | None = None
    relu: bool = False
    bf16_io: bool = False
    extra: dict = field(default_factory=dict)


@dataclass
class ConvCase:
    """One block-circulant convolution: weights ``w[r][r][p][q][k]``, input ``x[N][H][W][C]`` (channel last)."""
    name: str
    c_out: int
    c_in: int
    r: int
    pad: int
    k: int
    N: int
    H: int
    W: int
    w: np.ndarray
    x: np.ndarray
    bias: np.ndarray | None = None
    relu: bool = False
    bf16_io: bool = True


def fc_case(name: str, m: int, n: int, k: int, batch: int, *, w_var: float, x_dist: str,
            bias_var: float | None = None, relu: bool = False, bf16_io: bool = False,
            seed: int = BASE_SEED) -> FcCase:
    """Draw one FC problem.  ``x_dist`` is 'normal', 'uniform' (U(-1,1)) or 'absnormal' (|N(0,1)|)."""
    p, q = m // k, n // k
    w = normal((p, q, k), w_var, stream_id(name, "w"), seed)
    if x_dist == "normal":
        x = normal((batch, n), 1.0, stream_id(name, "x"), seed)
    elif x_dist == "uniform":
        x = uniform((batch, n), -1.0, 1.0, stream_id(name, "x"), seed)
    elif x_dist == "absnormal":
        x = normal((batch, n), 1.0, stream_id(name, "x"), seed, absolute=True)
    else:
        raise ValueError(x_dist)
    bias = None if bias_var is None else normal((m,), bias_var, stream_id(name, "bias"), seed)
    if bf16_io:
        x = round_to_bf16(x)
    return FcCase(name, m, n, k, batch, w, x, bias, relu, bf16_io)


def conv_case(name: str, c_out: int, c_in: int, r: int, pad: int, k: int, N: int, H: int, W: int, *,
              w_var: float, bf16_io: bool = True, bias_var: float | None = None, relu: bool = False,
              seed: int = BASE_SEED) -> ConvCase:
    """Draw one CONV problem with |N(0,1)| activations."""
    p, q = c_out // k, c_in // k
    w = normal((r, r, p, q, k), w_var, stream_id(name, "w"), seed)
    x = normal((N, H, W, c_in), 1.0, stream_id(name, "x"), seed, absolute=True)
    bias = None if bias_var is None else normal((c_out,), bias_var, stream_id(name, "bias"), seed)
    if bf16_io:
        x = round_to_bf16(x)
    return ConvCase(name, c_out, c_in, r, pad, k, N, H, W, w, x, bias, relu, bf16_io)


# ---- the benchmark configurations (shapes and distributions only) -------------------------------

def config1() -> FcCase:
    """256x256, k=16, batch 1, N(0,1) weights and inputs, no bias, no activation."""
    return fc_case("cfg1", 256, 256, 16, 1, w_var=1.0, x_dist="normal")


def config2(batch: int) -> FcCase:
    """4096x4096, k=64, weights N(0,1/4096), inputs U(-1,1), bias N(0,0.01), ReLU."""
    return fc_case(f"cfg2_b{batch}", 4096, 4096, 64, batch, w_var=1.0 / 4096, x_dist="uniform",
                   bias_var=0.01, relu=True)


def config3_layers(batch: int = 128) -> list[FcCase]:
    """9216->4096->4096->1024 stack, k=128; only the first case carries a drawn input."""
    dims = [(4096, 9216), (4096, 4096), (1024, 4096)]
    out = []
    for li, (m, n) in enumerate(dims):
        c = fc_case(f"cfg3_l{li}", m, n, 128, batch if li == 0 else 1, w_var=1.0 / n,
                    x_dist="absnormal", relu=(li < 2))
        c.batch = batch
        out.append(c)
    return out


def config4(N: int = 32, H: int = 28, W: int = 28) -> ConvCase:
    """3x3, stride 1, pad 1, 256->256 channels, k=16, bf16 activations."""
    return conv_case(f"cfg4_n{N}_h{H}_w{W}", 256, 256, 3, 1, 16, N, H, W, w_var=1.0 / (9 * 256))


def sweep_point(n: int, k: int, batch: int, bf16_io: bool) -> FcCase:
    """Square layer of the sweep: weights N(0,1/n), inputs U(-1,1)."""
    return fc_case(f"sweep_n{n}_k{k}_b{batch}_{'bf16' if bf16_io else 'f32'}", n, n, k, batch,
                   w_var=1.0 / n, x_dist="uniform", bf16_io=bf16_io)


SWEEP_N = (1024, 4096, 16384)
SWEEP_K = (4, 16, 64, 256)
SWEEP_B = (1, 64, 1024)
