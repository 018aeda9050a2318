"""Seeded synthetic inputs for the BITCOS GEMV path.

This module only draws inputs.  It holds none of the method's arithmetic: no packing,
no decoding, no dot product.  Both the CPU oracle's tests and the CUDA path's tests and
benchmarks take their trits, scales and activations from here, so that the two sides
always see the same bytes.

Generator: counter based.  Element `i` of stream `s` under seed `seed` is

    z = mix64((seed XOR s * 0xD1B54A32D192ED03) + (i + 1) * 0x9E3779B97F4A7C15)   (mod 2^64)
    u = (z >> 11) * 2^-53                                                   in [0, 1)

with `mix64` the splitmix64 output function.  Any element can be produced on its own,
in any order, on any machine.

Workload shapes follow the five configurations of the benchmark definition: ternary
symbols are i.i.d. with P(0) = z and P(+1) = P(-1) = (1 - z) / 2, one bf16 scale per
group of 128 reduction elements drawn from U[0.01, 0.05], int8 activations uniform in
[-127, 127] with one positive fp32 scale per token.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

GROUP = 128

STREAM_TRITS = 0
STREAM_SCALES = 1
STREAM_X = 2
STREAM_XS = 3
STREAM_EXPERTS = 4
STREAM_XF = 5

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_STREAM_MUL = np.uint64(0xD1B54A32D192ED03)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix64(z: np.ndarray) -> np.ndarray:
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def uniform(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """float64 uniforms in [0, 1) for counter values start .. start + count - 1."""
    with np.errstate(over="ignore"):
        base = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) ^ (np.uint64(stream) * _STREAM_MUL)
        idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        z = _mix64(base + idx * _GOLD)
    return (z >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def _chunks(total: int, step: int = 1 << 24):
    pos = 0
    while pos < total:
        n = min(step, total - pos)
        yield pos, n
        pos += n


_HERE = os.path.dirname(os.path.abspath(__file__))
_FILL_SRC = os.path.join(_HERE, "datagen_fill.c")
_FILL_LIB = os.path.join(_HERE, "libdatagen_fill.so")
_fill = None


def build_native(force: bool = False) -> str:
    """Compiles the native filler for large tensors (gcc); returns the library's path."""
    if force or not os.path.exists(_FILL_LIB) or os.path.getmtime(_FILL_LIB) < os.path.getmtime(_FILL_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _FILL_LIB, _FILL_SRC])
    return _FILL_LIB


def _native_fill():
    """The native filler, or None if it cannot be built here (the numpy formulation then serves)."""
    global _fill
    if _fill is None:
        try:
            L = C.CDLL(build_native())
            L.datagen_fill_trits.restype = None
            L.datagen_fill_trits.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint64, C.c_double, C.c_void_p]
            _fill = L
        except (OSError, subprocess.CalledProcessError):
            _fill = False
    return _fill or None


def trits(seed: int, M: int, K: int, z: float, native: bool = True) -> np.ndarray:
    """int8 [M, K] with values in {-1, 0, +1}: 0 with probability z, else +-1 evenly.  Large
    tensors are filled by the native helper (the same values, bit for bit)."""
    out = np.empty(M * K, dtype=np.int8)
    L = _native_fill() if (native and M * K >= (1 << 16)) else None
    if L is not None:
        L.datagen_fill_trits(seed & 0xFFFFFFFFFFFFFFFF, STREAM_TRITS, 0, M * K, float(z), out.ctypes.data)
        return out.reshape(M, K)
    half = z + (1.0 - z) / 2.0
    for pos, n in _chunks(M * K):
        u = uniform(seed, STREAM_TRITS, pos, n)
        t = np.where(u < z, 0, np.where(u < half, 1, -1)).astype(np.int8)
        out[pos:pos + n] = t
    return out.reshape(M, K)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of finite float32 values to bf16 bit patterns."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))
    return (rounded >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def scales(seed: int, M: int, K: int, lo: float = 0.01, hi: float = 0.05) -> np.ndarray:
    """uint16 [M, K / 128]: bf16 bit patterns of scales drawn from U[lo, hi]."""
    G = K // GROUP
    u = uniform(seed, STREAM_SCALES, 0, M * G)
    return f32_to_bf16_bits((lo + (hi - lo) * u).astype(np.float32)).reshape(M, G)


def activations(seed: int, B: int, K: int) -> tuple[np.ndarray, np.ndarray]:
    """(x int8 [B, K] uniform in [-127, 127], xs float32 [B] positive per-token scale)."""
    u = uniform(seed, STREAM_X, 0, B * K)
    x = (np.floor(255.0 * u) - 127.0).astype(np.int8).reshape(B, K)
    a = 1.0 + 3.0 * uniform(seed, STREAM_XS, 0, B)
    xs = (a / 127.0).astype(np.float32)
    return x, xs


def activations_bf16(seed: int, B: int, K: int, outlier_every: int = 97, outlier_gain: float = 24.0) -> np.ndarray:
    """uint16 [B, K]: bf16 bit patterns of unquantised activations, roughly normal (a sum of
    four uniforms, variance 1) with every `outlier_every`-th channel scaled up, the shape
    transformer activations have (a few channels carry most of the range)."""
    u = uniform(seed, STREAM_XF, 0, 4 * B * K).reshape(B * K, 4)
    v = (u.sum(axis=1) - 2.0) * np.sqrt(3.0)
    v = v.reshape(B, K)
    gain = np.where(np.arange(K) % outlier_every == outlier_every // 2, outlier_gain, 1.0)
    return f32_to_bf16_bits((v * gain[None, :]).astype(np.float32))


def expert_choices(seed: int, tokens: int, n_experts: int, top_k: int) -> np.ndarray:
    """int32 [tokens, top_k]: per token, top_k distinct expert ids drawn uniformly."""
    out = np.empty((tokens, top_k), dtype=np.int32)
    for t in range(tokens):
        u = uniform(seed, STREAM_EXPERTS, t * n_experts, n_experts)
        out[t] = np.sort(np.argsort(u, kind="stable")[:top_k]).astype(np.int32)
    return out


# ---------------------------------------------------------------------------------
# The five benchmark configurations (shapes and zero densities only).
# ---------------------------------------------------------------------------------
BASE_SEED = 20260916

CONFIG_TINY = {"name": "tiny", "z": 0.42, "shapes": [("w", 256, 512)], "batches": [1]}

CONFIG_BITNET_2B = {
    "name": "bitnet-b1.58-2B layer",
    "z": 0.4219,
    "shapes": [("q", 2560, 2560), ("k", 640, 2560), ("v", 640, 2560), ("o", 2560, 2560),
               ("gate", 6912, 2560), ("up", 6912, 2560), ("down", 2560, 6912)],
    "batches": [1],
}

CONFIG_SWEEP = {
    "name": "zero-density sweep",
    "zs": [0.30, 0.375, 0.42, 0.47, 0.515],
    "shapes": [("wide", 4096, 12288), ("tall", 12288, 4096)],
    "batches": [1],
}

CONFIG_QWEN3_32B = {
    "name": "qwen3-32B layer",
    "z": 0.4711,
    "shapes": [("q", 8192, 5120), ("k", 1024, 5120), ("v", 1024, 5120), ("o", 5120, 8192),
               ("gate", 25600, 5120), ("up", 25600, 5120), ("down", 5120, 25600)],
    "batches": [1, 2, 4, 8, 16],
}

CONFIG_QWEN3_MOE = {
    "name": "qwen3-30B-A3B experts",
    "z": 0.3288,
    "n_experts": 128,
    "top_k": 8,
    "shapes": [("gate", 768, 2048), ("up", 768, 2048), ("down", 2048, 768)],
    "batches": [1, 2, 4, 8, 16],
}


def config_seed(config_index: int, tensor_index: int) -> int:
    return BASE_SEED + 1000 * config_index + tensor_index
