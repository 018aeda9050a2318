"""CPU oracle for the BITCOS GEMV path -- TEST INFRASTRUCTURE, not product code.

Thin ctypes wrapper over ``bitcos_oracle.c`` (plain C, bit-at-a-time, written from the
paper).  Only the tests, the smoke check and the benchmark's CPU-baseline legs may import
this package; the CUDA library and its Python binding never do.

The shared object is built with ``gcc -O2 -fopenmp`` on first use if it is missing.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bitcos_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_bitcos.so")

GROUP = 128
ROWS = 32
FORMAT_BITCOS, FORMAT_TRIT5, FORMAT_BIT2 = 0, 1, 2


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u32p, i8p, u16p, u8p = (C.POINTER(C.c_uint32), C.POINTER(C.c_int8), C.POINTER(C.c_uint16),
                                C.POINTER(C.c_uint8))
        L.o_pdep32.restype = C.c_uint32
        L.o_pdep32.argtypes = [C.c_uint32, C.c_uint32]
        L.o_ternary_from_pn.restype = C.c_int
        L.o_ternary_from_pn.argtypes = [C.c_int, C.c_int]
        L.o_avx2_bytes.restype = None
        L.o_avx2_bytes.argtypes = [u8p, u8p, C.c_int, u8p, u8p, u8p]
        L.o_lut_entry.restype = C.c_int
        L.o_lut_entry.argtypes = [C.c_uint, C.c_uint, i8p]
        L.o_stream_pack.restype = C.c_int
        L.o_stream_pack.argtypes = [i8p, C.c_uint64, u32p, u32p, C.c_uint64, C.POINTER(C.c_uint64)]
        for name in ("o_stream_unpack",):
            f = getattr(L, name)
            f.restype = None
            f.argtypes = [u32p, C.c_uint64, C.c_uint64, u32p, C.c_uint64, i8p, C.POINTER(C.c_uint64)]
        for name in ("o_stream_unpack_windowed", "o_stream_unpack_lut"):
            f = getattr(L, name)
            f.restype = None
            f.argtypes = [u32p, C.c_uint64, C.c_uint64, u32p, C.c_uint64, i8p, C.POINTER(C.c_uint64)]
        L.o_padded_rows.restype = C.c_int64
        L.o_padded_rows.argtypes = [C.c_int64]
        L.o_num_tiles.restype = C.c_int64
        L.o_num_tiles.argtypes = [C.c_int64, C.c_int64]
        L.o_tile_order_pos.restype = C.c_uint64
        L.o_tile_order_pos.argtypes = [C.c_int64] * 4
        L.o_sign_words.restype = C.c_uint64
        L.o_sign_words.argtypes = [C.c_uint64]
        L.o_count_nnz.restype = C.c_uint64
        L.o_count_nnz.argtypes = [i8p, C.c_int64, C.c_int64]
        L.o_bitcos_pack.restype = C.c_int
        L.o_bitcos_pack.argtypes = [i8p, C.c_int64, C.c_int64, u32p, u32p, C.c_uint64, u32p,
                                    C.POINTER(C.c_uint64)]
        L.o_bitcos_unpack.restype = C.c_int
        L.o_bitcos_unpack.argtypes = [u32p, u32p, u32p, C.c_int64, C.c_int64, C.c_int, i8p]
        L.o_scales_to_tile_order.restype = None
        L.o_scales_to_tile_order.argtypes = [u16p, C.c_int64, C.c_int64, u16p]
        L.o_trit5_block_encode.restype = None
        L.o_trit5_block_encode.argtypes = [i8p, u8p]
        L.o_trit5_block_decode.restype = C.c_int
        L.o_trit5_block_decode.argtypes = [u8p, i8p]
        L.o_trit5_words_per_row.restype = C.c_int64
        L.o_trit5_words_per_row.argtypes = [C.c_int64]
        L.o_trit5_total_words.restype = C.c_int64
        L.o_trit5_total_words.argtypes = [C.c_int64, C.c_int64]
        L.o_trit5_pack.restype = C.c_int
        L.o_trit5_pack.argtypes = [i8p, C.c_int64, C.c_int64, u32p]
        L.o_trit5_unpack.restype = C.c_int
        L.o_trit5_unpack.argtypes = [u32p, C.c_int64, C.c_int64, i8p]
        L.o_bit2_total_words.restype = C.c_int64
        L.o_bit2_total_words.argtypes = [C.c_int64, C.c_int64]
        L.o_bit2_pack.restype = C.c_int
        L.o_bit2_pack.argtypes = [i8p, C.c_int64, C.c_int64, u32p]
        L.o_bit2_unpack.restype = C.c_int
        L.o_bit2_unpack.argtypes = [u32p, C.c_int64, C.c_int64, i8p]
        L.o_dense_acc.restype = None
        L.o_dense_acc.argtypes = [i8p, i8p, C.c_int64, C.c_int64, C.c_int64, C.POINTER(C.c_int32)]
        L.o_dense_y.restype = None
        L.o_dense_y.argtypes = [C.POINTER(C.c_int32), u16p, C.POINTER(C.c_float), C.c_int64, C.c_int64,
                                C.c_int64, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.o_gemv_packed.restype = C.c_int
        L.o_gemv_packed.argtypes = [C.c_int, u32p, u32p, u32p, u16p, i8p, C.POINTER(C.c_float), C.c_int64,
                                    C.c_int64, C.c_int64, C.POINTER(C.c_int32), C.POINTER(C.c_double),
                                    C.POINTER(C.c_double)]
        L.o_threads.restype = C.c_int
        L.o_threads.argtypes = []
        L.o_set_threads.restype = None
        L.o_set_threads.argtypes = [C.c_int]
        _lib = L
    return _lib


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(C.POINTER(ty))


def _i8(a):
    a = np.ascontiguousarray(a, dtype=np.int8)
    return a, _p(a, C.c_int8)


class OracleError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != 0:
        raise OracleError(f"{what}: oracle status {rc}")


# --- primitives --------------------------------------------------------------------
def pdep32(a: int, mask: int) -> int:
    return int(lib().o_pdep32(a & 0xFFFFFFFF, mask & 0xFFFFFFFF))


def ternary_from_pn(p: int, n: int) -> int:
    return int(lib().o_ternary_from_pn(p, n))


def avx2_bytes(p, n):
    p = np.ascontiguousarray(p, dtype=np.uint8)
    n = np.ascontiguousarray(n, dtype=np.uint8)
    P, T, W = (np.zeros(len(p), np.uint8) for _ in range(3))
    lib().o_avx2_bytes(_p(p, C.c_uint8), _p(n, C.c_uint8), len(p), _p(P, C.c_uint8), _p(T, C.c_uint8),
                       _p(W, C.c_uint8))
    return P, T, W


def lut_entry(m: int, s: int):
    c = np.zeros(4, np.int8)
    used = lib().o_lut_entry(m, s, _p(c, C.c_int8))
    return c, int(used)


def sign_words(nnz: int) -> int:
    return int(lib().o_sign_words(nnz))


def stream_pack(sym):
    sym, ps = _i8(np.asarray(sym).ravel())
    n = sym.size
    nnz_guess = int(np.count_nonzero(sym))
    sw = sign_words(nnz_guess)
    bitmap = np.zeros((n + 31) // 32, np.uint32)
    signs = np.zeros(sw, np.uint32)
    nnz = C.c_uint64(0)
    _check(lib().o_stream_pack(ps, n, _p(bitmap, C.c_uint32), _p(signs, C.c_uint32), sw, C.byref(nnz)),
           "stream_pack")
    return bitmap, signs, int(nnz.value)


def stream_unpack(bitmap, signs, n, decoder="bits", start_sign_bit=0):
    bitmap = np.ascontiguousarray(bitmap, np.uint32)
    signs = np.ascontiguousarray(signs, np.uint32)
    out = np.zeros((n + 31) // 32 * 32, np.int8)
    end = C.c_uint64(0)
    L = lib()
    if decoder == "bits":
        L.o_stream_unpack(_p(bitmap, C.c_uint32), 0, n, _p(signs, C.c_uint32), start_sign_bit,
                          _p(out, C.c_int8), C.byref(end))
    else:
        f = L.o_stream_unpack_windowed if decoder == "pdep" else L.o_stream_unpack_lut
        f(_p(bitmap, C.c_uint32), 0, (n + 31) // 32, _p(signs, C.c_uint32), start_sign_bit,
          _p(out, C.c_int8), C.byref(end))
    return out[:n], int(end.value)


# --- matrix layouts ------------------------------------------------------------------
def padded_rows(M: int) -> int:
    return int(lib().o_padded_rows(M))


def num_tiles(M: int, K: int) -> int:
    return int(lib().o_num_tiles(M, K))


def tile_order_pos(M, K, m, k) -> int:
    return int(lib().o_tile_order_pos(M, K, m, k))


class BitcosPacked:
    def __init__(self, M, K, bitmap, signs, tile_off, nnz):
        self.M, self.K, self.bitmap, self.signs, self.tile_off, self.nnz = M, K, bitmap, signs, tile_off, nnz

    def bits_per_weight(self):
        """Presence bits plus sign bits per stored weight (Eq. 1), slack and offsets excluded."""
        return (self.bitmap.size * 32 + self.nnz) / (padded_rows(self.M) * self.K)


def bitcos_pack(trits) -> BitcosPacked:
    t, pt = _i8(trits)
    M, K = t.shape
    L = lib()
    nnz = int(L.o_count_nnz(pt, M, K))
    sw = sign_words(nnz)
    bitmap = np.zeros(padded_rows(M) * K // 32, np.uint32)
    signs = np.zeros(sw, np.uint32)
    tile_off = np.zeros(num_tiles(M, K) + 1, np.uint32)
    out = C.c_uint64(0)
    _check(L.o_bitcos_pack(pt, M, K, _p(bitmap, C.c_uint32), _p(signs, C.c_uint32), sw,
                           _p(tile_off, C.c_uint32), C.byref(out)), "bitcos_pack")
    return BitcosPacked(M, K, bitmap, signs, tile_off, int(out.value))


_DECODERS = {"bits": 0, "pdep": 1, "lut": 2, "tiles": 3}


def bitcos_unpack(bitmap, signs, tile_off, M, K, decoder="bits") -> np.ndarray:
    bitmap = np.ascontiguousarray(bitmap, np.uint32)
    signs = np.ascontiguousarray(signs, np.uint32)
    tile_off = np.ascontiguousarray(tile_off, np.uint32)
    out = np.zeros((M, K), np.int8)
    _check(lib().o_bitcos_unpack(_p(bitmap, C.c_uint32), _p(signs, C.c_uint32), _p(tile_off, C.c_uint32),
                                 M, K, _DECODERS[decoder], _p(out, C.c_int8)), "bitcos_unpack")
    return out


def scales_to_tile_order(scales, M, K) -> np.ndarray:
    s = np.ascontiguousarray(scales, np.uint16)
    out = np.zeros(padded_rows(M) * (K // GROUP), np.uint16)
    lib().o_scales_to_tile_order(_p(s, C.c_uint16), M, K, _p(out, C.c_uint16))
    return out


def trit5_block_encode(t128) -> np.ndarray:
    t, pt = _i8(t128)
    out = np.zeros(26, np.uint8)
    lib().o_trit5_block_encode(pt, _p(out, C.c_uint8))
    return out


def trit5_block_decode(b26) -> np.ndarray:
    b = np.ascontiguousarray(b26, np.uint8)
    out = np.zeros(128, np.int8)
    _check(lib().o_trit5_block_decode(_p(b, C.c_uint8), _p(out, C.c_int8)), "trit5_block_decode")
    return out


def trit5_pack(trits) -> np.ndarray:
    t, pt = _i8(trits)
    M, K = t.shape
    words = np.zeros(int(lib().o_trit5_total_words(M, K)), np.uint32)
    _check(lib().o_trit5_pack(pt, M, K, _p(words, C.c_uint32)), "trit5_pack")
    return words


def trit5_unpack(words, M, K) -> np.ndarray:
    w = np.ascontiguousarray(words, np.uint32)
    out = np.zeros((M, K), np.int8)
    _check(lib().o_trit5_unpack(_p(w, C.c_uint32), M, K, _p(out, C.c_int8)), "trit5_unpack")
    return out


def bit2_pack(trits) -> np.ndarray:
    t, pt = _i8(trits)
    M, K = t.shape
    words = np.zeros(int(lib().o_bit2_total_words(M, K)), np.uint32)
    _check(lib().o_bit2_pack(pt, M, K, _p(words, C.c_uint32)), "bit2_pack")
    return words


def bit2_unpack(words, M, K) -> np.ndarray:
    w = np.ascontiguousarray(words, np.uint32)
    out = np.zeros((M, K), np.int8)
    _check(lib().o_bit2_unpack(_p(w, C.c_uint32), M, K, _p(out, C.c_int8)), "bit2_unpack")
    return out


# --- the product -----------------------------------------------------------------------
def dense_acc(W, x) -> np.ndarray:
    W, pW = _i8(W)
    x, px = _i8(np.atleast_2d(x))
    M, K = W.shape
    B = x.shape[0]
    acc = np.zeros((B, M, K // GROUP), np.int32)
    lib().o_dense_acc(pW, px, M, K, B, _p(acc, C.c_int32))
    return acc


def dense_y(acc, scales, xs, K):
    acc = np.ascontiguousarray(acc, np.int32)
    B, M, G = acc.shape
    s = np.ascontiguousarray(scales, np.uint16).reshape(M, G)
    xs = np.ascontiguousarray(xs, np.float32)
    y = np.zeros((B, M), np.float64)
    mag = np.zeros((B, M), np.float64)
    lib().o_dense_y(_p(acc, C.c_int32), _p(s, C.c_uint16), _p(xs, C.c_float), M, K, B,
                    _p(y, C.c_double), _p(mag, C.c_double))
    return y, mag


def gemv_dense(W, scales, x, xs):
    """Reference result from dense trits: (acc int32 [B,M,G], y float64 [B,M], mag [B,M])."""
    acc = dense_acc(W, x)
    y, mag = dense_y(acc, scales, xs, np.asarray(W).shape[1])
    return acc, y, mag


def gemv_packed(fmt: int, payload, signs, tile_off, scales, x, xs, M, K):
    """Decode the packed matrix, then the dense definition. scales are [M, G] row major."""
    payload = np.ascontiguousarray(payload, np.uint32)
    signs = np.ascontiguousarray(signs if signs is not None else np.zeros(1, np.uint32), np.uint32)
    tile_off = np.ascontiguousarray(tile_off if tile_off is not None else np.zeros(1, np.uint32), np.uint32)
    s = np.ascontiguousarray(scales, np.uint16)
    x, px = _i8(np.atleast_2d(x))
    xs = np.ascontiguousarray(xs, np.float32)
    B = x.shape[0]
    G = K // GROUP
    acc = np.zeros((B, M, G), np.int32)
    y = np.zeros((B, M), np.float64)
    mag = np.zeros((B, M), np.float64)
    _check(lib().o_gemv_packed(fmt, _p(payload, C.c_uint32), _p(signs, C.c_uint32), _p(tile_off, C.c_uint32),
                               _p(s, C.c_uint16), px, _p(xs, C.c_float), M, K, B, _p(acc, C.c_int32),
                               _p(y, C.c_double), _p(mag, C.c_double)), "gemv_packed")
    return acc, y, mag


def grouped_dense(expert_W, expert_scales, pair_expert, pair_xrow, x, xs):
    """Grouped (mixture-of-experts) product: pair p multiplies expert pair_expert[p]'s matrix
    with activation row pair_xrow[p]; no activation function, routing weight or sum over
    experts.  Returns lists (acc, y, mag), one entry per pair."""
    accs, ys, mags = [], [], []
    for e, r in zip(pair_expert, pair_xrow):
        a, y, m = gemv_dense(expert_W[e], expert_scales[e], x[r:r + 1], xs[r:r + 1])
        accs.append(a[0]); ys.append(y[0]); mags.append(m[0])
    return np.stack(accs), np.stack(ys), np.stack(mags)


# --- activations quantised per group of 128 (Section II-C: the integer contraction) ---------------
AMAX_FLOOR = np.float32(2.0 ** -100)


def quantize_activations(x, group: int = GROUP):
    """16- or 32-bit float activations [B, K] -> (int8 codes [B, K], float32 scales).

    Section II-C only says that the integer path quantises the activations to int8 per group
    of 128 and applies the scales once per group; the rule below is this build's reading of it
    (symmetric absmax quantisation), taken in float32, the precision the kernel decides in:

        a     = max(max |x| over the group, 2^-100)        (the floor keeps 127 / a finite)
        scale = a / 127                                     (float32, round to nearest)
        code  = rint(x * (127 / a))                         (float32 quotient and product, ties to even)

    so that x ~ scale * code with |code| <= 127.  `group` = 128 gives scales [B, K / 128];
    `group` = 0 takes the whole row as one group (one scale per token, [B]).
    """
    x = np.atleast_2d(np.asarray(x, dtype=np.float32))
    B, K = x.shape
    gs = K if group == 0 else group
    if gs < 1 or K % gs:
        raise ValueError("K must be a multiple of the group size")
    xg = x.reshape(B, K // gs, gs)
    a = np.maximum(np.abs(xg).max(axis=2), AMAX_FLOOR).astype(np.float32)
    scale = (a / np.float32(127.0)).astype(np.float32)
    inv = (np.float32(127.0) / a).astype(np.float32)
    prod = (xg * inv[:, :, None]).astype(np.float32)
    code = np.clip(np.rint(prod), -127, 127).astype(np.int8).reshape(B, K)
    return code, (scale.reshape(B) if group == 0 else scale)


def dense_y_group_scales(acc, scales, xs_g):
    """y[b, m] = sum over groups g of  s[m, g] * xs_g[b, g] * acc[b, m, g]   in float64
    (Section II-C: int32 group sums, weight and activation scale applied once per group);
    also the sum of the absolute values of the terms, for the tolerance."""
    acc = np.asarray(acc, np.int64)
    B, M, G = acc.shape
    s = (np.asarray(scales, np.uint16).reshape(M, G).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    xs_g = np.asarray(xs_g, np.float32).reshape(B, G).astype(np.float64)
    terms = acc.astype(np.float64) * s[None, :, :] * xs_g[:, None, :]
    return terms.sum(axis=2), np.abs(terms).sum(axis=2)


def gemv_dense_group_scales(W, scales, x, xs_g):
    """Dense definition with one activation scale per token and group: (acc, y, mag)."""
    acc = dense_acc(W, x)
    y, mag = dense_y_group_scales(acc, scales, xs_g)
    return acc, y, mag


# --- unquantised 16-bit activations against weights +-s (Sections II-B and II-D: the scale blended
# --- into the reconstructed weight, multiply-add against 16-bit activations) -----------------------
def gemv_dense_blend(W, scales, x):
    """y[b, m] = sum over k of (W[m, k] * s[m, k // 128]) * x[b, k] in float64, x = float values of
    16-bit activations [B, K] (no quantisation anywhere); also the sum of |terms| for the tolerance."""
    W = np.asarray(W, np.int8)
    M, K = W.shape
    G = K // GROUP
    s = (np.asarray(scales, np.uint16).reshape(M, G).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    x = np.atleast_2d(np.asarray(x, np.float64))
    B = x.shape[0]
    y = np.zeros((B, M), np.float64)
    mag = np.zeros((B, M), np.float64)
    for m in range(M):
        ws = W[m].astype(np.float64) * np.repeat(s[m], GROUP)          # the row's weights +-s (or 0)
        terms = x * ws[None, :]
        y[:, m] = terms.sum(axis=1)
        mag[:, m] = np.abs(terms).sum(axis=1)
    return y, mag


def threads() -> int:
    return int(lib().o_threads())


def set_threads(n: int) -> None:
    """Timing aid: the number of host threads the oracle's loops may use from now on."""
    lib().o_set_threads(int(n))
