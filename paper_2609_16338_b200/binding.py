"""ctypes binding of libbitcos.so: same names as the C ABI, argument marshalling only.

Host packers take and return numpy arrays.  Device entry points take torch CUDA tensors
(used here only as owners of device memory) and enqueue on torch's current stream.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

GROUP = 128
TILE_ROWS = 32
MAX_BATCH = 16

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbitcos.so")

EXPORTED_SYMBOLS = [
    "bitcos_status_string", "bitcos_last_cuda_error", "bitcos_pack_sizes", "bitcos_count_nnz", "bitcos_pack",
    "bitcos_unpack", "bitcos_scales_tile", "bitcos_scales_untile", "trit5_pack_sizes", "trit5_pack",
    "trit5_unpack", "bit2_pack_sizes", "bit2_pack", "bit2_unpack", "bitcos_gemv_workspace_bytes",
    "bitcos_workspace_init", "bitcos_workspace_status", "bitcos_gemv", "trit5_gemv", "bit2_gemv", "bitcos_gemv_grouped",
    "bitcos_gemv_host_staging_bytes", "bitcos_gemv_host", "bitcos_gemv_static", "bitcos_decode_probe", "bitcos_gemv_multi",
    "bitcos_gemv_multi_host", "bitcos_quantize_activations", "bitcos_gemv_group_scales",
    "bitcos_choose_format", "bitcos_count_nnz_device", "bitcos_pack_device", "bitcos_gemv_bf16", "bitcos_gemv_multi_bf16",
    "bitcos_gemv_multi_group_scales", "bitcos_gemv_blend_bf16", "bitcos_decode_probe_variant", "bitcos_gemv_phased", "bitcos_gemv_phases_host", "trit5_gemv_grouped", "bit2_gemv_grouped", "bitcos_gemv_static_status", "bitcos_wait_probe", "bitcos_group_pairs_device", "bitcos_gemv_grouped_lists", "bitcos_gemv_multi_chained", "bitcos_gemv_multi_plan",
]


class BitcosError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        super().__init__(f"{what}: status {status} ({detail})")


class _Job(C.Structure):
    _fields_ = [("W", C.c_void_p), ("x", C.c_void_p), ("x_scale", C.c_void_p), ("y", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class _HostJob(C.Structure):
    _fields_ = [("W", C.c_void_p), ("x_host", C.c_void_p), ("x_scale_host", C.c_void_p), ("y_host", C.c_void_p),
                ("staging", C.c_void_p), ("staging_bytes", C.c_size_t), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t)]


class _Weights(C.Structure):
    _fields_ = [("bitmap", C.c_void_p), ("signs", C.c_void_p), ("tile_off", C.c_void_p), ("scales", C.c_void_p),
                ("M", C.c_int64), ("K", C.c_int64), ("tile_off_host", C.c_void_p)]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libbitcos.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise BitcosError(-1, "load_library", f"{_LIB_PATH} is missing: run `python -m paper_2609_16338_b200.build`")
    L = C.CDLL(_LIB_PATH)
    vp, i64, sz, u64 = C.c_void_p, C.c_int64, C.c_size_t, C.c_uint64
    psz = C.POINTER(C.c_size_t)
    L.bitcos_status_string.restype = C.c_char_p
    L.bitcos_status_string.argtypes = [C.c_int]
    L.bitcos_last_cuda_error.restype = C.c_int
    L.bitcos_last_cuda_error.argtypes = []
    L.bitcos_pack_sizes.argtypes = [i64, i64, u64, psz, psz, psz, psz]
    L.bitcos_count_nnz.argtypes = [vp, i64, i64, C.POINTER(u64)]
    L.bitcos_pack.argtypes = [vp, vp, i64, i64, vp, vp, sz, vp, vp, C.POINTER(u64)]
    L.bitcos_unpack.argtypes = [vp, vp, vp, i64, i64, vp]
    L.bitcos_scales_tile.argtypes = [vp, i64, i64, vp]
    L.bitcos_scales_untile.argtypes = [vp, i64, i64, vp]
    for name in ("trit5", "bit2"):
        getattr(L, name + "_pack_sizes").argtypes = [i64, i64, psz]
        getattr(L, name + "_pack").argtypes = [vp, i64, i64, vp]
        getattr(L, name + "_unpack").argtypes = [vp, i64, i64, vp]
    L.bitcos_gemv_workspace_bytes.restype = sz
    L.bitcos_gemv_workspace_bytes.argtypes = [i64, i64]
    L.bitcos_workspace_init.argtypes = [vp, sz, vp]
    L.bitcos_workspace_status.argtypes = [vp, vp, C.POINTER(C.c_int)]
    L.bitcos_gemv.argtypes = [C.POINTER(_Weights), vp, vp, C.c_int, vp, vp, vp, sz, vp]
    for name in ("trit5_gemv", "bit2_gemv"):
        getattr(L, name).argtypes = [vp, vp, i64, i64, vp, vp, C.c_int, vp, vp, vp, sz, vp]
    for name in ("bitcos_gemv_grouped", "trit5_gemv_grouped", "bit2_gemv_grouped"):
        getattr(L, name).argtypes = [vp, C.c_int, i64, i64, vp, vp, C.c_int, vp, C.c_int, C.c_int, vp, C.c_int, vp, vp,
                                     vp, vp, sz, vp]
    L.bitcos_gemv_host_staging_bytes.restype = sz
    L.bitcos_gemv_host_staging_bytes.argtypes = [i64, i64, C.c_int]
    L.bitcos_gemv_host.argtypes = [C.POINTER(_Weights), vp, vp, C.c_int, vp, vp, sz, vp, sz, vp]
    L.bitcos_gemv_static.argtypes = [C.POINTER(_Weights), vp, vp, C.c_int, vp, vp]
    L.bitcos_decode_probe.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    L.bitcos_decode_probe_variant.argtypes = [C.c_int, vp, vp, sz, vp, C.c_int, vp, C.c_int, C.c_int, vp, vp, vp]
    L.bitcos_gemv_multi.argtypes = [C.POINTER(_Job), C.c_int, C.c_int, vp]
    pi = C.POINTER(C.c_int)
    L.bitcos_gemv_multi_plan.argtypes = [C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                         pi, pi, pi, pi, pi, pi, pi, pi]
    L.bitcos_gemv_multi_chained.argtypes = [C.POINTER(_Job), C.c_int, C.c_int, C.POINTER(C.c_void_p), C.c_int,
                                            C.POINTER(C.c_void_p), C.c_int, vp]
    L.bitcos_gemv_phased.argtypes = [C.POINTER(_Job), C.POINTER(C.c_int), C.c_int, C.c_int, vp, vp]
    L.bitcos_gemv_phases_host.argtypes = [C.POINTER(_Job), C.POINTER(C.c_int), C.c_int, C.c_int, vp, vp, sz, vp, vp, sz, vp]
    L.bitcos_group_pairs_device.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp, vp, vp, vp, vp]
    L.bitcos_gemv_grouped_lists.argtypes = [vp, C.c_int, i64, i64, vp, vp, vp, C.c_int, vp, C.c_int, C.c_int, vp, C.c_int,
                                            vp, vp, vp, vp, sz, vp]
    L.bitcos_gemv_static_status.argtypes = [vp, C.POINTER(C.c_int)]
    L.bitcos_wait_probe.argtypes = [vp, C.c_uint64, vp, vp]
    L.bitcos_gemv_multi_host.argtypes = [C.POINTER(_HostJob), C.c_int, C.c_int, vp]
    L.bitcos_quantize_activations.argtypes = [vp, C.c_int, i64, C.c_int, vp, vp, vp]
    L.bitcos_gemv_bf16.argtypes = [C.POINTER(_Weights), vp, C.c_int, vp, vp, vp, sz, vp]
    L.bitcos_gemv_multi_bf16.argtypes = [C.POINTER(_Job), C.c_int, C.c_int, vp]
    L.bitcos_gemv_blend_bf16.argtypes = [C.POINTER(_Weights), vp, C.c_int, vp, vp, sz, vp]
    L.bitcos_gemv_multi_group_scales.argtypes = [C.POINTER(_Job), C.c_int, C.c_int, vp]
    L.bitcos_choose_format.argtypes = [i64, i64, u64, C.POINTER(C.c_int), psz, psz]
    L.bitcos_count_nnz_device.argtypes = [vp, i64, i64, C.POINTER(u64), vp, vp]
    L.bitcos_pack_device.argtypes = [vp, vp, i64, i64, vp, vp, sz, vp, vp, vp, C.POINTER(u64), vp, vp]
    L.bitcos_gemv_group_scales.argtypes = [C.POINTER(_Weights), vp, vp, C.c_int, vp, vp, vp, sz, vp]
    _lib = L
    return L


def _check(status: int, what: str):
    if status != 0:
        L = load_library()
        detail = L.bitcos_status_string(status).decode()
        if status == 8:
            detail += f", cudaError {L.bitcos_last_cuda_error()}"
        raise BitcosError(status, what, detail)


def _np(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _ptr(a: np.ndarray):
    return C.c_void_p(a.ctypes.data)


# ---------------------------------------------------------------------------------------------
# host packers
# ---------------------------------------------------------------------------------------------
@dataclass
class PackedBitcos:
    M: int
    K: int
    nnz: int
    bitmap: np.ndarray      # uint32
    signs: np.ndarray       # uint32, zero slack included
    tile_off: np.ndarray    # uint32 [n_tiles + 1] (a view of tile_off_buf without its padding)
    scales: np.ndarray      # uint16, tile order
    tile_off_buf: np.ndarray = None     # tile_off zero padded to a multiple of 16 bytes, as uploaded

    def payload_bytes(self) -> int:
        """Bytes a GEMV has to read: bitmap, the sign bits (not the slack), offsets, scales."""
        return self.bitmap.nbytes + (self.nnz + 7) // 8 + self.tile_off.nbytes + self.scales.nbytes

    def to_device(self, device="cuda"):
        import torch
        off = self.tile_off_buf if self.tile_off_buf is not None else self.tile_off
        t = [torch.from_numpy(a.view(np.int32) if a.dtype == np.uint32 else a.view(np.int16)).to(device)
             for a in (self.bitmap, self.signs, off, self.scales)]
        return DeviceBitcos(self.M, self.K, self.nnz, *t, tile_off_host=np.ascontiguousarray(self.tile_off))


class DeviceBitcos:
    """A BITCOS matrix resident in device memory (tensors only own the bytes)."""

    def __init__(self, M, K, nnz, bitmap, signs, tile_off, scales, tile_off_host=None):
        self.M, self.K, self.nnz = M, K, nnz
        self.bitmap, self.signs, self.tile_off, self.scales = bitmap, signs, tile_off, scales
        self.tile_off_host = tile_off_host           # optional host copy (numpy uint32), kept alive here
        self.desc = _Weights(bitmap.data_ptr(), signs.data_ptr(), tile_off.data_ptr(), scales.data_ptr(), M, K,
                             tile_off_host.ctypes.data if tile_off_host is not None else None)

    def clone(self):
        return DeviceBitcos(self.M, self.K, self.nnz, self.bitmap.clone(), self.signs.clone(),
                            self.tile_off.clone(), self.scales.clone(), self.tile_off_host)

    def without_host_offsets(self):
        """The same device buffers, described without the host copy of tile_off."""
        return DeviceBitcos(self.M, self.K, self.nnz, self.bitmap, self.signs, self.tile_off, self.scales, None)

    def payload_bytes(self) -> int:
        n_tiles = (self.M + TILE_ROWS - 1) // TILE_ROWS * (self.K // GROUP)
        return self.bitmap.numel() * 4 + (self.nnz + 7) // 8 + (n_tiles + 1) * 4 + self.scales.numel() * 2


class DevicePlain:
    """A five-trit or 2-bit matrix in device memory: payload words + scales in tile order."""

    def __init__(self, M, K, words, scales):
        self.M, self.K, self.words, self.scales = M, K, words, scales

    def clone(self):
        return DevicePlain(self.M, self.K, self.words.clone(), self.scales.clone())

    def payload_bytes(self) -> int:
        return self.words.numel() * 4 + self.scales.numel() * 2


def bitcos_pack(trits, scales_bf16) -> PackedBitcos:
    L = load_library()
    t = _np(trits, np.int8)
    M, K = t.shape
    s = _np(scales_bf16, np.uint16)
    nnz = C.c_uint64(0)
    _check(L.bitcos_count_nnz(_ptr(t), M, K, C.byref(nnz)), "bitcos_count_nnz")
    sizes = [C.c_size_t(0) for _ in range(4)]
    _check(L.bitcos_pack_sizes(M, K, nnz.value, *[C.byref(v) for v in sizes]), "bitcos_pack_sizes")
    bitmap = np.zeros(sizes[0].value // 4, np.uint32)
    signs = np.zeros(sizes[1].value // 4, np.uint32)
    tile_off_buf = np.zeros(sizes[2].value // 4, np.uint32)
    scales = np.zeros(sizes[3].value // 2, np.uint16)
    out = C.c_uint64(0)
    _check(L.bitcos_pack(_ptr(t), _ptr(s), M, K, _ptr(bitmap), _ptr(signs), signs.nbytes, _ptr(tile_off_buf),
                         _ptr(scales), C.byref(out)), "bitcos_pack")
    n_tiles = (M + TILE_ROWS - 1) // TILE_ROWS * (K // GROUP)
    return PackedBitcos(M, K, int(out.value), bitmap, signs, tile_off_buf[:n_tiles + 1], scales, tile_off_buf)


def bitcos_choose_format(M: int, K: int, nnz: int):
    """('bitcos' or 'trit5', BITCOS bytes, five-trit bytes): the format that stores the matrix in fewer bytes."""
    fmt, a, b = C.c_int(0), C.c_size_t(0), C.c_size_t(0)
    _check(load_library().bitcos_choose_format(M, K, nnz, C.byref(fmt), C.byref(a), C.byref(b)), "bitcos_choose_format")
    return ("bitcos", "trit5")[fmt.value], int(a.value), int(b.value)


PACK_SCRATCH_BYTES = 256


def bitcos_count_nnz_device(trits) -> int:
    """Non-zero weights of an int8 [M, K] tensor in device memory (waits for the stream)."""
    import torch
    M, K = trits.shape
    scratch = torch.empty(PACK_SCRATCH_BYTES, dtype=torch.uint8, device=trits.device)
    nnz = C.c_uint64(0)
    _check(load_library().bitcos_count_nnz_device(trits.data_ptr(), M, K, C.byref(nnz), scratch.data_ptr(), _stream()),
           "bitcos_count_nnz_device")
    return int(nnz.value)


def bitcos_pack_device(trits, scales_bf16) -> "DeviceBitcos":
    """Packs an int8 [M, K] tensor of trits and an int16/bfloat16 [M, K / 128] tensor of bf16 scales,
    both in device memory, into a DeviceBitcos (with the host copy of tile_off) on the same device."""
    import torch
    L = load_library()
    if trits.dtype != torch.int8 or trits.dim() != 2 or not trits.is_contiguous() or not scales_bf16.is_contiguous():
        raise ValueError("trits must be a contiguous int8 [M, K] tensor, scales contiguous")
    M, K = trits.shape
    # the sign vector is sized for the worst case (every weight non-zero) and cut to size afterwards:
    # one pass over the trits less than counting first
    Mp = (M + TILE_ROWS - 1) // TILE_ROWS * TILE_ROWS
    sizes = [C.c_size_t(0) for _ in range(4)]
    _check(L.bitcos_pack_sizes(M, K, min(Mp * K, 0xFFFFFFFF), *[C.byref(v) for v in sizes]), "bitcos_pack_sizes")
    dev = trits.device
    bitmap = torch.empty(sizes[0].value // 4, dtype=torch.int32, device=dev)
    signs_max = torch.empty(sizes[1].value // 4, dtype=torch.int32, device=dev)
    tile_off = torch.empty(sizes[2].value // 4, dtype=torch.int32, device=dev)
    scales = torch.empty(sizes[3].value // 2, dtype=torch.int16, device=dev)
    off_host = np.zeros(sizes[2].value // 4, np.uint32)
    scratch = torch.empty(PACK_SCRATCH_BYTES, dtype=torch.uint8, device=dev)
    out = C.c_uint64(0)
    _check(L.bitcos_pack_device(trits.data_ptr(), scales_bf16.data_ptr(), M, K, bitmap.data_ptr(), signs_max.data_ptr(),
                                sizes[1].value, tile_off.data_ptr(), scales.data_ptr(), _ptr(off_host), C.byref(out),
                                scratch.data_ptr(), _stream()), "bitcos_pack_device")
    need = C.c_size_t(0)
    _check(L.bitcos_pack_sizes(M, K, out.value, None, C.byref(need), None, None), "bitcos_pack_sizes")
    signs = signs_max[:need.value // 4].clone()
    del signs_max
    n_tiles = (M + TILE_ROWS - 1) // TILE_ROWS * (K // GROUP)
    return DeviceBitcos(M, K, int(out.value), bitmap, signs, tile_off, scales,
                        tile_off_host=np.ascontiguousarray(off_host[:n_tiles + 1]))


def bitcos_unpack(p: PackedBitcos) -> np.ndarray:
    out = np.zeros((p.M, p.K), np.int8)
    _check(load_library().bitcos_unpack(_ptr(p.bitmap), _ptr(p.signs), _ptr(p.tile_off), p.M, p.K, _ptr(out)),
           "bitcos_unpack")
    return out


def scales_tile(scales_bf16, M, K) -> np.ndarray:
    s = _np(scales_bf16, np.uint16)
    Mp = (M + TILE_ROWS - 1) // TILE_ROWS * TILE_ROWS
    out = np.zeros(Mp * (K // GROUP), np.uint16)
    _check(load_library().bitcos_scales_tile(_ptr(s), M, K, _ptr(out)), "bitcos_scales_tile")
    return out


def scales_untile(tiled, M, K) -> np.ndarray:
    t = _np(tiled, np.uint16)
    out = np.zeros((M, K // GROUP), np.uint16)
    _check(load_library().bitcos_scales_untile(_ptr(t), M, K, _ptr(out)), "bitcos_scales_untile")
    return out


def _plain_pack(name, trits):
    L = load_library()
    t = _np(trits, np.int8)
    M, K = t.shape
    n = C.c_size_t(0)
    _check(getattr(L, name + "_pack_sizes")(M, K, C.byref(n)), name + "_pack_sizes")
    words = np.zeros(n.value // 4, np.uint32)
    _check(getattr(L, name + "_pack")(_ptr(t), M, K, _ptr(words)), name + "_pack")
    return words


def _plain_unpack(name, words, M, K):
    w = _np(words, np.uint32)
    out = np.zeros((M, K), np.int8)
    _check(getattr(load_library(), name + "_unpack")(_ptr(w), M, K, _ptr(out)), name + "_unpack")
    return out


def trit5_pack(trits) -> np.ndarray:
    return _plain_pack("trit5", trits)


def trit5_unpack(words, M, K) -> np.ndarray:
    return _plain_unpack("trit5", words, M, K)


def bit2_pack(trits) -> np.ndarray:
    return _plain_pack("bit2", trits)


def bit2_unpack(words, M, K) -> np.ndarray:
    return _plain_unpack("bit2", words, M, K)


def plain_to_device(words, scales_tiled, M, K, device="cuda") -> DevicePlain:
    import torch
    return DevicePlain(M, K, torch.from_numpy(_np(words, np.uint32).view(np.int32)).to(device),
                       torch.from_numpy(_np(scales_tiled, np.uint16).view(np.int16)).to(device))


# ---------------------------------------------------------------------------------------------
# device entry points
# ---------------------------------------------------------------------------------------------
def bitcos_gemv_workspace_bytes(M: int, K: int) -> int:
    return int(load_library().bitcos_gemv_workspace_bytes(M, K))


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_workspace(M: int, K: int, device="cuda", copies: int = 1):
    """Device scratch for the GEMV entry points, zero filled through bitcos_workspace_init."""
    import torch
    n = bitcos_gemv_workspace_bytes(M, K) * copies
    ws = torch.empty(max(n, 256), dtype=torch.uint8, device=device)
    _check(load_library().bitcos_workspace_init(C.c_void_p(ws.data_ptr()), ws.numel(), _stream()),
           "bitcos_workspace_init")
    return ws


def workspace_status(workspace) -> int:
    """0 if every call that used this workspace completed normally (waits for the stream)."""
    v = C.c_int(0)
    _check(load_library().bitcos_workspace_status(C.c_void_p(workspace.data_ptr()), _stream(), C.byref(v)),
           "bitcos_workspace_status")
    return int(v.value)


def _outputs(M, K, batch, y, acc_debug, device):
    import torch
    if y is None:
        y = torch.empty((batch, M), dtype=torch.float32, device=device)
    acc = None
    if acc_debug is True:
        acc = torch.empty((batch, M, K // GROUP), dtype=torch.int32, device=device)
    elif acc_debug is not None and acc_debug is not False:
        acc = acc_debug
    return y, acc


def bitcos_gemv(W: DeviceBitcos, x, x_scale, y=None, acc_debug=None, workspace=None):
    """y[b][m] = x_scale[b] * sum_g scale[m][g] * sum_{k in g} W[m][k] x[b][k]; returns (y, acc or None)."""
    batch = x.shape[0]
    if workspace is None:
        workspace = make_workspace(W.M, W.K, x.device)
    y, acc = _outputs(W.M, W.K, batch, y, acc_debug, x.device)
    _check(load_library().bitcos_gemv(C.byref(W.desc), x.data_ptr(), x_scale.data_ptr(), batch, y.data_ptr(),
                                      acc.data_ptr() if acc is not None else None, workspace.data_ptr(),
                                      workspace.numel(), _stream()), "bitcos_gemv")
    return y, acc


def bitcos_gemv_group_scales(W: DeviceBitcos, x, x_group_scale, y=None, acc_debug=None, workspace=None):
    """bitcos_gemv with one activation scale per token and group of 128: x_group_scale float32 [batch, K / 128]."""
    batch = x.shape[0]
    if tuple(x_group_scale.shape) != (batch, W.K // 128):
        raise ValueError("x_group_scale must be [batch, K / 128]")
    if workspace is None:
        workspace = make_workspace(W.M, W.K, x.device)
    y, acc = _outputs(W.M, W.K, batch, y, acc_debug, x.device)
    _check(load_library().bitcos_gemv_group_scales(C.byref(W.desc), x.data_ptr(), x_group_scale.data_ptr(), batch,
                                                   y.data_ptr(), acc.data_ptr() if acc is not None else None,
                                                   workspace.data_ptr(), workspace.numel(), _stream()),
           "bitcos_gemv_group_scales")
    return y, acc


def bitcos_gemv_bf16(W: DeviceBitcos, x_bf16, y=None, acc_debug=None, workspace=None):
    """The product from bfloat16 activations [batch, K] (batch 1 or 2), quantised per group of 128 inside the launch."""
    import torch
    if x_bf16.dtype != torch.bfloat16 or x_bf16.dim() != 2 or not x_bf16.is_contiguous():
        raise ValueError("x_bf16 must be a contiguous bfloat16 [batch, K] tensor")
    batch = x_bf16.shape[0]
    if workspace is None:
        workspace = make_workspace(W.M, W.K, x_bf16.device)
    y, acc = _outputs(W.M, W.K, batch, y, acc_debug, x_bf16.device)
    _check(load_library().bitcos_gemv_bf16(C.byref(W.desc), x_bf16.data_ptr(), batch, y.data_ptr(),
                                           acc.data_ptr() if acc is not None else None, workspace.data_ptr(),
                                           workspace.numel(), _stream()), "bitcos_gemv_bf16")
    return y, acc


def bitcos_gemv_blend_bf16(W: DeviceBitcos, x_bf16, y=None, workspace=None):
    """The 16-bit variant: weights rebuilt as +-s times unquantised bfloat16 activations [batch, K], batch 1..8."""
    import torch
    if x_bf16.dtype != torch.bfloat16 or x_bf16.dim() != 2 or not x_bf16.is_contiguous():
        raise ValueError("x_bf16 must be a contiguous bfloat16 [batch, K] tensor")
    batch = x_bf16.shape[0]
    if workspace is None:
        workspace = make_workspace(W.M, W.K, x_bf16.device)
    y, _ = _outputs(W.M, W.K, batch, y, None, x_bf16.device)
    _check(load_library().bitcos_gemv_blend_bf16(C.byref(W.desc), x_bf16.data_ptr(), batch, y.data_ptr(),
                                                 workspace.data_ptr(), workspace.numel(), _stream()),
           "bitcos_gemv_blend_bf16")
    return y


def bitcos_quantize_activations(x_bf16, group: int = 128, xq=None, x_scale=None):
    """bf16 activations [batch, K] on the device -> (int8 codes [batch, K], float32 scales
    [batch, K / 128] for group = 128, [batch] for group = 0)."""
    import torch
    if x_bf16.dtype != torch.bfloat16 or x_bf16.dim() != 2 or not x_bf16.is_contiguous():
        raise ValueError("x_bf16 must be a contiguous bfloat16 [batch, K] tensor")
    batch, K = x_bf16.shape
    if xq is None:
        xq = torch.empty((batch, K), dtype=torch.int8, device=x_bf16.device)
    if x_scale is None:
        shape = (batch,) if group == 0 else (batch, K // 128)
        x_scale = torch.empty(shape, dtype=torch.float32, device=x_bf16.device)
    _check(load_library().bitcos_quantize_activations(x_bf16.data_ptr(), batch, K, group, xq.data_ptr(),
                                                      x_scale.data_ptr(), _stream()), "bitcos_quantize_activations")
    return xq, x_scale


def _plain_gemv(name, W: DevicePlain, x, x_scale, y, acc_debug, workspace):
    batch = x.shape[0]
    if workspace is None:
        workspace = make_workspace(W.M, W.K, x.device)
    y, acc = _outputs(W.M, W.K, batch, y, acc_debug, x.device)
    _check(getattr(load_library(), name)(W.words.data_ptr(), W.scales.data_ptr(), W.M, W.K, x.data_ptr(),
                                         x_scale.data_ptr(), batch, y.data_ptr(),
                                         acc.data_ptr() if acc is not None else None, workspace.data_ptr(),
                                         workspace.numel(), _stream()), name)
    return y, acc


def trit5_gemv(W: DevicePlain, x, x_scale, y=None, acc_debug=None, workspace=None):
    return _plain_gemv("trit5_gemv", W, x, x_scale, y, acc_debug, workspace)


def bit2_gemv(W: DevicePlain, x, x_scale, y=None, acc_debug=None, workspace=None):
    return _plain_gemv("bit2_gemv", W, x, x_scale, y, acc_debug, workspace)


class DeviceExperts:
    """Descriptors of E same-shaped BITCOS matrices, copied to the device once."""

    def __init__(self, experts):
        """experts: DeviceBitcos matrices, or DevicePlain ones (five-trit / 2-bit) of one format."""
        import torch
        self.experts = experts
        self.M, self.K = experts[0].M, experts[0].K
        descs = [e.desc if isinstance(e, DeviceBitcos) else
                 _Weights(e.words.data_ptr(), None, None, e.scales.data_ptr(), e.M, e.K, None) for e in experts]
        arr = (_Weights * len(experts))(*descs)
        raw = np.frombuffer(bytes(arr), dtype=np.uint8).copy()
        self.table = torch.from_numpy(raw).to(experts[0].scales.device)


def group_pairs(pair_expert, pair_xrow):
    """Sorts (expert, activation row) pairs by expert.  Returns (order, group_expert, group_begin,
    xrow_sorted, max_group_size): pair i of the sorted list is input pair order[i]."""
    pe = np.asarray(pair_expert, np.int32)
    pr = np.asarray(pair_xrow, np.int32)
    order = np.argsort(pe, kind="stable")
    pe_s, pr_s = pe[order], pr[order]
    ge, first = np.unique(pe_s, return_index=True)
    begin = np.concatenate([first, [len(pe_s)]]).astype(np.int32)
    return order, ge.astype(np.int32), begin, pr_s, int(np.diff(begin).max())


def _grouped(name, E: DeviceExperts, group_expert, group_begin, pair_xrow, max_group_size, x, x_scale, y, acc_debug, workspace):
    import torch
    n_groups, n_pairs = group_expert.numel(), pair_xrow.numel()
    if workspace is None:
        workspace = make_workspace(E.M, E.K, x.device, copies=n_groups)
    if y is None:
        y = torch.empty((n_pairs, E.M), dtype=torch.float32, device=x.device)
    acc = None
    if acc_debug is True:
        acc = torch.empty((n_pairs, E.M, E.K // GROUP), dtype=torch.int32, device=x.device)
    _check(getattr(load_library(), name)(E.table.data_ptr(), len(E.experts), E.M, E.K, group_expert.data_ptr(),
                                         group_begin.data_ptr(), n_groups, pair_xrow.data_ptr(), n_pairs,
                                         max_group_size, x.data_ptr(), x.shape[0], x_scale.data_ptr(), y.data_ptr(),
                                         acc.data_ptr() if acc is not None else None, workspace.data_ptr(),
                                         workspace.numel(), _stream()), name)
    return y, acc


def bitcos_gemv_grouped(E: DeviceExperts, group_expert, group_begin, pair_xrow, max_group_size, x, x_scale,
                        y=None, acc_debug=None, workspace=None):
    """Grouped product: pairs listed per expert (device int32 tensors); y is [P, M] in list order."""
    return _grouped("bitcos_gemv_grouped", E, group_expert, group_begin, pair_xrow, max_group_size, x, x_scale, y, acc_debug, workspace)


def bitcos_group_pairs_device(pair_expert, pair_xrow, n_experts: int):
    """Groups (expert, activation row) pairs by expert on the device (device int32 tensors in, device tensors out):
    returns (group_expert, group_begin, pair_xrow_sorted, order, n_groups), n_groups a one-element device tensor."""
    import torch
    P = pair_expert.numel()
    cap = min(P, n_experts)
    dev = pair_expert.device
    ge = torch.zeros(cap, dtype=torch.int32, device=dev)
    gb = torch.zeros(cap + 1, dtype=torch.int32, device=dev)
    xr = torch.zeros(P, dtype=torch.int32, device=dev)
    order = torch.full((P,), -1, dtype=torch.int32, device=dev)
    ng = torch.zeros(1, dtype=torch.int32, device=dev)
    _check(load_library().bitcos_group_pairs_device(pair_expert.data_ptr(), pair_xrow.data_ptr(), P, n_experts, ge.data_ptr(),
                                                    gb.data_ptr(), xr.data_ptr(), order.data_ptr(), ng.data_ptr(), _stream()),
           "bitcos_group_pairs_device")
    return ge, gb, xr, order, ng


def bitcos_gemv_grouped_lists(E: DeviceExperts, group_expert, group_begin, n_groups_dev, pair_xrow, max_group_size, x, x_scale,
                              y=None, acc_debug=None, workspace=None):
    """bitcos_gemv_grouped with the number of groups left on the device (see bitcos_group_pairs_device)."""
    import torch
    max_groups, n_pairs = group_expert.numel(), pair_xrow.numel()
    if workspace is None:
        workspace = make_workspace(E.M, E.K, x.device, copies=max_groups)
    if y is None:
        y = torch.empty((n_pairs, E.M), dtype=torch.float32, device=x.device)
    acc = None
    if acc_debug is True:
        acc = torch.empty((n_pairs, E.M, E.K // GROUP), dtype=torch.int32, device=x.device)
    _check(load_library().bitcos_gemv_grouped_lists(E.table.data_ptr(), len(E.experts), E.M, E.K, group_expert.data_ptr(),
                                                    group_begin.data_ptr(), n_groups_dev.data_ptr(), max_groups,
                                                    pair_xrow.data_ptr(), n_pairs, max_group_size, x.data_ptr(), x.shape[0],
                                                    x_scale.data_ptr(), y.data_ptr(), acc.data_ptr() if acc is not None else None,
                                                    workspace.data_ptr(), workspace.numel(), _stream()), "bitcos_gemv_grouped_lists")
    return y, acc


def trit5_gemv_grouped(E: DeviceExperts, group_expert, group_begin, pair_xrow, max_group_size, x, x_scale,
                       y=None, acc_debug=None, workspace=None):
    """The grouped product from five-trit experts (DeviceExperts over DevicePlain matrices)."""
    return _grouped("trit5_gemv_grouped", E, group_expert, group_begin, pair_xrow, max_group_size, x, x_scale, y, acc_debug, workspace)


def bit2_gemv_grouped(E: DeviceExperts, group_expert, group_begin, pair_xrow, max_group_size, x, x_scale,
                      y=None, acc_debug=None, workspace=None):
    """The grouped product from 2-bit experts (DeviceExperts over DevicePlain matrices)."""
    return _grouped("bit2_gemv_grouped", E, group_expert, group_begin, pair_xrow, max_group_size, x, x_scale, y, acc_debug, workspace)


class MultiJobs:
    """Argument block of bitcos_gemv_multi, built once and reusable: jobs = [(W, x, x_scale, y, workspace)]."""

    def __init__(self, jobs):
        self.keep = jobs
        self.batch = jobs[0][1].shape[0]
        self.arr = (_Job * len(jobs))(*[_Job(C.addressof(W.desc), x.data_ptr(), xs.data_ptr() if xs is not None else None,
                                             y.data_ptr(), ws.data_ptr(), ws.numel()) for (W, x, xs, y, ws) in jobs])


class NextWeights:
    """A `prev` or `next` argument of bitcos_gemv_multi_chained, built once: the matrices of the launch before,
    or of a later launch."""

    def __init__(self, weights):
        self.keep = list(weights)
        self.arr = (C.c_void_p * len(self.keep))(*[C.addressof(W.desc) for W in self.keep])


def bitcos_gemv_multi_plan(shapes, batch=1, multiprocessors=148, busy_multiprocessors=0):
    """The split of a multi launch over thread blocks (host only): shapes = [(M, K)].  Returns a dict with
    per-block arrays job / first_item / items and per-job arrays items / tiles_per_item / column_blocks /
    chunk_stride."""
    L = load_library()
    n = len(shapes)
    M = (C.c_int64 * n)(*[int(s[0]) for s in shapes])
    K = (C.c_int64 * n)(*[int(s[1]) for s in shapes])
    cap = 256
    blk = [(C.c_int * cap)() for _ in range(3)]
    job = [(C.c_int * n)() for _ in range(4)]
    nb = C.c_int(0)
    _check(L.bitcos_gemv_multi_plan(M, K, n, batch, multiprocessors, busy_multiprocessors, cap, *blk, *job, C.byref(nb)),
           "bitcos_gemv_multi_plan")
    keys_b, keys_j = ("job", "first_item", "items"), ("items", "tiles_per_item", "column_blocks", "chunk_stride")
    return {"n_blocks": nb.value, "block": {k: list(a[:nb.value]) for k, a in zip(keys_b, blk)},
            "per_job": {k: list(a) for k, a in zip(keys_j, job)}}


def bitcos_gemv_multi(jobs, next=None, prev=None):
    """Up to eight (BITCOS_MAX_JOBS) independent BITCOS products in one launch; `jobs` is a MultiJobs or a list of
    (W, x, x_scale, y, workspace) tuples with a common batch size.  Hints for a launch inside a fixed sequence
    (bitcos_gemv_multi_chained; each a NextWeights or a list of DeviceBitcos): `next` = matrices a later launch
    will read, which this launch asks to be brought into L2; `prev` = the matrices of the launch directly before
    this one in the stream, from which the launch works out how many of its blocks will start late."""
    mj = jobs if isinstance(jobs, MultiJobs) else MultiJobs(jobs)
    if next is None and prev is None:
        _check(load_library().bitcos_gemv_multi(mj.arr, len(mj.arr), mj.batch, _stream()), "bitcos_gemv_multi")
    else:
        nw = next if isinstance(next, NextWeights) else NextWeights(next or [])
        pw = prev if isinstance(prev, NextWeights) else NextWeights(prev or [])
        _check(load_library().bitcos_gemv_multi_chained(mj.arr, len(mj.arr), mj.batch, pw.arr, len(pw.keep), nw.arr,
                                                        len(nw.keep), _stream()), "bitcos_gemv_multi_chained")
    return [j[3] for j in mj.keep]


PHASED_SYNC_BYTES = 64


def make_phased_sync(device="cuda"):
    """Zero-filled device scratch for bitcos_gemv_phased (the launch leaves it zero)."""
    import torch
    return torch.zeros(PHASED_SYNC_BYTES, dtype=torch.uint8, device=device)


class PhasedJobs(MultiJobs):
    """Argument block of bitcos_gemv_phased: jobs as for MultiJobs plus one phase per job."""

    def __init__(self, jobs, phases, sync=None):
        super().__init__(jobs)
        self.phases = (C.c_int * len(jobs))(*[int(p) for p in phases])
        self.sync = sync if sync is not None else make_phased_sync()


def bitcos_gemv_phased(jobs, phases=None, sync=None):
    """Jobs in dependency order in one launch: `jobs` is a PhasedJobs, or a list of (W, x, x_scale, y, workspace)
    tuples with `phases` (one int per job, non-decreasing from 0) and a sync buffer from make_phased_sync."""
    pj = jobs if isinstance(jobs, PhasedJobs) else PhasedJobs(jobs, phases, sync)
    _check(load_library().bitcos_gemv_phased(pj.arr, pj.phases, len(pj.arr), pj.batch, pj.sync.data_ptr(), _stream()),
           "bitcos_gemv_phased")
    return [j[3] for j in pj.keep]


class HostPhases:
    """Everything bitcos_gemv_phases_host needs for a fixed set of matrices, built once: one pinned host block and
    one device block for all jobs' activations and scales, one of each for all outputs, and the job list.
    weights = [(DeviceBitcos, workspace)], phases = one int per job; fill x[j] / x_scale[j] (numpy views
    of the pinned block), call run(), read y[j]."""

    def __init__(self, weights, phases, batch: int = 1):
        import torch
        self.batch = batch
        off, self.x_off, self.xs_off = 0, [], []
        for W, _ in weights:
            self.x_off.append(off)
            off += (batch * W.K + 15) // 16 * 16
            self.xs_off.append(off)
            off += (batch * 4 + 15) // 16 * 16
        self.in_bytes = off
        off, self.y_off = 0, []
        for W, _ in weights:
            self.y_off.append(off)
            off += (batch * W.M * 4 + 15) // 16 * 16
        self.out_bytes = off
        self.in_host = torch.zeros(self.in_bytes, dtype=torch.uint8).pin_memory()
        self.out_host = torch.zeros(self.out_bytes, dtype=torch.uint8).pin_memory()
        self.in_dev = torch.zeros(self.in_bytes, dtype=torch.uint8, device="cuda")
        self.out_dev = torch.zeros(self.out_bytes, dtype=torch.uint8, device="cuda")
        hin, hout = self.in_host.numpy(), self.out_host.numpy()
        self.x = [hin[o:o + batch * W.K].view(np.int8).reshape(batch, W.K) for o, (W, _) in zip(self.x_off, weights)]
        self.x_scale = [hin[o:o + batch * 4].view(np.float32) for o in self.xs_off]
        self.y = [hout[o:o + batch * W.M * 4].view(np.float32).reshape(batch, W.M) for o, (W, _) in zip(self.y_off, weights)]
        base_in, base_out = self.in_dev.data_ptr(), self.out_dev.data_ptr()
        self.keep = weights
        self.arr = (_Job * len(weights))(*[_Job(C.addressof(W.desc), base_in + xo, base_in + so, base_out + yo,
                                                ws.data_ptr(), ws.numel())
                                           for (W, ws), xo, so, yo in zip(weights, self.x_off, self.xs_off, self.y_off)])
        self.phases = (C.c_int * len(weights))(*[int(p) for p in phases])

    def run(self):
        _check(load_library().bitcos_gemv_phases_host(self.arr, self.phases, len(self.arr), self.batch,
                                                      self.in_host.data_ptr(), self.in_dev.data_ptr(), self.in_bytes,
                                                      self.out_host.data_ptr(), self.out_dev.data_ptr(), self.out_bytes,
                                                      _stream()), "bitcos_gemv_phases_host")
        return self.y


def bitcos_gemv_multi_group_scales(jobs):
    """bitcos_gemv_multi with one activation scale per token and group: jobs = MultiJobs or a list of
    (W, x, x_group_scale [batch, K / 128], y, workspace) tuples."""
    mj = jobs if isinstance(jobs, MultiJobs) else MultiJobs(jobs)
    _check(load_library().bitcos_gemv_multi_group_scales(mj.arr, len(mj.arr), mj.batch, _stream()),
           "bitcos_gemv_multi_group_scales")
    return [j[3] for j in mj.keep]


def bitcos_gemv_multi_bf16(jobs):
    """bitcos_gemv_multi with bfloat16 activations quantised inside the launch: jobs = MultiJobs or a list of
    (W, x_bf16, None, y, workspace) tuples, batch 1 or 2."""
    mj = jobs if isinstance(jobs, MultiJobs) else MultiJobs(jobs)
    _check(load_library().bitcos_gemv_multi_bf16(mj.arr, len(mj.arr), mj.batch, _stream()), "bitcos_gemv_multi_bf16")
    return [j[3] for j in mj.keep]


def bitcos_decode_probe(fmt: int, warps_per_block: int, iters: int, blocks: int):
    """Cycles per 32 weights per multiprocessor of the on-chip decode (the roofline's gamma)."""
    import torch
    cyc = torch.zeros(blocks, dtype=torch.int64, device="cuda")
    _check(load_library().bitcos_decode_probe(fmt, warps_per_block, iters, blocks, cyc.data_ptr(), _stream()),
           "bitcos_decode_probe")
    torch.cuda.synchronize()
    c = cyc.cpu().numpy().astype(np.float64)
    return float(np.median(c)) / (iters * warps_per_block * 128.0)


PROBE_VARIANTS = ("shifted window", "running position", "byte table", "no table", "lane = bit", "split row 1+3",
                  "split row 2+2", "split row 3+1")


def bitcos_decode_probe_variant(variant: int, W: DeviceBitcos, first_tile: int, n_tiles: int, x, iters: int, blocks: int,
                                want_acc: bool = False):
    """On-chip cost of one BITCOS decoder on tiles first_tile .. first_tile + n_tiles - 1 of W (x = int8
    [n_tiles, 128], the activations of each tile's group): cycles per 32 weights per multiprocessor, and the
    int32 accumulators [n_tiles, 32] of the last pass if asked for."""
    import torch
    cyc = torch.zeros(blocks, dtype=torch.int64, device="cuda")
    acc = torch.zeros((n_tiles, TILE_ROWS), dtype=torch.int32, device="cuda") if want_acc else None
    _check(load_library().bitcos_decode_probe_variant(
        variant, W.bitmap.data_ptr() + first_tile * 512, W.signs.data_ptr(), W.signs.numel() * 4,
        W.tile_off.data_ptr() + first_tile * 4, n_tiles, x.data_ptr(), iters, blocks, cyc.data_ptr(),
        acc.data_ptr() if acc is not None else None, _stream()), "bitcos_decode_probe_variant")
    torch.cuda.synchronize()
    c = cyc.cpu().numpy().astype(np.float64)
    gamma = float(np.median(c)) / (iters * n_tiles * 128.0)
    return (gamma, acc) if want_acc else gamma


STATIC_WORKSPACE_BYTES = 8 * 1024 * 1024


def bitcos_gemv_static_status() -> int:
    """Status word of the library's built-in scratch array after the last bitcos_gemv_static call (waits for the stream)."""
    v = C.c_int(-1)
    _check(load_library().bitcos_gemv_static_status(_stream(), C.byref(v)), "bitcos_gemv_static_status")
    return int(v.value)


def bitcos_wait_probe(workspace, limit_ns: int = 1_000_000):
    """Lets one bounded wait run out on purpose (no fault): sets the workspace's status word to 1; returns the
    nanoseconds the kernel spent polling."""
    import torch
    waited = torch.zeros(1, dtype=torch.int64, device=workspace.device)
    _check(load_library().bitcos_wait_probe(workspace.data_ptr(), int(limit_ns), waited.data_ptr(), _stream()), "bitcos_wait_probe")
    torch.cuda.synchronize()
    return int(waited.item())


def bitcos_gemv_static(W: DeviceBitcos, x, x_scale, y):
    """bitcos_gemv for callers that may not allocate: the scratch memory is a fixed array inside
    the library (at most STATIC_WORKSPACE_BYTES), so nothing is allocated here either -- `y` must be
    the caller's own [batch, M] float32 CUDA tensor.  Calls on one device share that array: do not
    let two of them overlap on the GPU.  The first call on a device must not be inside a stream
    capture."""
    _check(load_library().bitcos_gemv_static(C.byref(W.desc), x.data_ptr(), x_scale.data_ptr(), x.shape[0],
                                             y.data_ptr(), _stream()), "bitcos_gemv_static")
    return y


class MultiHostJobs:
    """Argument block of bitcos_gemv_multi_host, built once and reusable:
    jobs = [(W, x_host, x_scale_host, y_host, staging, workspace)] with numpy host arrays."""

    def __init__(self, jobs):
        self.keep = jobs
        self.batch = jobs[0][1].shape[0]
        self.arr = (_HostJob * len(jobs))(*[
            _HostJob(C.addressof(W.desc), xh.ctypes.data, xsh.ctypes.data, yh.ctypes.data, st.data_ptr(), st.numel(),
                     ws.data_ptr(), ws.numel()) for (W, xh, xsh, yh, st, ws) in jobs])


def bitcos_gemv_multi_host(jobs):
    """Several independent products from host buffers with one launch and one wait."""
    mj = jobs if isinstance(jobs, MultiHostJobs) else MultiHostJobs(jobs)
    _check(load_library().bitcos_gemv_multi_host(mj.arr, len(mj.arr), mj.batch, _stream()), "bitcos_gemv_multi_host")
    return [j[3] for j in mj.keep]


def bitcos_gemv_host_staging_bytes(M: int, K: int, batch: int) -> int:
    return int(load_library().bitcos_gemv_host_staging_bytes(M, K, batch))


def bitcos_gemv_host(W: DeviceBitcos, x_host: np.ndarray, x_scale_host: np.ndarray, y_host: np.ndarray, staging,
                     workspace):
    """Host-buffer form: copies x and x_scale to the device, multiplies, copies y back and
    waits for the stream.  x_host int8 [B, K], x_scale_host float32 [B], y_host float32 [B, M]."""
    batch = x_host.shape[0]
    _check(load_library().bitcos_gemv_host(C.byref(W.desc), x_host.ctypes.data, x_scale_host.ctypes.data, batch,
                                           y_host.ctypes.data, staging.data_ptr(), staging.numel(),
                                           workspace.data_ptr(), workspace.numel(), _stream()), "bitcos_gemv_host")
    return y_host
