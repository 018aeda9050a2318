"""CPU tests of the C-ABI library: it loads, exports what include/bitcos.h declares, and its
host packers produce byte for byte the layout the oracle builds from the paper's definition.
No compute entry point is called here (there is no GPU)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import datagen
import oracle
import paper_2609_16338_b200 as bc
from paper_2609_16338_b200 import build as bc_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    bc_build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bitcos.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:bitcos|trit5|bit2)_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = bc.load_library()
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(L, n), n
    assert sorted(bc.EXPORTED_SYMBOLS) == names


@pytest.mark.parametrize("M,K,z", [(256, 512, 0.42), (32, 128, 0.3), (100, 384, 0.47), (1, 128, 0.5), (640, 256, 0.33)])
def test_bitcos_pack_matches_oracle_bytes(M, K, z):
    W = datagen.trits(31, M, K, z)
    S = datagen.scales(31, M, K)
    p = bc.bitcos_pack(W, S)
    o = oracle.bitcos_pack(W)
    assert p.nnz == o.nnz == np.count_nonzero(W)
    assert np.array_equal(p.bitmap, o.bitmap)
    assert np.array_equal(p.signs, o.signs)
    assert np.array_equal(p.tile_off, o.tile_off)
    assert np.array_equal(p.scales, oracle.scales_to_tile_order(S, M, K))
    # both decoders read both packings
    assert np.array_equal(bc.bitcos_unpack(p), W)
    assert np.array_equal(oracle.bitcos_unpack(p.bitmap, p.signs, p.tile_off, M, K, "pdep"), W)
    assert np.array_equal(bc.scales_untile(p.scales, M, K), S)
    # rate: presence + sign bits = (2 - z_hat) per stored weight
    Mp = oracle.padded_rows(M)
    assert (p.bitmap.size * 32 + p.nnz) == Mp * K + np.count_nonzero(W)


@pytest.mark.parametrize("M,K", [(64, 256), (33, 384), (256, 512)])
def test_trit5_bit2_pack_match_oracle_bytes(M, K):
    W = datagen.trits(32, M, K, 0.4)
    t5, b2 = bc.trit5_pack(W), bc.bit2_pack(W)
    assert np.array_equal(t5, oracle.trit5_pack(W))
    assert np.array_equal(b2, oracle.bit2_pack(W))
    assert np.array_equal(bc.trit5_unpack(t5, M, K), W)
    assert np.array_equal(bc.bit2_unpack(b2, M, K), W)
    assert np.array_equal(oracle.trit5_unpack(t5, M, K), W)
    assert np.array_equal(oracle.bit2_unpack(b2, M, K), W)


def test_special_matrices():
    M, K = 64, 256
    for fill in (0, 1, -1):
        W = np.full((M, K), fill, np.int8)
        S = datagen.scales(33, M, K)
        p = bc.bitcos_pack(W, S)
        assert p.nnz == (M * K if fill else 0)
        assert np.array_equal(bc.bitcos_unpack(p), W)
        assert np.array_equal(p.signs, oracle.bitcos_pack(W).signs)


def test_error_codes():
    L = bc.load_library()
    M, K = 32, 128
    W = np.zeros((M, K), np.int8)
    S = np.full((M, 1), 0x3C00, np.uint16)
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_pack(np.zeros((32, 100), np.int8), S)
    assert e.value.status == 2
    W[3, 7] = 5
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_pack(W, S)
    assert e.value.status == 4
    with pytest.raises(bc.BitcosError) as e:
        bc.trit5_pack(W)
    assert e.value.status == 4
    with pytest.raises(bc.BitcosError) as e:
        bc.bit2_pack(W)
    assert e.value.status == 4
    W[3, 7] = 1
    for bad in (0x8001, 0x7F80, 0x7FC0, 0xBC00):       # negative, +Inf, NaN, -small
        S2 = S.copy()
        S2[5, 0] = bad
        with pytest.raises(bc.BitcosError) as e:
            bc.bitcos_pack(W, S2)
        assert e.value.status == 5
    # capacity: a sign buffer one byte short
    sizes = [C.c_size_t(0) for _ in range(4)]
    assert L.bitcos_pack_sizes(M, K, 1, *[C.byref(v) for v in sizes]) == 0
    bitmap = np.zeros(sizes[0].value // 4, np.uint32)
    signs = np.zeros(sizes[1].value // 4, np.uint32)
    off = np.zeros(sizes[2].value // 4, np.uint32)
    sc = np.zeros(sizes[3].value // 2, np.uint16)
    rc = L.bitcos_pack(W.ctypes.data, S.ctypes.data, M, K, bitmap.ctypes.data, signs.ctypes.data,
                       signs.nbytes - 1, off.ctypes.data, sc.ctypes.data, None)
    assert rc == 6
    assert L.bitcos_pack(None, S.ctypes.data, M, K, bitmap.ctypes.data, signs.ctypes.data, signs.nbytes,
                         off.ctypes.data, sc.ctypes.data, None) == 1
    # invalid packed codes
    assert L.trit5_unpack(np.full(32 * 7, 0xFFFFFFFF, np.uint32).ctypes.data, M, K, W.ctypes.data) == 4
    assert L.bit2_unpack(np.full(32 * 8, 0xFFFFFFFF, np.uint32).ctypes.data, M, K, W.ctypes.data) == 4
    # a tile offset that disagrees with the bitmap
    W2 = datagen.trits(34, M, K, 0.4)
    p = bc.bitcos_pack(W2, S)
    p.tile_off[1] += 1
    with pytest.raises(bc.BitcosError):
        bc.bitcos_unpack(p)
    assert L.bitcos_status_string(3).decode().startswith("device pointer")
    # device entry points validate before touching CUDA
    assert L.bitcos_gemv(None, None, None, 1, None, None, None, 0, None) == 1
    assert L.bitcos_gemv_workspace_bytes(32, 100) == 0
    assert L.bitcos_gemv_workspace_bytes(2560, 6912) >= 256
    assert L.trit5_gemv(C.c_void_p(16), C.c_void_p(16), 32, 100, C.c_void_p(16), C.c_void_p(16), 1, C.c_void_p(16),
                        None, C.c_void_p(16), 1 << 20, None) == 2
    assert L.bit2_gemv(C.c_void_p(16), C.c_void_p(16), 32, 128, C.c_void_p(16), C.c_void_p(16), 17, C.c_void_p(16),
                       None, C.c_void_p(16), 1 << 20, None) == 2
    assert L.bit2_gemv(C.c_void_p(24), C.c_void_p(16), 32, 128, C.c_void_p(16), C.c_void_p(16), 1, C.c_void_p(16),
                       None, C.c_void_p(16), 1 << 20, None) == 3
    assert L.bit2_gemv(C.c_void_p(16), C.c_void_p(16), 32, 128, C.c_void_p(16), C.c_void_p(16), 1, C.c_void_p(16),
                       None, C.c_void_p(16), 8, None) == 6


def test_group_pairs_helper():
    order, ge, gb, xr, mx = bc.group_pairs([5, 2, 5, 7, 2, 5], [0, 0, 1, 1, 2, 2])
    assert list(ge) == [2, 5, 7] and list(gb) == [0, 2, 5, 6] and mx == 3
    assert list(xr) == [0, 2, 0, 1, 2, 1] and list(order) == [1, 4, 0, 2, 5, 3]


def test_benchmark_byte_count_is_the_packed_size():
    """The roofline's numerator (bench.algorithmic_bytes) is exactly what a product has to move:
    the packed buffers as the packer sizes them (sign bits rounded up to bytes, no slack), the
    activations with their scales, and the outputs; and it reproduces 2 - z bits per weight plus
    the scale and entry-offset overheads (Eq. 1, Eq. 5)."""
    import sys
    sys.path.insert(0, ROOT)
    import bench
    for (M, K, z, B) in ((256, 512, 0.42, 1), (100, 1280, 0.3, 3), (640, 2560, 0.4219, 16)):
        W, S = datagen.trits(77, M, K, z), datagen.scales(77, M, K)
        p = bc.bitcos_pack(W, S)
        Mp = (M + 31) // 32 * 32
        tiles = Mp // 32 * (K // 128)
        io = B * (K + 4) + 4 * B * M
        assert bench.algorithmic_bytes(M, K, p.nnz, B) == p.bitmap.nbytes + (p.nnz + 7) // 8 + p.scales.nbytes + 4 * (tiles + 1) + io
        assert p.payload_bytes() == bench.algorithmic_bytes(M, K, p.nnz, B) - io
        # bits per weight of bitmap + signs = 2 - z_realised exactly (padding rows hold no weights)
        z_real = 1.0 - p.nnz / float(M * K)
        assert abs((Mp * K + p.nnz) / float(Mp * K) - (2.0 - z_real * M / Mp - (Mp - M) / Mp)) < 1e-12
        t5 = bc.trit5_pack(W)
        b2 = bc.bit2_pack(W)
        assert bench.algorithmic_bytes(M, K, p.nnz, B, "trit5") == t5.nbytes + p.scales.nbytes + io
        assert bench.algorithmic_bytes(M, K, p.nnz, B, "bit2") == b2.nbytes + p.scales.nbytes + io


def test_choose_format_breaks_even_near_three_eighths():
    """Section II-A: 2 - z bits per weight against 26 bytes per 128 weights (1.625 bits) break even
    at z = 0.375; with the entry offsets counted (32 bits per 4096 weights) a little above it.
    The byte counts are those of the oracle's packed buffers."""
    M, K = 256, 1024
    for z in (0.30, 0.36, 0.40, 0.47):
        W = datagen.trits(77, M, K, z)
        pk = oracle.bitcos_pack(W)
        fmt, b_bytes, t_bytes = bc.bitcos_choose_format(M, K, pk.nnz)
        assert b_bytes == pk.bitmap.nbytes + (pk.nnz + 7) // 8 + pk.tile_off.nbytes
        assert t_bytes == oracle.trit5_pack(W).nbytes
        assert fmt == ("bitcos" if b_bytes <= t_bytes else "trit5")
        assert fmt == ("bitcos" if z >= 0.40 else "trit5")
    # the exact crossing: bits per weight 2 - z + 32/4096 (+ the last offset) against 1.625
    n = M * K
    nnz_even = n - int(round(0.375 * n))
    assert bc.bitcos_choose_format(M, K, nnz_even)[0] == "trit5"                  # offsets tip it
    nnz_cross = n - int(np.ceil((0.375 + 32.0 / 4096) * n + 32))
    assert bc.bitcos_choose_format(M, K, nnz_cross)[0] == "bitcos"
    with pytest.raises(bc.BitcosError):
        bc.bitcos_choose_format(M, 100, 5)
