"""GPU parity for the device-side BITCOS packer: byte for byte the buffers the oracle builds from
the paper's layout (Section II-A: presence bitmap, compacted signs in the same order; entry
offsets per tile), and usable by the product as packed."""
import numpy as np
import pytest

import datagen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_16338_b200 as m
    from paper_2609_16338_b200 import build
    build.build()
    m.load_library()
    return m


def u32(t):
    return t.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("M,K,z", [(32, 128, 0.42), (1, 128, 0.5), (100, 384, 0.47), (640, 2560, 0.4219), (2560, 6912, 0.33),
                                   (4097, 1280, 0.42), (64, 256, 1.0), (64, 256, 0.0), (8192, 5120, 0.4711)])
def test_device_pack_matches_oracle_bytes(bc, M, K, z):
    W = datagen.trits(3000 + M, M, K, z)
    if z == 0.0:
        W[W == 0] = 1
    S = datagen.scales(3000 + M, M, K)
    ref = oracle.bitcos_pack(W)
    Wd = bc.bitcos_pack_device(torch.from_numpy(W).cuda(), torch.from_numpy(S.view(np.int16)).cuda())
    assert Wd.nnz == ref.nnz == bc.bitcos_count_nnz_device(torch.from_numpy(W).cuda())
    assert np.array_equal(u32(Wd.bitmap), ref.bitmap)
    n_tiles = oracle.num_tiles(M, K)
    off = u32(Wd.tile_off)
    assert np.array_equal(off[:n_tiles + 1], ref.tile_off) and not off[n_tiles + 1:].any()
    assert np.array_equal(Wd.tile_off_host, ref.tile_off)
    sg = u32(Wd.signs)
    n_words = (ref.nnz + 31) // 32
    assert np.array_equal(sg[:n_words], np.asarray(ref.signs, np.uint32)[:n_words]) and not sg[n_words:].any()
    assert np.array_equal(Wd.scales.cpu().numpy().view(np.uint16), oracle.scales_to_tile_order(S, M, K).reshape(-1))
    # and the library's host packer wrote the same bytes (sign slack included)
    host = bc.bitcos_pack(W, S)
    assert np.array_equal(sg, host.signs) and np.array_equal(off, host.tile_off_buf)


def test_device_packed_matrix_multiplies(bc):
    M, K, B = 2560, 2560, 3
    W, S = datagen.trits(3100, M, K, 0.4219), datagen.scales(3100, M, K)
    x, xs = datagen.activations(3100, B, K)
    acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
    Wd = bc.bitcos_pack_device(torch.from_numpy(W).cuda(), torch.from_numpy(S.view(np.int16)).cuda())
    y, acc = bc.bitcos_gemv(Wd, torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda(), acc_debug=True)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy(), acc_ref)
    assert (np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= 1e-5 * mag).all()


def test_device_pack_error_codes(bc):
    M, K = 64, 256
    W = datagen.trits(3200, M, K, 0.4)
    S = datagen.scales(3200, M, K)
    bad = W.copy()
    bad[5, 17] = 2
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_pack_device(torch.from_numpy(bad).cuda(), torch.from_numpy(S.view(np.int16)).cuda())
    assert e.value.status == 4
    bad[5, 17] = -2
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_count_nnz_device(torch.from_numpy(bad).cuda())
    assert e.value.status == 4
    Sb = S.copy()
    Sb[3, 1] = 0x7F80                                  # +Inf
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_pack_device(torch.from_numpy(W).cuda(), torch.from_numpy(Sb.view(np.int16)).cuda())
    assert e.value.status == 5
    Sb[3, 1] = 0x8000 | 0x3C00                         # negative
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_pack_device(torch.from_numpy(W).cuda(), torch.from_numpy(Sb.view(np.int16)).cuda())
    assert e.value.status == 5
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_pack_device(torch.zeros((4, 100), dtype=torch.int8, device="cuda"),
                              torch.zeros((4, 1), dtype=torch.int16, device="cuda"))
    assert e.value.status == 2
