"""GPU parity for the 16-bit variant (Sections II-B / II-D): weights rebuilt as +-s, multiplied
with unquantised bf16 activations on the tensor cores.

Bar: every product (bf16 x bf16) is exact in fp32; a group's 128 products are accumulated in fp32
inside the tensor cores and at most 200 groups are then added in fp32, so the outputs are held to
(128 + G) * 2^-24 < 2e-5 of sum|terms| with every rounding to nearest (measured errors are some five times smaller still).
"""
import numpy as np
import pytest

import datagen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL = 2e-5


@pytest.fixture(scope="module")
def bc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_16338_b200 as m
    from paper_2609_16338_b200 import build
    build.build()
    m.load_library()
    return m


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("M,K,B", [(64, 128, 1), (32, 256, 8), (2560, 2560, 1), (2560, 2560, 3), (640, 6912, 2), (2560, 6912, 8),
                                   (333, 1280, 5), (6912, 2560, 1), (96, 25600, 4), (1000, 5120, 7)])
def test_blend_product(bc, M, K, B):
    W, S = datagen.trits(4000 + M, M, K, 0.4219), datagen.scales(4000 + M, M, K)
    bits = datagen.activations_bf16(4000 + K + B, B, K)
    x = datagen.bf16_bits_to_f32(bits)
    y_ref, mag = oracle.gemv_dense_blend(W, S, x)
    Wd = bc.bitcos_pack(W, S).to_device()
    ws = bc.make_workspace(M, K)
    worst = 0.0
    for rep in range(2):
        y = bc.bitcos_gemv_blend_bf16(Wd, dev_bf16(bits), workspace=ws)
        torch.cuda.synchronize()
        yv = y.cpu().numpy().astype(np.float64)
        err = np.abs(yv - y_ref)
        assert (err <= REL * mag).all(), (M, K, B, rep, float((err / np.maximum(mag, 1e-300)).max()))
        assert (yv[mag == 0] == 0).all()
        worst = max(worst, float((err / np.maximum(mag, 1e-300)).max()))
    assert bc.workspace_status(ws) == 0
    assert worst < 1e-5, worst          # in practice well inside the integer path's bar too


def test_blend_product_exact_cases(bc):
    """Inputs on which every partial sum is exactly representable: activations that are small
    integers, scales that are powers of two.  The result must then be exact, which pins the order of
    the weights and activations inside the tensor-core fragments (any mix-up changes the sum)."""
    M, K, B = 96, 1024, 6
    W = datagen.trits(4100, M, K, 0.4)
    G = K // 128
    expo = (np.arange(M * G).reshape(M, G) % 5).astype(np.int64)
    S = datagen.f32_to_bf16_bits((2.0 ** -expo).astype(np.float32)).reshape(M, G)
    q, _ = datagen.activations(4100, B, K)
    x = q.astype(np.float32)                      # integers up to 127: bf16 values
    bits = datagen.f32_to_bf16_bits(x)
    y_ref, _ = oracle.gemv_dense_blend(W, S, x)
    Wd = bc.bitcos_pack(W, S).to_device()
    y = bc.bitcos_gemv_blend_bf16(Wd, dev_bf16(bits))
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy().astype(np.float64), y_ref)
    # one non-zero weight at a time, every position of a group: picks out single activations
    for k in (0, 1, 2, 3, 4, 31, 32, 33, 63, 64, 100, 127, 128, 129, 1023):
        W1 = np.zeros((M, K), np.int8)
        W1[np.arange(M), (k + 7 * np.arange(M)) % K] = np.where(np.arange(M) % 2, -1, 1)
        y1 = bc.bitcos_gemv_blend_bf16(bc.bitcos_pack(W1, S).to_device(), dev_bf16(bits))
        torch.cuda.synchronize()
        ref1, _ = oracle.gemv_dense_blend(W1, S, x)
        assert np.array_equal(y1.cpu().numpy().astype(np.float64), ref1), k


def test_blend_product_rejects_large_batches(bc):
    W, S = datagen.trits(4200, 64, 256, 0.4), datagen.scales(4200, 64, 256)
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_gemv_blend_bf16(bc.bitcos_pack(W, S).to_device(), torch.zeros((9, 256), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == 2
