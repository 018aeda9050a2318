"""The no-allocation entry point, bitcos_gemv_static, against bitcos_gemv.

Some callers cannot call cudaMalloc where they multiply (memory handed out once at start-up, a
plug-in inside another program's pool, a path that must not take cudaMalloc's device-wide
synchronisation).  For them the library carries its scratch memory as a fixed array; this test
calls that entry point through the C ABI twice in a row -- the array is shared and keeps the
previous call's contents -- and checks both results against the ordinary entry point, on shapes
whose row sums are split over several thread blocks (so the scratch is really used).

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest

import datagen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL = 1e-5


@pytest.fixture(scope="module")
def bc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_16338_b200 as m
    from paper_2609_16338_b200 import build
    build.build()
    m.load_library()
    return m


@pytest.mark.parametrize("M,K,B", [(96, 6912, 1), (320, 8192, 3), (2560, 6912, 1), (256, 512, 2)])
def test_static_workspace_entry_point_matches_bitcos_gemv(bc, M, K, B):
    W, S = datagen.trits(700 + M, M, K, 0.4219), datagen.scales(700 + M, M, K)
    x, xs = datagen.activations(700 + K, B, K)
    _, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
    Wd = bc.bitcos_pack(W, S).to_device()
    xd, xsd = torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda()
    y_plain, _ = bc.bitcos_gemv(Wd, xd, xsd)
    torch.cuda.synchronize()
    want = y_plain.cpu().numpy().astype(np.float64)
    assert (np.abs(want - y_ref) <= REL * mag).all()
    for call in range(2):
        y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
        bc.bitcos_gemv_static(Wd, xd, xsd, y)
        torch.cuda.synchronize()
        got = y.cpu().numpy().astype(np.float64)
        assert (np.abs(got - want) <= REL * mag).all(), f"call {call}: differs from bitcos_gemv"
        assert (np.abs(got - y_ref) <= REL * mag).all(), f"call {call}: differs from the oracle"


def test_static_workspace_rejects_what_does_not_fit(bc):
    L = bc.load_library()
    assert bc.bitcos_gemv_workspace_bytes(2560, 6912) <= bc.binding.STATIC_WORKSPACE_BYTES
    # 64 row-block-heavy rows x a very long reduction: the scratch requirement exceeds the array
    M, K = 32 * 4096, 128 * 64
    assert bc.bitcos_gemv_workspace_bytes(M, K) > bc.binding.STATIC_WORKSPACE_BYTES
    import ctypes as C
    desc = bc.binding._Weights(16, 16, 16, 16, M, K)
    rc = L.bitcos_gemv_static(C.byref(desc), C.c_void_p(16), C.c_void_p(16), 1, C.c_void_p(16), None)
    assert rc == 6      # BITCOS_ERR_CAPACITY, before anything touches the GPU
