"""Seeded sweep of shapes, batch sizes, densities and formats against the CPU oracle.

Complements the hand-picked parity cases: row counts around the 32-row tile edge, group counts
that are prime, smaller and larger than the decoder warps of a block, every batch size (so all
five kernel instantiations and both contraction paths run), and the degenerate densities.
"""
import numpy as np
import pytest

import datagen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL = 1e-5
ROWS = [1, 7, 31, 32, 33, 64, 100, 257, 640, 1000, 2049, 3000]
GROUPS = [1, 2, 3, 5, 8, 10, 16, 17, 20, 21, 27, 40, 54, 64]
DENSITIES = [0.0, 0.1, 0.3, 0.42, 0.6, 0.95, 1.0]
FORMATS = ["bitcos", "bitcos", "trit5", "bit2", "multi"]


@pytest.fixture(scope="module")
def bc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_16338_b200 as m
    from paper_2609_16338_b200 import build
    build.build()
    m.load_library()
    return m


def dev(a):
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_seeded_sweep(bc, seed):
    rng = np.random.default_rng(seed)
    for it in range(16):
        M = int(rng.choice(ROWS))
        K = 128 * int(rng.choice(GROUPS))
        B = int(rng.integers(1, 17))
        z = float(rng.choice(DENSITIES))
        fmt = str(rng.choice(FORMATS))
        what = f"seed {seed} case {it}: {fmt} {M}x{K} batch {B} z {z}"
        s = 5000 + 100 * seed + it
        W, S = datagen.trits(s, M, K, z), datagen.scales(s, M, K)
        x, xs = datagen.activations(s, B, K)
        acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
        xd, xsd = dev(x), dev(xs)
        ws = bc.make_workspace(M, K)
        st = bc.scales_tile(S, M, K)
        acc = None
        if fmt == "bitcos":
            y, acc = bc.bitcos_gemv(bc.bitcos_pack(W, S).to_device(), xd, xsd, acc_debug=True, workspace=ws)
        elif fmt == "trit5":
            y, acc = bc.trit5_gemv(bc.plain_to_device(bc.trit5_pack(W), st, M, K), xd, xsd, acc_debug=True, workspace=ws)
        elif fmt == "bit2":
            y, acc = bc.bit2_gemv(bc.plain_to_device(bc.bit2_pack(W), st, M, K), xd, xsd, acc_debug=True, workspace=ws)
        else:
            # two jobs in one launch, one with and one without the host copy of the entry offsets
            Wd = bc.bitcos_pack(W, S).to_device()
            y = torch.empty((B, M), dtype=torch.float32, device="cuda")
            y2 = torch.empty((B, M), dtype=torch.float32, device="cuda")
            bc.bitcos_gemv_multi([(Wd, xd, xsd, y, ws), (Wd.without_host_offsets(), xd, xsd, y2, bc.make_workspace(M, K))])
            torch.cuda.synchronize()
            assert torch.equal(y, y2), what
        torch.cuda.synchronize()
        if acc is not None:
            assert np.array_equal(acc.cpu().numpy(), acc_ref), what + ": int32 accumulators differ"
        yv = y.cpu().numpy().astype(np.float64)
        assert (np.abs(yv - y_ref) <= REL * mag).all(), what
        assert (yv[mag == 0] == 0).all(), what
        assert bc.workspace_status(ws) == 0, what


@pytest.mark.parametrize("seed", [21, 22])
def test_seeded_sweep_quantised_front_end(bc, seed):
    """The same sweep for the quantised-activation entry points: quantiser (both granularities),
    product with group scales (every batch size), product from bf16 activations (one and two
    tokens, single and multi launch), and the device packer in front of them."""
    rng = np.random.default_rng(seed)
    for it in range(14):
        M = int(rng.choice(ROWS))
        K = 128 * int(rng.choice(GROUPS))
        B = int(rng.integers(1, 17))
        z = float(rng.choice(DENSITIES))
        what = f"seed {seed} case {it}: {M}x{K} batch {B} z {z}"
        s = 7000 + 100 * seed + it
        W, S = datagen.trits(s, M, K, z), datagen.scales(s, M, K)
        bits = datagen.activations_bf16(s, B, K)
        xf = datagen.bf16_bits_to_f32(bits)
        xb = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
        Wd = bc.bitcos_pack_device(torch.from_numpy(W).cuda(), torch.from_numpy(S.view(np.int16)).cuda())
        ws = bc.make_workspace(M, K)
        q_ref, s_ref = oracle.quantize_activations(xf, 128)
        acc_ref, y_ref, mag = oracle.gemv_dense_group_scales(W, S, q_ref, s_ref)
        q, sg = bc.bitcos_quantize_activations(xb, 128)
        y, acc = bc.bitcos_gemv_group_scales(Wd, q, sg, acc_debug=True, workspace=ws)
        torch.cuda.synchronize()
        assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(sg.cpu().numpy(), s_ref), what
        assert np.array_equal(acc.cpu().numpy(), acc_ref), what
        assert (np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= REL * mag).all(), what
        qt_ref, st_ref = oracle.quantize_activations(xf, 0)
        qt, st = bc.bitcos_quantize_activations(xb, 0)
        torch.cuda.synchronize()
        assert np.array_equal(qt.cpu().numpy(), qt_ref) and np.array_equal(st.cpu().numpy(), st_ref), what
        nb = min(B, 1 + it % 2)
        if nb * K <= 49152:
            y2, acc2 = bc.bitcos_gemv_bf16(Wd, xb[:nb].contiguous(), acc_debug=True, workspace=ws)
            y3 = torch.empty((nb, M), dtype=torch.float32, device="cuda")
            bc.bitcos_gemv_multi_bf16([(Wd, xb[:nb].contiguous(), None, y3, bc.make_workspace(M, K))])
            torch.cuda.synchronize()
            assert np.array_equal(acc2.cpu().numpy(), acc_ref[:nb]), what
            assert (np.abs(y2.cpu().numpy().astype(np.float64) - y_ref[:nb]) <= REL * mag[:nb]).all(), what
            assert (np.abs(y3.cpu().numpy().astype(np.float64) - y_ref[:nb]) <= REL * mag[:nb]).all(), what
        nbl = min(B, 1 + it % 8)
        yb = bc.bitcos_gemv_blend_bf16(Wd, xb[:nbl].contiguous(), workspace=ws)
        torch.cuda.synchronize()
        yb_ref, magb = oracle.gemv_dense_blend(W, S, xf[:nbl])
        assert (np.abs(yb.cpu().numpy().astype(np.float64) - yb_ref) <= 4e-5 * magb).all(), what
        assert bc.workspace_status(ws) == 0, what
