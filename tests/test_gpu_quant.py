"""GPU parity for the quantised-activation front end (Section II-C): the int8 quantiser per
group of 128 / per token, and the product with one activation scale per token and group.

Bar: codes, scales and int32 group accumulators bit-exact (the quantiser decides in float32
on both sides); fp32 outputs within 1e-5 of sum|terms|.
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


def dev(a):
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_bf16(bits):
    return dev(bits).view(torch.bfloat16)


def special_rows(bits):
    """Plants the degenerate groups into row 0: all zero, a single non-zero, a negative largest
    magnitude, ties of the rounding, very small and very large values."""
    x = datagen.bf16_bits_to_f32(bits).copy()
    K = x.shape[1]
    x[0, 0:128] = 0
    if K >= 256:
        x[0, 128:256] = 0
        x[0, 200] = -3.0
    if K >= 384:
        x[0, 256:384] = np.float32(0.25) * np.arange(128, dtype=np.float32)     # largest 31.75
        x[0, 256] = -127.0                                                   # factor exactly 1: ties at .5
        x[0, 257:265] = [0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 126.5, -126.5]
    if K >= 512:
        x[0, 384:512] *= np.float32(2.0 ** -110)
    if K >= 640:
        x[0, 512:640] *= np.float32(2.0 ** 100)
    return datagen.f32_to_bf16_bits(x)


@pytest.mark.parametrize("B,K", [(1, 128), (1, 2560), (3, 6912), (16, 5120), (2, 25600), (5, 640)])
def test_quantiser_matches_oracle(bc, B, K):
    bits = special_rows(datagen.activations_bf16(2000 + B + K, B, K))
    xf = datagen.bf16_bits_to_f32(bits)
    xd = dev_bf16(bits)
    for group in (128, 0):
        q_ref, s_ref = oracle.quantize_activations(xf, group)
        for rep in range(2):
            q, s = bc.bitcos_quantize_activations(xd, group)
            torch.cuda.synchronize()
            assert np.array_equal(q.cpu().numpy(), q_ref), (B, K, group)
            assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32)), (B, K, group)


def test_quantiser_rejects_bad_arguments(bc):
    x = torch.zeros((1, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bc.BitcosError):
        bc.bitcos_quantize_activations(x, 64)
    with pytest.raises(bc.BitcosError):
        bc.bitcos_quantize_activations(torch.zeros((1, 192), dtype=torch.bfloat16, device="cuda"), 0)
    with pytest.raises(bc.BitcosError):
        bc.bitcos_quantize_activations(torch.zeros((17, 256), dtype=torch.bfloat16, device="cuda"), 128)
    # a misaligned activation pointer
    buf = torch.zeros(256 + 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bc.BitcosError):
        bc.bitcos_quantize_activations(buf[4:260].view(1, 256), 128)


@pytest.mark.parametrize("M,K,B", [
    (64, 128, 1), (2560, 2560, 1), (2560, 2560, 2), (6912, 2560, 3), (2560, 6912, 1), (2560, 6912, 2),
    (640, 6912, 5), (1000, 5120, 8), (333, 1280, 16), (96, 25600, 1), (96, 25600, 12), (8192, 5120, 4),
])
def test_group_scale_product(bc, M, K, B):
    """Random positive scales per token and group (a factor of up to 50 between groups)."""
    W, S = datagen.trits(2100 + M, M, K, 0.4219), datagen.scales(2100 + M, M, K)
    x, _ = datagen.activations(2100 + K + B, B, K)
    G = K // 128
    xg = (0.001 * (1.0 + 49.0 * datagen.uniform(2100 + B, datagen.STREAM_XS, 0, B * G))).astype(np.float32).reshape(B, G)
    acc_ref, y_ref, mag = oracle.gemv_dense_group_scales(W, S, x, xg)
    Wd = bc.bitcos_pack(W, S).to_device()
    ws = bc.make_workspace(M, K)
    xd, xgd = dev(x), dev(xg)
    for rep in range(2):
        y, acc = bc.bitcos_gemv_group_scales(Wd, xd, xgd, acc_debug=(rep == 0) or None, workspace=ws)
        torch.cuda.synchronize()
        if acc is not None:
            assert np.array_equal(acc.cpu().numpy(), acc_ref), (M, K, B)
        yv = y.cpu().numpy().astype(np.float64)
        assert (np.abs(yv - y_ref) <= REL * mag).all(), (M, K, B, rep)
    assert bc.workspace_status(ws) == 0
    # equal scales in every group: the per-token entry point, to rounding
    xs = xg[:, 0].copy()
    y1, _ = bc.bitcos_gemv(Wd, xd, dev(xs), workspace=ws)
    y2, _ = bc.bitcos_gemv_group_scales(Wd, xd, dev(np.repeat(xs[:, None], G, axis=1)), workspace=ws)
    torch.cuda.synchronize()
    _, y_tok, mag_tok = oracle.gemv_dense(W, S, x, xs)
    assert (np.abs(y1.cpu().numpy() - y_tok) <= REL * mag_tok).all()
    assert (np.abs(y2.cpu().numpy() - y_tok) <= REL * mag_tok).all()


def test_group_scale_product_two_tiles_per_warp(bc):
    """Large matrices (one and two tokens), where a decoder warp takes two tiles per item."""
    for (M, K, B) in ((19200, 5120, 1), (38400, 2560, 2)):
        W, S = datagen.trits(2200 + K, M, K, 0.4219), datagen.scales(2200 + K, M, K)
        x, _ = datagen.activations(2200 + K, B, K)
        G = K // 128
        xg = (0.002 * (1.0 + 9.0 * datagen.uniform(2200 + B, datagen.STREAM_XS, 0, B * G))).astype(np.float32).reshape(B, G)
        rows = np.unique(np.concatenate([np.arange(0, M, M // 211), [M - 1, M - 32, M - 33, 31, 32, 63, 64]]))
        acc_ref, y_ref, mag = oracle.gemv_dense_group_scales(W[rows], S[rows], x, xg)
        Wd = bc.bitcos_pack(W, S).to_device()
        ws = bc.make_workspace(M, K)
        y, acc = bc.bitcos_gemv_group_scales(Wd, dev(x), dev(xg), acc_debug=True, workspace=ws)
        torch.cuda.synchronize()
        assert np.array_equal(acc.cpu().numpy()[:, rows], acc_ref)
        assert (np.abs(y.cpu().numpy().astype(np.float64)[:, rows] - y_ref) <= REL * mag).all()
        assert bc.workspace_status(ws) == 0


@pytest.mark.parametrize("B", [1, 2, 4, 16])
def test_quantise_then_multiply_on_one_stream(bc, B):
    """bf16 activations -> quantiser -> product, back to back on one stream with no host wait in
    between (the product starts while the quantiser still runs and must wait for its codes and
    scales), against the same chain in the oracle; both scale granularities."""
    M, K = 2560, 6912
    W, S = datagen.trits(2300, M, K, 0.4219), datagen.scales(2300, M, K)
    Wd = bc.bitcos_pack(W, S).to_device()
    ws = bc.make_workspace(M, K)
    G = K // 128
    for rep in range(3):
        bits = datagen.activations_bf16(2300 + 10 * B + rep, B, K)
        xf = datagen.bf16_bits_to_f32(bits)
        xd = dev_bf16(bits)
        q = torch.empty((B, K), dtype=torch.int8, device="cuda")
        sg = torch.empty((B, G), dtype=torch.float32, device="cuda")
        st = torch.empty((B,), dtype=torch.float32, device="cuda")
        y = torch.empty((B, M), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        bc.bitcos_quantize_activations(xd, 128, xq=q, x_scale=sg)
        bc.bitcos_gemv_group_scales(Wd, q, sg, y=y, workspace=ws)
        q_ref, s_ref = oracle.quantize_activations(xf, 128)
        _, y_ref, mag = oracle.gemv_dense_group_scales(W, S, q_ref, s_ref)
        torch.cuda.synchronize()
        assert np.array_equal(q.cpu().numpy(), q_ref)
        assert (np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= REL * mag).all(), (B, rep, "groups")
        # the unquantised product is met within the quantisation bound
        Sf = datagen.bf16_bits_to_f32(S).astype(np.float64)
        exact = xf.astype(np.float64) @ (W.astype(np.float64) * np.repeat(Sf, 128, axis=1)).T
        nnz = np.abs(W).reshape(M, G, 128).sum(axis=2).astype(np.float64)
        bound = 0.5 * (1 + 2.0 ** -14) * np.einsum("mg,bg->bm", Sf * nnz, s_ref.astype(np.float64))
        assert (np.abs(y.cpu().numpy().astype(np.float64) - exact) <= bound + REL * mag).all()
        # one scale per token in front of the ordinary entry point
        bc.bitcos_quantize_activations(xd, 0, xq=q, x_scale=st)
        bc.bitcos_gemv(Wd, q, st, y=y, workspace=ws)
        q_ref, s_ref = oracle.quantize_activations(xf, 0)
        _, y_ref, mag = oracle.gemv_dense(W, S, q_ref, s_ref)
        torch.cuda.synchronize()
        assert np.array_equal(q.cpu().numpy(), q_ref)
        assert (np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= REL * mag).all(), (B, rep, "tokens")
    assert bc.workspace_status(ws) == 0


@pytest.mark.parametrize("M,K,B", [(64, 128, 1), (2560, 2560, 1), (2560, 2560, 2), (2560, 6912, 1), (2560, 6912, 2),
                                   (6912, 2560, 1), (333, 1280, 2), (640, 640, 1), (96, 25600, 1), (1000, 5120, 2)])
def test_product_from_bf16_activations(bc, M, K, B):
    """The quantiser fused into the product: the same codes (seen through the bit-exact int32
    accumulators), scales and outputs as the oracle's quantise-then-multiply chain."""
    W, S = datagen.trits(2400 + M, M, K, 0.4219), datagen.scales(2400 + M, M, K)
    bits = special_rows(datagen.activations_bf16(2400 + K + B, B, K))
    xf = datagen.bf16_bits_to_f32(bits)
    q_ref, s_ref = oracle.quantize_activations(xf, 128)
    acc_ref, y_ref, mag = oracle.gemv_dense_group_scales(W, S, q_ref, s_ref)
    Wd = bc.bitcos_pack(W, S).to_device()
    ws = bc.make_workspace(M, K)
    xd = dev_bf16(bits)
    for rep in range(2):
        y, acc = bc.bitcos_gemv_bf16(Wd, xd, acc_debug=(rep == 0) or None, workspace=ws)
        torch.cuda.synchronize()
        if acc is not None:
            assert np.array_equal(acc.cpu().numpy(), acc_ref), (M, K, B)
        yv = y.cpu().numpy().astype(np.float64)
        assert (np.abs(yv - y_ref) <= REL * mag).all(), (M, K, B, rep)
        assert (yv[mag == 0] == 0).all()
    assert bc.workspace_status(ws) == 0


def test_product_from_bf16_activations_large_and_multi(bc):
    """Two tiles per warp (a large matrix), and a layer's worth of jobs in fused launches."""
    M, K, B = 19200, 5120, 1
    W, S = datagen.trits(2500, M, K, 0.4219), datagen.scales(2500, M, K)
    bits = datagen.activations_bf16(2500, B, K)
    q_ref, s_ref = oracle.quantize_activations(datagen.bf16_bits_to_f32(bits), 128)
    rows = np.unique(np.concatenate([np.arange(0, M, M // 211), [M - 1, M - 32, M - 33, 31, 32, 63, 64]]))
    acc_ref, y_ref, mag = oracle.gemv_dense_group_scales(W[rows], S[rows], q_ref, s_ref)
    Wd = bc.bitcos_pack(W, S).to_device()
    y, acc = bc.bitcos_gemv_bf16(Wd, dev_bf16(bits), acc_debug=True)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy()[:, rows], acc_ref)
    assert (np.abs(y.cpu().numpy().astype(np.float64)[:, rows] - y_ref) <= REL * mag).all()
    del Wd
    for B in (1, 2):
        shapes = [(2560, 2560), (640, 2560), (640, 2560), (96, 6912), (33, 1280)]
        jobs, refs = [], []
        for i, (M, K) in enumerate(shapes):
            W, S = datagen.trits(2600 + i, M, K, 0.4219), datagen.scales(2600 + i, M, K)
            bits = datagen.activations_bf16(2600 + i + B, B, K)
            q_ref, s_ref = oracle.quantize_activations(datagen.bf16_bits_to_f32(bits), 128)
            refs.append(oracle.gemv_dense_group_scales(W, S, q_ref, s_ref))
            yj = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
            jobs.append((bc.bitcos_pack(W, S).to_device(), dev_bf16(bits), None, yj, bc.make_workspace(M, K)))
        for n in (5, 3, 1):
            for j in jobs:
                j[3].fill_(float("nan"))
            bc.bitcos_gemv_multi_bf16(jobs[:n])
            torch.cuda.synchronize()
            for (Wd, _, _, yj, ws), (_, y_ref, mag) in zip(jobs[:n], refs[:n]):
                assert (np.abs(yj.cpu().numpy().astype(np.float64) - y_ref) <= REL * mag).all(), (Wd.M, Wd.K, B, n)
                assert bc.workspace_status(ws) == 0


def test_product_from_bf16_activations_rejects_what_it_cannot_do(bc):
    W, S = datagen.trits(2700, 64, 256, 0.4), datagen.scales(2700, 64, 256)
    Wd = bc.bitcos_pack(W, S).to_device()
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_gemv_bf16(Wd, torch.zeros((3, 256), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == 2
    W, S = datagen.trits(2701, 32, 25600, 0.4), datagen.scales(2701, 32, 25600)
    Wl = bc.bitcos_pack(W, S).to_device()
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_gemv_bf16(Wl, torch.zeros((2, 25600), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == 2
    with pytest.raises(bc.BitcosError) as e:
        bc.bitcos_gemv_multi_bf16([(Wd, torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda"), None,
                                    torch.zeros((4, 64), dtype=torch.float32, device="cuda"), bc.make_workspace(64, 256))])
    assert e.value.status == 2


@pytest.mark.parametrize("B", [1, 2, 5, 16])
def test_multi_launch_with_group_scales(bc, B):
    shapes = [(2560, 2560), (640, 2560), (96, 6912), (320, 1280), (33, 2560)]
    jobs, refs = [], []
    for i, (M, K) in enumerate(shapes):
        W, S = datagen.trits(2800 + i, M, K, 0.4219), datagen.scales(2800 + i, M, K)
        x, _ = datagen.activations(2800 + i + B, B, K)
        G = K // 128
        xg = (0.001 * (1.0 + 19.0 * datagen.uniform(2800 + i, datagen.STREAM_XS, 0, B * G))).astype(np.float32).reshape(B, G)
        refs.append(oracle.gemv_dense_group_scales(W, S, x, xg))
        y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
        jobs.append((bc.bitcos_pack(W, S).to_device(), dev(x), dev(xg), y, bc.make_workspace(M, K)))
    for n in (5, 2):
        for j in jobs:
            j[3].fill_(float("nan"))
        bc.bitcos_gemv_multi_group_scales(jobs[:n])
        torch.cuda.synchronize()
        for (Wd, x, xg, y, ws), (_, y_ref, mag) in zip(jobs[:n], refs[:n]):
            assert (np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= REL * mag).all(), (Wd.M, Wd.K, B, n)
            y1, _ = bc.bitcos_gemv_group_scales(Wd, x, xg, workspace=ws)
            torch.cuda.synchronize()
            assert torch.equal(y1, y)
            assert bc.workspace_status(ws) == 0


def test_entry_points_inside_a_cuda_graph(bc):
    """Quantiser, products with group scales, from bf16 activations and the 16-bit variant captured
    into one CUDA graph (after a first eager call each, which does the one-time set-up) and
    replayed: the same bits as the eager calls."""
    M, K, B = 2560, 2560, 2
    W, S = datagen.trits(2900, M, K, 0.4219), datagen.scales(2900, M, K)
    Wd = bc.bitcos_pack(W, S).to_device()
    ws = bc.make_workspace(M, K)
    xb = dev_bf16(datagen.activations_bf16(2900, B, K))
    q = torch.empty((B, K), dtype=torch.int8, device="cuda")
    sg = torch.empty((B, K // 128), dtype=torch.float32, device="cuda")
    y1, y2, y3 = (torch.empty((B, M), dtype=torch.float32, device="cuda") for _ in range(3))

    def run():
        bc.bitcos_quantize_activations(xb, 128, xq=q, x_scale=sg)
        bc.bitcos_gemv_group_scales(Wd, q, sg, y=y1, workspace=ws)
        bc.bitcos_gemv_bf16(Wd, xb, y=y2, workspace=ws)
        bc.bitcos_gemv_blend_bf16(Wd, xb, y=y3, workspace=ws)

    run()
    torch.cuda.synchronize()
    eager = [t.clone() for t in (q, sg, y1, y2, y3)]
    assert torch.equal(y1, y2)                       # the fused product is the two-step chain, bit for bit
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            run()
        for rep in range(2):
            for t in (q, sg, y1, y2, y3):
                t.zero_()
            g.replay()
            stream.synchronize()
            for t, e in zip((q, sg, y1, y2, y3), eager):
                assert torch.equal(t, e), rep
    assert bc.workspace_status(ws) == 0
