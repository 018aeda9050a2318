"""GPU parity of every BITCOS decoder the library carries (the decode-rate probe runs each of them
on real packed tiles and hands the int32 group accumulators back): bit-exact against the oracle's
dense accumulators, on zero densities from all-non-zero to all-zero and on the edge patterns."""
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


def tile_accumulators(W, x_groups):
    """acc[t][r] of tile t = (row block t // G, group t % G) against x_groups[t] (brute force through
    the oracle's dense product on the one group)."""
    M, K = W.shape
    G = K // 128
    out = np.zeros((M // 32 * G, 32), dtype=np.int32)
    S = np.full((M, G), 0x3F80, dtype=np.uint16)
    for t in range(out.shape[0]):
        rb, g = divmod(t, G)
        x = np.zeros((1, K), dtype=np.int8)
        x[0, 128 * g:128 * g + 128] = x_groups[t]
        acc, _, _ = oracle.gemv_dense(W[32 * rb:32 * rb + 32], S[32 * rb:32 * rb + 32], x, np.ones(1, dtype=np.float32))
        out[t] = acc[0, :, g]
    return out


def special_matrix(seed, M, K):
    """Row blocks with the degenerate patterns: all +1, all -1, all zero, single non-zeros, dense
    alternating signs, and random fill at several densities."""
    rng = np.random.default_rng(seed)
    W = np.zeros((M, K), dtype=np.int8)
    W[0:32] = 1
    W[32:64] = -1
    W[96:128] = np.where(np.arange(K) % 2 == 0, 1, -1).astype(np.int8)
    for i, k in enumerate((0, 31, 32, 127, 128, K - 1)):
        W[128 + i, k] = -1 if i % 2 else 1
    for i, z in enumerate((0.05, 0.3, 0.5, 0.9, 0.99)):
        rows = slice(160 + 32 * i, 192 + 32 * i)
        u = rng.random((32, K))
        W[rows] = np.where(u < z, 0, np.where(rng.random((32, K)) < 0.5, 1, -1))
    return W


@pytest.mark.parametrize("variant", range(8))
def test_every_decoder_matches_the_oracle(bc, variant):
    for case, (M, K) in enumerate(((320, 384), (64, 1024))):
        W = special_matrix(100 + case, M, K) if case == 0 else datagen.trits(77, M, K, 0.42)
        S = datagen.scales(78, M, K)
        Wd = bc.bitcos_pack(W, S).to_device()
        G = K // 128
        n_all = M // 32 * G
        rng = np.random.default_rng(5 + case)
        xg = rng.integers(-128, 128, size=(n_all, 128), dtype=np.int64).astype(np.int8)
        ref = tile_accumulators(W, xg)
        for first, n in ((0, min(20, n_all)), (3, min(7, n_all - 3)), (n_all - 1, 1), (max(0, n_all - 32), min(32, n_all))):
            x = torch.from_numpy(np.ascontiguousarray(xg[first:first + n])).cuda()
            gamma, acc = bc.bitcos_decode_probe_variant(variant, Wd, first, n, x, 3, 2, want_acc=True)
            assert gamma > 0
            assert np.array_equal(acc.cpu().numpy(), ref[first:first + n]), (bc.PROBE_VARIANTS[variant], case, first, n)
