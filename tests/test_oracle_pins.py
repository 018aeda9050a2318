"""Pins for the CPU oracle: values the paper prints, closed forms, invariants, brute force.

Every check here compares the oracle with something other than itself, so that a dropped
term, a wrong sign, a wrong bit order or a transposed index in the oracle fails a test.
No GPU and no product code is involved.
"""
import numpy as np
import pytest

import datagen
import oracle


def bits_lsb_first(bits):
    return sum(int(b) << i for i, b in enumerate(bits))


# --- Fig. 4: pdep ---------------------------------------------------------------------
def test_pdep_fig4_example(golden):
    g = golden("pdep_fig4.txt")
    mask = bits_lsb_first(g["mask"][0])
    a = bits_lsb_first(g["a"][0])
    dst = bits_lsb_first(g["dst"][0])
    assert (mask, a, dst) == (0x4D, 0x0D, 0x49)
    assert oracle.pdep32(a, mask) == dst


def test_pdep_identities_and_bruteforce():
    rng = np.random.default_rng(1)
    for _ in range(300):
        a, mask = (int(v) for v in rng.integers(0, 2**32, 2, dtype=np.uint64))
        # independent construction: list the set positions, hand the source bits out in order
        pos = [i for i in range(32) if (mask >> i) & 1]
        want = sum(((a >> j) & 1) << p for j, p in enumerate(pos))
        assert oracle.pdep32(a, mask) == want
        assert oracle.pdep32(a, 0xFFFFFFFF) == a
        assert oracle.pdep32(a, 0) == 0
        assert oracle.pdep32(0xFFFFFFFF, mask) == mask
        assert oracle.pdep32(a, mask) & ~mask == 0


# --- Section II-C: the column example, Eq. 2 and the byte arithmetic ---------------------
def test_column_example(golden):
    g = golden("column_example_sec2c.txt")
    values = np.array([int(v) for v in g["values"][0]], np.int8)
    p = [int(v) for v in g["p"][0]]
    n = [int(v) for v in g["n"][0]]
    stored = [int(v) for v in g["stored_signs"][0]]
    bitmap, signs, nnz = oracle.stream_pack(values)
    assert bitmap[0] == int(g["bitmap_hex"][0][0], 16) == 0xDF
    assert nnz == 7 == sum(p)
    assert signs[0] == bits_lsb_first(stored) == 0x30
    # recovering n from the stored bits is the deposit
    assert oracle.pdep32(int(signs[0]), int(bitmap[0])) == bits_lsb_first(n) == 0x50
    # Eq. 2 returns the column
    assert [oracle.ternary_from_pn(pi, ni) for pi, ni in zip(p, n)] == list(values)
    # byte arithmetic
    P, T, W = oracle.avx2_bytes(p, n)
    assert [f"{v:02X}" for v in P] == g["P_bytes"][0]
    assert [f"{v:02X}" for v in T] == g["T_bytes"][0]
    assert [f"{v:02X}" for v in W] == g["W_bytes"][0]
    assert list(W.view(np.int8)) == list(values)
    # the sign of row 6 is the sixth stored bit (index 5), not the seventh
    assert stored[5] == 1 and n[6] == 1
    for dec in ("bits", "pdep", "lut"):
        out, end = oracle.stream_unpack(bitmap, signs, 8, dec)
        assert list(out) == list(values) and end == 7


def test_eq2_truth_table():
    assert oracle.ternary_from_pn(0, 0) == 0
    assert oracle.ternary_from_pn(1, 0) == 1
    assert oracle.ternary_from_pn(1, 1) == -1


# --- Section II-D: the lookup table ---------------------------------------------------------
def test_lut_printed_entries(golden):
    g = golden("lut_entries_sec2d.txt")
    for key in ("B6", "66"):
        row = g[key][0]
        k = int(key, 16)
        c, used = oracle.lut_entry(k >> 4, k & 0xF)
        assert list(c) == [int(v) for v in row[:4]]
        assert used == int(row[4])
    assert int(g["entries"][0][0]) == 256


def test_lut_is_a_four_bit_deposit():
    live = set()
    for m in range(16):
        for s in range(16):
            c, used = oracle.lut_entry(m, s)
            n = oracle.pdep32(s, m)
            want = [((m >> i) & 1) - 2 * ((n >> i) & 1) for i in range(4)]
            assert list(c) == want
            assert used == bin(m).count("1")
            live.add((m, s & ((1 << used) - 1)))
    # sum over m of 2^popcount(m) = 3^4 distinct (mask, consumed sign bits) pairs
    assert len(live) == 81


# --- Section II-A: sizes -------------------------------------------------------------------
def test_8x8_example_bits(golden):
    g = golden("layout_8x8_fig2.txt")
    n, zeros = int(g["weights"][0][0]), int(g["zeros"][0][0])
    rng = np.random.default_rng(2)
    for _ in range(5):
        sym = np.zeros(n, np.int8)
        nz = rng.choice(n, n - zeros, replace=False)
        sym[nz] = rng.choice([-1, 1], n - zeros)
        bitmap, signs, nnz = oracle.stream_pack(sym)
        assert bitmap.size * 32 == int(g["presence_bits"][0][0])
        assert nnz == int(g["sign_bits"][0][0])
        bpw = (bitmap.size * 32 + nnz) / n
        assert round(bpw, 3) == float(g["bits_per_weight"][0][0])
        assert round(zeros / n, 3) == float(g["z"][0][0])
        for dec in ("bits", "pdep", "lut"):
            out, end = oracle.stream_unpack(bitmap, signs, n, dec)
            assert np.array_equal(out, sym) and end == nnz


def exact_density_matrix(M, K, z_percent, seed):
    n = M * K
    zeros = int(round(z_percent / 100.0 * n))
    rng = np.random.default_rng(seed)
    flat = rng.choice([-1, 1], n).astype(np.int8)
    flat[rng.choice(n, zeros, replace=False)] = 0
    return flat.reshape(M, K), zeros


def test_table1_rates(golden):
    g = golden("table1_rows.txt")
    M, K = 64, 6400                      # 409600 weights: 1/n is far below the table's rounding
    for i, (model, row) in enumerate(g.items()):
        zp, sym_b, bc_s, b2_s, red2, t5_s, red5 = (float(v) for v in row[0])
        W, zeros = exact_density_matrix(M, K, zp, 10 + i)
        pk = oracle.bitcos_pack(W)
        z_hat = zeros / (M * K)
        assert pk.nnz == M * K - zeros
        assert pk.bits_per_weight() == pytest.approx(2.0 - z_hat, abs=1e-12)          # Eq. 1
        assert abs(pk.bits_per_weight() - sym_b) <= 0.00051, model
        scale_bits = 16 * M * (K // 128)
        bitcos_total = (pk.bitmap.size * 32 + pk.nnz + scale_bits) / (M * K)
        assert abs(bitcos_total - bc_s) <= 0.00051, model
        t5_total = (oracle.trit5_pack(W).size * 32 + scale_bits) / (M * K)
        b2_total = (oracle.bit2_pack(W).size * 32 + scale_bits) / (M * K)
        assert t5_total == t5_s == 1.75 and b2_total == b2_s == 2.125
        assert abs(b2_total / bitcos_total - red2) <= 0.0051, model
        assert abs(t5_total / bitcos_total - red5) <= 0.0051, model


def test_break_even_and_bytes_per_32_weights():
    # five-trit break-even at z = 0.375; always below 2 bits
    M, K = 32, 1280
    W, zeros = exact_density_matrix(M, K, 37.5, 3)
    pk = oracle.bitcos_pack(W)
    assert pk.bits_per_weight() == 1.625 == oracle.trit5_pack(W).size * 32 / (M * K)
    # bytes read per 32 weights with a 16-bit scale per 128: 4 + 4(1-z) + 0.5 = 8.5 - 4z; 6.9 at z = 0.4
    W, zeros = exact_density_matrix(M, K, 40.0, 4)
    pk = oracle.bitcos_pack(W)
    per32 = (pk.bitmap.size * 4 + pk.nnz / 8 + 2 * M * (K // 128)) / (M * K / 32)
    assert per32 == pytest.approx(6.9, abs=1e-9)


# --- matrix layout: tensor order, entry offsets, decoders ---------------------------------------
@pytest.mark.parametrize("M,K", [(32, 128), (64, 256), (33, 128), (100, 384), (1, 128)])
def test_tile_order_is_a_bijection(M, K):
    Mp = oracle.padded_rows(M)
    assert Mp % 32 == 0 and 0 <= Mp - M < 32
    seen = np.zeros(Mp * K, bool)
    for m in range(Mp):
        for k in range(0, K, 7):
            seen[oracle.tile_order_pos(M, K, m, k)] = True
    pos = np.array([[oracle.tile_order_pos(M, K, m, k) for k in range(K)] for m in range(min(M, 40))])
    assert len(np.unique(pos)) == pos.size and pos.max() < Mp * K
    # inside a tile: row major, k ascending; tiles: row block major, group minor
    assert oracle.tile_order_pos(M, K, 0, 0) == 0
    assert oracle.tile_order_pos(M, K, 0, 127) == 127
    if Mp >= 2:
        assert oracle.tile_order_pos(M, K, 1, 0) == 128
    if K >= 256:
        assert oracle.tile_order_pos(M, K, 0, 128) == 32 * 128
    if Mp >= 64:
        assert oracle.tile_order_pos(M, K, 32, 0) == 32 * K


@pytest.mark.parametrize("M,K,z", [(32, 128, 0.42), (96, 512, 0.3), (40, 256, 0.515), (7, 128, 0.47)])
def test_round_trip_all_decoders(M, K, z):
    W = datagen.trits(5, M, K, z)
    pk = oracle.bitcos_pack(W)
    assert pk.nnz == np.count_nonzero(W)
    # offsets are the running number of nonzeros at each tile boundary
    Mp, G = oracle.padded_rows(M), K // 128
    Wp = np.zeros((Mp, K), np.int8)
    Wp[:M] = W
    per_tile = [np.count_nonzero(Wp[rb * 32:(rb + 1) * 32, g * 128:(g + 1) * 128])
                for rb in range(Mp // 32) for g in range(G)]
    assert list(pk.tile_off) == list(np.concatenate([[0], np.cumsum(per_tile)]))
    for dec in ("bits", "pdep", "lut", "tiles"):
        assert np.array_equal(oracle.bitcos_unpack(pk.bitmap, pk.signs, pk.tile_off, M, K, dec), W), dec
    # padding bits and slack words are zero
    assert pk.signs.size == oracle.sign_words(pk.nnz)
    assert pk.signs.size * 32 >= pk.nnz + 256 and pk.signs.size % 4 == 0
    tail = pk.nnz
    assert (int(pk.signs[tail // 32]) >> (tail % 32)) == 0 and not pk.signs[tail // 32 + 1:].any()


def test_first_weight_of_row_r_takes_the_right_sign():
    # one nonzero per row at k = 5, alternating sign: sign bit j belongs to row j of the tile
    M, K = 32, 128
    W = np.zeros((M, K), np.int8)
    W[:, 5] = np.where(np.arange(M) % 3 == 0, -1, 1)
    pk = oracle.bitcos_pack(W)
    assert pk.nnz == 32
    assert int(pk.signs[0]) == bits_lsb_first([1 if r % 3 == 0 else 0 for r in range(32)])
    assert all(int(pk.bitmap[4 * r]) == 1 << 5 for r in range(32))


def test_special_cases():
    M, K = 32, 256
    for fill, nnz in ((0, 0), (1, M * K), (-1, M * K)):
        W = np.full((M, K), fill, np.int8)
        pk = oracle.bitcos_pack(W)
        assert pk.nnz == nnz
        assert pk.bits_per_weight() == (2.0 if fill else 1.0)     # z = 0 -> 2 b/w, z = 1 -> 1 b/w
        if fill == -1:
            assert (pk.signs[:nnz // 32] == 0xFFFFFFFF).all()
        if fill == 1:
            assert not pk.signs.any()
        for dec in ("bits", "pdep", "lut", "tiles"):
            assert np.array_equal(oracle.bitcos_unpack(pk.bitmap, pk.signs, pk.tile_off, M, K, dec), W)
    for k in (0, 31, 32, 127, 128, K - 1):
        W = np.zeros((M, K), np.int8)
        W[3, k] = -1
        pk = oracle.bitcos_pack(W)
        word = (((0 * 2 + k // 128) * 32 + 3) * 128 + k % 128) // 32
        assert pk.bitmap[word] == 1 << (k % 32) and np.count_nonzero(pk.bitmap) == 1
        assert pk.signs[0] == 1 and pk.nnz == 1


def test_invalid_symbol_rejected():
    W = np.zeros((32, 128), np.int8)
    W[0, 0] = 2
    with pytest.raises(oracle.OracleError):
        oracle.bitcos_pack(W)
    with pytest.raises(oracle.OracleError):
        oracle.trit5_pack(W)
    with pytest.raises(oracle.OracleError):
        oracle.bit2_pack(W)


# --- five-trit and 2-bit ------------------------------------------------------------------------
def test_trit5_block_bytes():
    t = np.zeros(128, np.int8)
    assert list(oracle.trit5_block_encode(t)) == [121] * 26          # 1 + 3 + 9 + 27 + 81
    assert oracle.trit5_block_encode(t).size == 26                    # ceil(128 / 5)
    t[:] = -1
    b = oracle.trit5_block_encode(t)
    assert list(b[:25]) == [0] * 25 and b[25] == 27 + 81              # trits 125..127 = -1 (digit 0), digits 3, 4 = 1
    t[:] = 1
    b = oracle.trit5_block_encode(t)
    assert list(b[:25]) == [242] * 25 and b[25] == 2 + 6 + 18 + 27 + 81
    t[:] = 0
    t[0] = 1
    assert oracle.trit5_block_encode(t)[0] == 122
    t[:] = 0
    t[4] = 1
    assert oracle.trit5_block_encode(t)[0] == 1 + 3 + 9 + 27 + 162
    t[:] = 0
    t[127] = -1
    assert oracle.trit5_block_encode(t)[25] == 1 + 3 + 0 + 27 + 81


def test_trit5_all_byte_values_round_trip():
    # a block whose first 25 bytes walk through base-3 values; all 243 values appear over 10 blocks
    seen = set()
    for start in range(0, 243, 25):
        t = np.zeros(128, np.int8)
        for j in range(25):
            v = (start + j) % 243
            for i in range(5):
                t[5 * j + i] = v % 3 - 1
                v //= 3
        b = oracle.trit5_block_encode(t)
        seen.update(int(x) for x in b[:25])
        assert np.array_equal(oracle.trit5_block_decode(b), t)
    assert seen == set(range(243))
    bad = np.full(26, 121, np.uint8)
    bad[3] = 243
    with pytest.raises(oracle.OracleError):
        oracle.trit5_block_decode(bad)


def test_bit2_code_positions():
    M, K = 32, 128

    def word0(i, val):
        W = np.zeros((M, K), np.int8)
        W[0, i] = val
        return int(oracle.bit2_pack(W)[0])

    assert word0(0, 0) == 0x55555555
    assert word0(0, 1) == 0x55555556
    assert word0(0, -1) == 0x55555554
    assert word0(1, 1) == 0x55555655
    assert word0(4, 1) == 0x55555559
    assert word0(15, 1) == 0x95555555


@pytest.mark.parametrize("M,K", [(32, 128), (64, 384), (45, 256)])
def test_trit5_bit2_round_trip_and_sizes(M, K):
    W = datagen.trits(6, M, K, 0.4)
    Mp = oracle.padded_rows(M)
    t5 = oracle.trit5_pack(W)
    b2 = oracle.bit2_pack(W)
    assert t5.size * 4 == Mp * ((26 * (K // 128) + 3) // 4) * 4
    if (K // 128) % 2 == 0:
        assert t5.size * 4 == Mp * 26 * (K // 128)                    # 26 bytes per 128 weights
    assert b2.size * 32 == Mp * K * 2
    assert np.array_equal(oracle.trit5_unpack(t5, M, K), W)
    assert np.array_equal(oracle.bit2_unpack(b2, M, K), W)
    # row interleave: word 0 of row r of block 0 is at index r (five-trit) / 4r (2-bit)
    W2 = np.zeros((M, K), np.int8)
    W2[5, :5] = [1, 1, 1, 1, 1]
    assert oracle.trit5_pack(W2)[5] & 0xFF == 242
    W2[5, :] = 0
    W2[5, 0] = 1
    assert oracle.bit2_pack(W2)[4 * 5] == 0x55555556


# --- the product ------------------------------------------------------------------------------------
def test_dense_product_bruteforce_tiny():
    rng = np.random.default_rng(7)
    for M, K, B in ((3, 128, 1), (3, 256, 3), (5, 384, 2)):
        W = rng.integers(-1, 2, (M, K)).astype(np.int8)
        x = rng.integers(-128, 128, (B, K)).astype(np.int8)
        xs = rng.uniform(0.01, 0.04, B).astype(np.float32)
        S = datagen.scales(8, M, K)
        acc, y, mag = oracle.gemv_dense(W, S, x, xs)
        Sf = datagen.bf16_bits_to_f32(S).astype(np.float64)
        for b in range(B):
            for m in range(M):
                tot = 0.0
                for g in range(K // 128):
                    a = sum(int(W[m, k]) * int(x[b, k]) for k in range(128 * g, 128 * g + 128))
                    assert acc[b, m, g] == a
                    tot += Sf[m, g] * a
                assert y[b, m] == pytest.approx(float(xs[b]) * tot, rel=1e-14, abs=1e-300)
                assert mag[b, m] >= abs(y[b, m]) * (1 - 1e-12)


def test_dense_product_closed_forms():
    M, K = 4, 256
    x, xs = datagen.activations(9, 2, K)
    ones = np.full((M, K // 128), 0x3F80, np.uint16)                  # bf16 1.0
    for fill in (1, -1, 0):
        W = np.full((M, K), fill, np.int8)
        acc, y, _ = oracle.gemv_dense(W, ones, x, np.ones(2, np.float32))
        want = fill * x.astype(np.int64).reshape(2, 2, 128).sum(-1)
        assert np.array_equal(acc, np.broadcast_to(want[:, None, :], acc.shape))
        assert np.array_equal(y, np.broadcast_to(want.sum(-1)[:, None].astype(np.float64), y.shape))
    for k in (0, 127, 128, 255):
        W = np.zeros((M, K), np.int8)
        W[2, k] = -1
        acc, y, _ = oracle.gemv_dense(W, ones, x, np.ones(2, np.float32))
        assert acc[0, 2, k // 128] == -int(x[0, k]) and np.count_nonzero(acc[0]) == (x[0, k] != 0)
    # linearity in x (no int8 overflow: halves)
    W = datagen.trits(10, M, K, 0.4)
    x1 = (x // 2).astype(np.int8)
    x2 = (x - x1).astype(np.int8)
    a, _, _ = oracle.gemv_dense(W, ones, x, np.ones(2, np.float32))
    a1, _, _ = oracle.gemv_dense(W, ones, x1, np.ones(2, np.float32))
    a2, _, _ = oracle.gemv_dense(W, ones, x2, np.ones(2, np.float32))
    assert np.array_equal(a, a1 + a2)
    # x = -128 is accepted
    xm = np.full((1, K), -128, np.int8)
    a, _, _ = oracle.gemv_dense(np.ones((M, K), np.int8), ones, xm, np.ones(1, np.float32))
    assert (a == -128 * 128).all()
    # the activation scale multiplies the whole output
    S = datagen.scales(11, M, K)
    _, y1, _ = oracle.gemv_dense(W, S, x, np.array([1.0, 1.0], np.float32))
    _, y2, _ = oracle.gemv_dense(W, S, x, np.array([0.5, 2.0], np.float32))
    assert np.array_equal(y2[0], 0.5 * y1[0]) and np.array_equal(y2[1], 2.0 * y1[1])


@pytest.mark.parametrize("M,K,B,z", [(256, 512, 1, 0.42), (40, 384, 3, 0.33)])
def test_packed_formats_agree_with_dense(M, K, B, z):
    W = datagen.trits(12, M, K, z)
    S = datagen.scales(12, M, K)
    x, xs = datagen.activations(12, B, K)
    acc, y, mag = oracle.gemv_dense(W, S, x, xs)
    pk = oracle.bitcos_pack(W)
    for fmt, payload, signs, off in ((oracle.FORMAT_BITCOS, pk.bitmap, pk.signs, pk.tile_off),
                                     (oracle.FORMAT_TRIT5, oracle.trit5_pack(W), None, None),
                                     (oracle.FORMAT_BIT2, oracle.bit2_pack(W), None, None)):
        a2, y2, m2 = oracle.gemv_packed(fmt, payload, signs, off, S, x, xs, M, K)
        assert np.array_equal(a2, acc) and np.array_equal(y2, y) and np.array_equal(m2, mag)


def test_scales_tile_order():
    M, K = 40, 384
    S = datagen.scales(13, M, K)
    T = oracle.scales_to_tile_order(S, M, K)
    G = K // 128
    assert T.size == 64 * G
    for m in (0, 1, 31, 32, 39):
        for g in range(G):
            assert T[((m // 32) * G + g) * 32 + m % 32] == S[m, g]
    assert T.reshape(2, G, 32)[1, :, 8:].sum() == 0


def test_grouped_equals_independent_calls():
    E, M, K = 4, 32, 128
    Ws = [datagen.trits(20 + e, M, K, 0.33) for e in range(E)]
    Ss = [datagen.scales(20 + e, M, K) for e in range(E)]
    x, xs = datagen.activations(14, 3, K)
    pe, pr = [0, 2, 2, 3], [0, 0, 1, 2]
    acc, y, mag = oracle.grouped_dense(Ws, Ss, pe, pr, x, xs)
    for i, (e, r) in enumerate(zip(pe, pr)):
        a1, y1, _ = oracle.gemv_dense(Ws[e], Ss[e], x[r:r + 1], xs[r:r + 1])
        assert np.array_equal(acc[i], a1[0]) and np.array_equal(y[i], y1[0])


def test_generator_is_counter_based_and_has_the_stated_distribution():
    a = datagen.uniform(1, 0, 0, 1000)
    b = datagen.uniform(1, 0, 500, 10)
    assert np.array_equal(a[500:510], b) and (a >= 0).all() and (a < 1).all()
    W = datagen.trits(2, 512, 1024, 0.42)
    assert abs((W == 0).mean() - 0.42) < 0.005 and abs((W == 1).mean() - 0.29) < 0.005
    S = datagen.bf16_bits_to_f32(datagen.scales(2, 64, 1024))
    assert S.min() >= 0.0099 and S.max() <= 0.0501
    x, xs = datagen.activations(2, 4, 4096)
    assert x.min() >= -127 and x.max() <= 127 and (xs > 0).all()
    ids = datagen.expert_choices(2, 16, 128, 8)
    assert all(len(set(r)) == 8 for r in ids) and ids.min() >= 0 and ids.max() < 128


# --- Section II-C: activations quantised per group of 128, scales applied once per group ---------
def _bf16(vals):
    return datagen.bf16_bits_to_f32(datagen.f32_to_bf16_bits(np.asarray(vals, np.float32)))


def test_quantiser_worked_examples():
    """Two groups worked out by hand.  Largest magnitude 1: the factor is 127, and 0.5 lands on
    the tie 63.5, which goes to the even 64.  Largest magnitude 127: the factor is 1, the scale
    exactly 1, and the ties 0.5, 2.5, 126.5 go to the even 0, 2, 126, while 1.5 goes to 2."""
    x = np.zeros((2, 128), np.float32)
    x[0, :7] = [1.0, -0.5, 0.25, 0.0, 1.0 / 256, -1.0, 0.75]
    x[1, 5:13] = [127.0, 0.5, 1.5, 2.5, -2.5, 126.5, -0.5, -1.5]
    assert np.array_equal(_bf16(x), x)                    # all of them are bf16 values
    q, s = oracle.quantize_activations(x)
    assert q.dtype == np.int8 and s.dtype == np.float32 and s.shape == (2, 1)
    assert q[0, :7].tolist() == [127, -64, 32, 0, 0, -127, 95] and not q[0, 7:].any()
    assert q[1, 5:13].tolist() == [127, 0, 2, 2, -2, 126, 0, -2] and not q[1, :5].any() and not q[1, 13:].any()
    assert s[1, 0] == np.float32(1.0)
    assert s[0, 0] == np.float32(1.0) / np.float32(127.0) and abs(float(s[0, 0]) * 127 - 1) < 2.0 ** -23


def _round_to_f32(fr):
    """Nearest float32 (ties to even) of a rational of normal magnitude, in exact arithmetic."""
    from fractions import Fraction
    if fr == 0:
        return Fraction(0)
    e = 0
    a = abs(fr)
    while a >= 2:
        a /= 2
        e += 1
    while a < 1:
        a *= 2
        e -= 1
    quantum = Fraction(2) ** (e - 23)
    return round(fr / quantum) * quantum               # round() of a Fraction: ties to even


def test_quantiser_against_exact_rational_arithmetic():
    """The stated rule carried out in exact rationals with explicit roundings, element by
    element, on a few groups (with outliers, a tiny group and an all-zero group)."""
    from fractions import Fraction
    x = datagen.bf16_bits_to_f32(datagen.activations_bf16(31, 3, 256))
    x[1, 128:] *= np.float32(2.0 ** -60)
    x[2, :128] = 0
    q, s = oracle.quantize_activations(x)
    for b in range(3):
        for g in range(2):
            grp = [Fraction(float(v)) for v in x[b, 128 * g:128 * g + 128]]
            a = max(max(abs(v) for v in grp), Fraction(2) ** -100)
            scale = _round_to_f32(a / 127)
            inv = _round_to_f32(Fraction(127) / a)
            assert Fraction(float(s[b, g])) == scale
            for k, v in enumerate(grp):
                code = round(_round_to_f32(v * inv))
                assert -127 <= code <= 127
                assert int(q[b, 128 * g + k]) == code, (b, g, k)
    assert not q[2, :128].any() and Fraction(float(s[2, 0])) == _round_to_f32(Fraction(2) ** -100 / 127)


def test_quantiser_invariants():
    B, K = 4, 1024
    x = datagen.bf16_bits_to_f32(datagen.activations_bf16(32, B, K))
    for group in (128, 0):
        q, s = oracle.quantize_activations(x, group)
        sg = s.reshape(B, -1)
        gs = K // sg.shape[1]
        xg, qg = x.reshape(B, -1, gs), q.reshape(B, -1, gs).astype(np.float64)
        # reconstruction error at most half a step (plus the rounding of the float32 factor)
        err = np.abs(xg.astype(np.float64) - qg * sg[:, :, None].astype(np.float64))
        assert (err <= 0.5 * sg[:, :, None] * (1 + 2.0 ** -14)).all()
        # the largest magnitude of every group gets code +-127, with its sign
        am = np.abs(xg).argmax(axis=2)
        top = np.take_along_axis(qg, am[:, :, None], 2)[:, :, 0]
        assert np.array_equal(top, 127 * np.sign(np.take_along_axis(xg, am[:, :, None], 2)[:, :, 0]))
        assert np.abs(q.astype(np.int32)).max() == 127
        # odd symmetry, and scaling by a power of two moves only the scale
        q2, s2 = oracle.quantize_activations(-x, group)
        assert np.array_equal(q2, -q) and np.array_equal(s2, s)
        q3, s3 = oracle.quantize_activations(x * np.float32(2.0 ** -9), group)
        assert np.array_equal(q3, q) and np.array_equal(s3, s * np.float32(2.0 ** -9))
    # groups do not see each other: swapping two groups swaps their codes and scales
    q, s = oracle.quantize_activations(x)
    xs = x.copy()
    xs[:, 0:128], xs[:, 256:384] = x[:, 256:384], x[:, 0:128]
    q4, s4 = oracle.quantize_activations(xs)
    assert np.array_equal(q4[:, 0:128], q[:, 256:384]) and np.array_equal(s4[:, 0], s[:, 2])
    assert np.array_equal(q4[:, 128:256], q[:, 128:256])
    # one scale per token = one group as long as the row
    q5, s5 = oracle.quantize_activations(x[:, :128], 0)
    assert np.array_equal(q5, q[:, :128]) and np.array_equal(s5, s[:, 0])
    with pytest.raises(ValueError):
        oracle.quantize_activations(x[:, :100])


def test_group_scale_product_bruteforce_and_special_cases():
    rng = np.random.default_rng(33)
    M, K, B = 5, 384, 2
    G = K // 128
    W = rng.integers(-1, 2, (M, K)).astype(np.int8)
    S = datagen.scales(33, M, K)
    Sf = datagen.bf16_bits_to_f32(S).astype(np.float64)
    x = rng.integers(-127, 128, (B, K)).astype(np.int8)
    xg = rng.uniform(0.001, 0.05, (B, G)).astype(np.float32)
    acc, y, mag = oracle.gemv_dense_group_scales(W, S, x, xg)
    for b in range(B):
        for m in range(M):
            tot, tot_abs = 0.0, 0.0
            for g in range(G):
                a = sum(int(W[m, k]) * int(x[b, k]) for k in range(128 * g, 128 * g + 128))
                assert acc[b, m, g] == a
                tot += Sf[m, g] * float(xg[b, g]) * a
                tot_abs += abs(Sf[m, g] * float(xg[b, g]) * a)
            assert y[b, m] == pytest.approx(tot, rel=1e-13, abs=1e-300)
            assert mag[b, m] == pytest.approx(tot_abs, rel=1e-13)
    # as a dense float64 matrix product of the two de-quantised operands
    Wd = W.astype(np.float64) * np.repeat(Sf, 128, axis=1)
    xd = x.astype(np.float64) * np.repeat(xg.astype(np.float64), 128, axis=1)
    assert np.allclose(y, xd @ Wd.T, rtol=0, atol=1e-12 * mag.max())
    # the same scale in every group: the per-token product
    xs = np.array([0.02, 0.007], np.float32)
    _, y1, m1 = oracle.gemv_dense(W, S, x, xs)
    _, y2, m2 = oracle.gemv_dense_group_scales(W, S, x, np.repeat(xs[:, None], G, axis=1))
    assert np.allclose(y1, y2, rtol=0, atol=1e-13 * m1.max()) and np.allclose(m1, m2, rtol=1e-13)
    # a scale of zero removes its group; scaling one group's scale scales that group's term
    xz = xg.copy()
    xz[:, 1] = 0
    _, y3, _ = oracle.gemv_dense_group_scales(W, S, x, xz)
    x0 = x.copy()
    x0[:, 128:256] = 0
    _, y4, _ = oracle.gemv_dense_group_scales(W, S, x0, xg)
    assert np.allclose(y3, y4, rtol=0, atol=1e-13 * mag.max())


def test_quantised_product_stays_within_the_quantisation_bound():
    """Quantise, multiply, compare with the product of the unquantised activations: every
    weight of a group contributes an error of at most half a quantisation step."""
    M, K, B = 64, 1024, 3
    W = datagen.trits(34, M, K, 0.42)
    S = datagen.scales(34, M, K)
    Sf = datagen.bf16_bits_to_f32(S).astype(np.float64)
    x = datagen.bf16_bits_to_f32(datagen.activations_bf16(34, B, K))
    exact = x.astype(np.float64) @ (W.astype(np.float64) * np.repeat(Sf, 128, axis=1)).T
    nnz = np.abs(W).reshape(M, K // 128, 128).sum(axis=2).astype(np.float64)
    errs = {}
    for group in (128, 0):
        q, s = oracle.quantize_activations(x, group)
        sg = s.reshape(B, -1) if group else np.repeat(s[:, None], K // 128, axis=1)
        _, y, _ = oracle.gemv_dense_group_scales(W, S, q, sg)
        bound = 0.5 * (1 + 2.0 ** -14) * np.einsum("mg,bg->bm", Sf * nnz, sg.astype(np.float64))
        assert (np.abs(y - exact) <= bound + 1e-12).all()
        errs[group] = np.sqrt(np.mean((y - exact) ** 2))
    # with outlier channels, scales per group lose less than one scale per token
    assert errs[128] < errs[0]


# --- Sections II-B / II-D: weights rebuilt as +-s, multiplied with unquantised 16-bit activations ---
def test_blend_product_bruteforce_and_cross_checks():
    rng = np.random.default_rng(35)
    M, K, B = 4, 256, 2
    W = rng.integers(-1, 2, (M, K)).astype(np.int8)
    S = datagen.scales(35, M, K)
    Sf = datagen.bf16_bits_to_f32(S).astype(np.float64)
    x = datagen.bf16_bits_to_f32(datagen.activations_bf16(35, B, K)).astype(np.float64)
    y, mag = oracle.gemv_dense_blend(W, S, x)
    for b in range(B):
        for m in range(M):
            tot = sum(int(W[m, k]) * Sf[m, k // 128] * x[b, k] for k in range(K))
            tot_abs = sum(abs(int(W[m, k]) * Sf[m, k // 128] * x[b, k]) for k in range(K))
            assert y[b, m] == pytest.approx(tot, rel=1e-12, abs=1e-300)
            assert mag[b, m] == pytest.approx(tot_abs, rel=1e-12)
    # as a library matrix product
    assert np.allclose(y, x @ (W.astype(np.float64) * np.repeat(Sf, 128, axis=1)).T, rtol=0, atol=1e-12 * mag.max())
    # activations that are small integers times a power of two are 16-bit values and int8 codes at
    # once: then this product is the integer path's (pinned on its own), with that power as the scale
    q, _ = datagen.activations(36, B, K)
    xq = q.astype(np.float64) * 2.0 ** -7
    assert np.array_equal(datagen.bf16_bits_to_f32(datagen.f32_to_bf16_bits(xq.astype(np.float32))).astype(np.float64), xq)
    y2, m2 = oracle.gemv_dense_blend(W, S, xq)
    _, y_int, m_int = oracle.gemv_dense(W, S, q, np.full(B, 2.0 ** -7, np.float32))
    assert np.allclose(y2, y_int, rtol=0, atol=1e-12 * m2.max())
    assert (m2 >= m_int * (1 - 1e-12)).all()          # |sum over a group| <= sum of |terms|
    # closed forms: all +1 with unit scales sums the activations; a single -1 picks one of them
    ones = np.full((M, K // 128), 0x3F80, np.uint16)
    y3, _ = oracle.gemv_dense_blend(np.ones((M, K), np.int8), ones, x)
    assert np.allclose(y3, np.repeat(x.sum(axis=1)[:, None], M, axis=1), rtol=1e-13)
    Wz = np.zeros((M, K), np.int8)
    Wz[1, 200] = -1
    y4, m4 = oracle.gemv_dense_blend(Wz, S, x)
    assert np.array_equal(y4[:, 1], -Sf[1, 1] * x[:, 200]) and not y4[:, [0, 2, 3]].any() and np.array_equal(m4, np.abs(y4))


# --- row interleave of the two baseline layouts away from the first row block and the first word -----
def test_trit5_word_lands_at_the_hand_computed_index_in_a_later_row_block():
    """Row 70 = row block 2, lane 6; k = 130 = block 1 of the row, trit 2 of that block.  A 256-wide row
    holds 52 bytes = 13 words (WPR); byte 26 opens block 1 and sits in word 6 at byte position 2.
    Word q of row 32 rb + r is stored at (rb * WPR + q) * 32 + r = (2 * 13 + 6) * 32 + 6 = 1030.
    An all-zero block byte is 1 + 3 + 9 + 27 + 81 = 121 (every digit holds trit + 1 = 1, and the 26th
    byte pads its two unused places with digit 1); trit +1 in digit 2 adds 9: 130."""
    M, K = 96, 256
    W = np.zeros((M, K), dtype=np.int8)
    zero_words = oracle.trit5_pack(W)
    W[70, 130] = 1
    words = oracle.trit5_pack(W)
    assert words.size == 3 * 13 * 32
    changed = np.flatnonzero(words != zero_words)
    assert changed.tolist() == [1030]
    assert int(words[1030]) == 121 | (121 << 8) | (130 << 16) | (121 << 24)
    assert int(zero_words[1030]) == 121 * 0x01010101


def test_bit2_word_lands_at_the_hand_computed_index_in_a_later_row_block():
    """Row 70 = row block 2, lane 6; k = 130 = word 8 of the row (weight 2 of it), i.e. 16-byte chunk 2,
    word 0.  Word j of chunk c of row 32 rb + r is stored at ((rb * (K / 64) + c) * 32 + r) * 4 + j
    = ((2 * 4 + 2) * 32 + 6) * 4 = 1304.  Code = trit + 1, weight i at bits [8 (i % 4) + 2 (i / 4), + 2):
    weight 2 sits at bits 16..17, where +1 turns code 01 into 10."""
    M, K = 96, 256
    W = np.zeros((M, K), dtype=np.int8)
    zero_words = oracle.bit2_pack(W)
    assert (zero_words == 0x55555555).all()
    W[70, 130] = 1
    words = oracle.bit2_pack(W)
    changed = np.flatnonzero(words != zero_words)
    assert changed.tolist() == [1304]
    assert int(words[1304]) == 0x55565555
    W[70, 130] = -1
    assert int(oracle.bit2_pack(W)[1304]) == 0x55545555
