/*
 * bitcos_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, obviously-correct CPU statement of what the BITCOS GEMV path computes,
 * written from the paper ("Breaking the 1.58-bit Barrier for Ternary LLMs") and used only
 * to check the CUDA library and as the timed CPU baseline.  It shares no source, header,
 * table or helper with the CUDA path and must never be called from it.
 *
 * What is an exact definition and what is an encoding:
 *   - The GEMV result is exactly the dense ternary dot product, so o_dense_acc / o_dense_y
 *     are that definition written out as a triple loop (int32 per group of 128, then a
 *     double-precision scale-and-sum).
 *   - The storage layouts (BITCOS, five-trit, 2-bit) are encodings: they follow the paper's
 *     steps (Section II-A; Fig. 4; Eq. 2; Eq. 4) bit by bit, with no popcount tricks, no
 *     blocking and no fusion.
 *
 * Parity pins (tests/test_oracle_*.py): the pdep example of Fig. 4, the column example of
 * Section II-C (0xDF / Eq. 3 and its byte arithmetic), the LUT entries 0xB6 and 0x66 of
 * Section II-D, the 8x8 example's 98 bits, B(z) = 2 - z, 26 bytes per 128-weight five-trit
 * block, Table I rows, 8.5 - 4z bytes per 32 weights, round trips, and brute-force dense
 * products on tiny inputs.  No function here is "parity unpinned".
 *
 * Readings where the paper is silent are listed next to each function.
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define O_GROUP 128      /* reduction elements per scale (Section III-B.2: group size 128) */
#define O_ROWS 32        /* output rows interleaved in one block, as the paper's 32-row panels */

#define O_OK 0
#define O_ERR_SHAPE (-1)
#define O_ERR_TRIT (-2)
#define O_ERR_CAPACITY (-3)
#define O_ERR_CODE (-4)
#define O_ERR_CURSOR (-5)

/* ------------------------------------------------------------------------------------
 * Bit deposit (the operation of Fig. 4): the low bits of `a` are handed out, one by one
 * and lowest first, to the positions where `mask` has a one; every other bit of the
 * result is zero.  Written here as a walk over the ones of the mask: take the lowest
 * one still standing, give it the next bit of `a`, strike it out.  Bit m of a word is
 * (word >> m) & 1, i.e. LSB first.
 * ---------------------------------------------------------------------------------- */
uint32_t o_pdep32(uint32_t a, uint32_t mask)
{
    uint32_t out = 0;
    uint32_t left = mask;
    while (left) {
        uint32_t lowest = left & (~left + 1u);     /* the lowest one of the mask, alone */
        if (a & 1u) out |= lowest;
        a >>= 1;
        left ^= lowest;
    }
    return out;
}

/* Eq. 2: w = p - 2n, with p the presence bit and n the "present and negative" bit. */
int o_ternary_from_pn(int p, int n)
{
    return p - 2 * n;
}

/* Section II-C byte arithmetic: P = -p and N = -n as bytes (0xFF / 0x00), T = N & 0xFE
 * (= -2n), W = T - P (byte subtraction) = p - 2n.  lanes = number of byte lanes. */
void o_avx2_bytes(const uint8_t *p, const uint8_t *n, int lanes, uint8_t *P, uint8_t *T, uint8_t *W)
{
    for (int i = 0; i < lanes; ++i) {
        P[i] = p[i] ? 0xFF : 0x00;
        uint8_t N = n[i] ? 0xFF : 0x00;
        T[i] = (uint8_t)(N & 0xFE);
        W[i] = (uint8_t)(T[i] - P[i]);
    }
}

/* Eq. 4: entry (m, s) of the 256-entry table.  m = four presence bits of rows 4g..4g+3,
 * s = the next four bits of the compact sign stream.  c_i = 0 if m_i = 0; +1 if m_i = 1 and
 * s_{r_i} = 0; -1 if m_i = 1 and s_{r_i} = 1, with r_i = sum_{j<i} m_j.  Returns the number
 * of sign bits consumed, popcount(m). */
int o_lut_entry(unsigned m, unsigned s, int8_t c[4])
{
    int r = 0;
    for (int i = 0; i < 4; ++i) {
        if ((m >> i) & 1u) {
            c[i] = ((s >> r) & 1u) ? -1 : +1;
            r = r + 1;
        } else {
            c[i] = 0;
        }
    }
    return r;
}

/* ------------------------------------------------------------------------------------
 * Section II-A: the layout of a stream of n ternary symbols given in tensor order:
 *   (1) presence bitmap, one bit per symbol, set where the symbol is non-zero;
 *   (2) sign vector, one bit per NON-ZERO symbol in the same order, so that the j-th sign
 *       bit belongs to the j-th set bit of the bitmap; a set sign bit means negative
 *       (Eq. 4: s = 1 -> -1).
 * Bit i of either vector is bit (i & 31) of 32-bit word (i >> 5).
 * bitmap must hold ceil(n/32) words, signs must hold sign_words words; both are zeroed
 * here so that padding bits are zero.  Returns the number of sign bits in *nnz.
 * ---------------------------------------------------------------------------------- */
int o_stream_pack(const int8_t *sym, uint64_t n, uint32_t *bitmap, uint32_t *signs,
                  uint64_t sign_words, uint64_t *nnz)
{
    memset(bitmap, 0, (size_t)((n + 31) / 32) * 4);
    memset(signs, 0, (size_t)sign_words * 4);
    uint64_t j = 0;
    for (uint64_t i = 0; i < n; ++i) {
        int w = sym[i];
        if (w != -1 && w != 0 && w != 1) return O_ERR_TRIT;
        if (w != 0) {
            bitmap[i >> 5] |= 1u << (i & 31);
            if ((j >> 5) >= sign_words) return O_ERR_CAPACITY;
            if (w < 0) signs[j >> 5] |= 1u << (j & 31);
            j = j + 1;
        }
    }
    *nnz = j;
    return O_OK;
}

/* Inverse of o_stream_pack, one bit at a time: walk the bitmap, and every time a set bit
 * is met take the next unread sign bit.  start_sign_bit is where this stream's first
 * nonzero sits in the sign vector (0 for a whole tensor, an entry offset for a block). */
void o_stream_unpack(const uint32_t *bitmap, uint64_t first_bit, uint64_t n, const uint32_t *signs,
                     uint64_t start_sign_bit, int8_t *sym, uint64_t *end_sign_bit)
{
    uint64_t j = start_sign_bit;
    for (uint64_t q = 0; q < n; ++q) {
        uint64_t i = first_bit + q;
        int p = (bitmap[i >> 5] >> (i & 31)) & 1u;
        int nbit = 0;
        if (p) {
            nbit = (signs[j >> 5] >> (j & 31)) & 1u;
            j = j + 1;
        }
        sym[q] = (int8_t)o_ternary_from_pn(p, nbit);
    }
    *end_sign_bit = j;
}

/* The x86 sequences of Section II-B / II-C for one 32-bit bitmap word: read a 64-bit
 * window of the sign vector at the 32-bit word that holds the cursor, shift it right by
 * (cursor & 31), deposit its low bits onto the set positions of the mask (pdep), form
 * w = p - 2n, and advance the cursor by the population count of the mask.
 * n = number of symbols, a multiple of 32.  signs must be readable one word past the
 * word holding the last sign bit. */
void o_stream_unpack_windowed(const uint32_t *bitmap, uint64_t first_word, uint64_t n_words,
                              const uint32_t *signs, uint64_t start_sign_bit, int8_t *sym,
                              uint64_t *end_sign_bit)
{
    uint64_t cursor = start_sign_bit;
    for (uint64_t q = 0; q < n_words; ++q) {
        uint32_t mask = bitmap[first_word + q];
        uint64_t word = cursor >> 5;
        uint64_t window64 = (uint64_t)signs[word] | ((uint64_t)signs[word + 1] << 32);
        uint32_t window = (uint32_t)(window64 >> (cursor & 31));
        uint32_t neg = o_pdep32(window, mask);
        int count = 0;
        for (int b = 0; b < 32; ++b) {
            int p = (mask >> b) & 1u;
            int nb = (neg >> b) & 1u;
            sym[q * 32 + b] = (int8_t)o_ternary_from_pn(p, nb);
            count += p;
        }
        cursor += (uint64_t)count;
    }
    *end_sign_bit = cursor;
}

/* The Xe2 sequence of Section II-D for one 32-bit bitmap word: align a window of the
 * sign vector at the cursor, then for each of the eight 4-symbol groups form the key
 * (presence nibble m, low four bits s of the running window), take the table entry of
 * Eq. 4, and shift the window right by popcount(m).  The block cursor advances by the
 * population count of the whole word. */
void o_stream_unpack_lut(const uint32_t *bitmap, uint64_t first_word, uint64_t n_words,
                         const uint32_t *signs, uint64_t start_sign_bit, int8_t *sym,
                         uint64_t *end_sign_bit)
{
    uint64_t rank = start_sign_bit;
    for (uint64_t q = 0; q < n_words; ++q) {
        uint32_t bmp = bitmap[first_word + q];
        uint64_t word = rank >> 5;
        unsigned b = (unsigned)(rank & 31);
        uint32_t lo = signs[word] >> b;
        uint32_t hi = (b == 0) ? 0u : (signs[word + 1] << ((32 - b) & 31));
        uint32_t window = lo | hi;
        int block_count = 0;
        for (int g = 0; g < 8; ++g) {
            unsigned m = (bmp >> (4 * g)) & 0xFu;
            unsigned s = window & 0xFu;
            int8_t c[4];
            int used = o_lut_entry(m, s, c);
            for (int i = 0; i < 4; ++i) sym[q * 32 + 4 * g + i] = c[i];
            window >>= used;
            block_count += used;
        }
        rank += (uint64_t)block_count;
    }
    *end_sign_bit = rank;
}

/* ------------------------------------------------------------------------------------
 * Tensor order used for an [M][K] weight matrix (M output rows, K reduction length,
 * K % 128 == 0).  The paper only requires the sign bits to follow the order of the tensor
 * and itself uses three orders
 * (32 rows per mask on AVX-512, 8 rows x 4 k on AVX2, 32 k per output column with
 * adjacent columns adjacent on Xe2).  Reading taken here: rows are taken in blocks of 32
 * (the last block padded with all-zero rows), the reduction in groups of 128; a "tile" is
 * one group of one row block.  Tiles are ordered row block major, group minor; inside a
 * tile the order is row major: row r of the block, then k ascending.  Stream position of
 * weight (m, k):
 *     pos = (((m / 32) * (K / 128) + k / 128) * 32 + m % 32) * 128 + k % 128.
 * Each tile's first sign bit is recorded in tile_off[tile] (the per-column entry points
 * into the sign vector of Fig. 8): tile_off has n_tiles + 1 entries, the last = nnz.
 * ---------------------------------------------------------------------------------- */
int64_t o_padded_rows(int64_t M) { return (M + O_ROWS - 1) / O_ROWS * O_ROWS; }
int64_t o_num_tiles(int64_t M, int64_t K) { return (o_padded_rows(M) / O_ROWS) * (K / O_GROUP); }

uint64_t o_tile_order_pos(int64_t M, int64_t K, int64_t m, int64_t k)
{
    (void)M;
    int64_t G = K / O_GROUP;
    return (uint64_t)((((m / O_ROWS) * G + k / O_GROUP) * O_ROWS + m % O_ROWS) * O_GROUP + k % O_GROUP);
}

/* Number of 32-bit words a sign buffer needs for nnz sign bits: the bits themselves rounded
 * up to 16 bytes, plus 32 bytes of zero slack so that a decoder may read a fixed-size
 * aligned window at the last cursor (the x86 sequences likewise read a 64-bit window).
 * The slack is not part of the bits-per-weight accounting. */
uint64_t o_sign_words(uint64_t nnz)
{
    uint64_t bytes = (nnz + 7) / 8;
    bytes = (bytes + 15) / 16 * 16 + 32;
    return bytes / 4;
}

uint64_t o_count_nnz(const int8_t *trits, int64_t M, int64_t K)
{
    uint64_t c = 0;
    for (int64_t i = 0; i < M * K; ++i) c += (trits[i] != 0);
    return c;
}

/* Gather the matrix into tensor order (padding rows are zero). out has Mp * K entries. */
void o_to_tile_order(const int8_t *trits, int64_t M, int64_t K, int8_t *out)
{
    int64_t Mp = o_padded_rows(M);
    memset(out, 0, (size_t)(Mp * K));
    for (int64_t m = 0; m < M; ++m)
        for (int64_t k = 0; k < K; ++k)
            out[o_tile_order_pos(M, K, m, k)] = trits[m * K + k];
}

void o_from_tile_order(const int8_t *in, int64_t M, int64_t K, int8_t *trits)
{
    for (int64_t m = 0; m < M; ++m)
        for (int64_t k = 0; k < K; ++k)
            trits[m * K + k] = in[o_tile_order_pos(M, K, m, k)];
}

/* BITCOS pack of an [M][K] matrix: bitmap (Mp*K/32 words), signs (o_sign_words(nnz) words),
 * tile_off (n_tiles + 1). */
int o_bitcos_pack(const int8_t *trits, int64_t M, int64_t K, uint32_t *bitmap, uint32_t *signs,
                  uint64_t sign_words, uint32_t *tile_off, uint64_t *nnz_out)
{
    if (M < 1 || K < O_GROUP || K % O_GROUP != 0) return O_ERR_SHAPE;
    int64_t Mp = o_padded_rows(M);
    int8_t *ordered = (int8_t *)malloc((size_t)(Mp * K));
    if (!ordered) return O_ERR_CAPACITY;
    o_to_tile_order(trits, M, K, ordered);
    uint64_t nnz = 0;
    int rc = o_stream_pack(ordered, (uint64_t)(Mp * K), bitmap, signs, sign_words, &nnz);
    if (rc == O_OK) {
        /* entry offsets: number of nonzeros that precede each tile in tensor order */
        int64_t T = o_num_tiles(M, K);
        uint64_t run = 0;
        for (int64_t t = 0; t < T; ++t) {
            tile_off[t] = (uint32_t)run;
            for (int64_t i = 0; i < O_ROWS * O_GROUP; ++i) run += (ordered[t * O_ROWS * O_GROUP + i] != 0);
        }
        tile_off[T] = (uint32_t)run;
        if (run != nnz || nnz > 0xFFFFFFFFull) rc = O_ERR_CURSOR;
        *nnz_out = nnz;
    }
    free(ordered);
    return rc;
}

/* decoder: 0 = bit at a time from the start of the stream, 1 = pdep windows (x86),
 * 2 = nibble table (Xe2), 3 = bit at a time, each tile entered at its own tile_off. */
int o_bitcos_unpack(const uint32_t *bitmap, const uint32_t *signs, const uint32_t *tile_off,
                    int64_t M, int64_t K, int decoder, int8_t *trits)
{
    if (M < 1 || K < O_GROUP || K % O_GROUP != 0) return O_ERR_SHAPE;
    int64_t Mp = o_padded_rows(M);
    int64_t T = o_num_tiles(M, K);
    uint64_t n = (uint64_t)(Mp * K);
    int8_t *ordered = (int8_t *)malloc((size_t)n);
    if (!ordered) return O_ERR_CAPACITY;
    uint64_t end = 0;
    int rc = O_OK;
    if (decoder == 0) {
        o_stream_unpack(bitmap, 0, n, signs, 0, ordered, &end);
    } else if (decoder == 1) {
        o_stream_unpack_windowed(bitmap, 0, n / 32, signs, 0, ordered, &end);
    } else if (decoder == 2) {
        o_stream_unpack_lut(bitmap, 0, n / 32, signs, 0, ordered, &end);
    } else {
        const uint64_t tile_syms = O_ROWS * O_GROUP;
        #pragma omp parallel for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            uint64_t e = 0;
            o_stream_unpack(bitmap, (uint64_t)t * tile_syms, tile_syms, signs, tile_off[t],
                            ordered + (uint64_t)t * tile_syms, &e);
            if (e != tile_off[t + 1]) {
                #pragma omp atomic write
                rc = O_ERR_CURSOR;
            }
        }
        end = tile_off[T];
    }
    if (end != tile_off[T]) rc = O_ERR_CURSOR;
    o_from_tile_order(ordered, M, K, trits);
    free(ordered);
    return rc;
}

/* Group scales in the same block order as the weights: scale of (row m, group g) sits at
 * ((m/32) * G + g) * 32 + m%32; padding rows get +0. bf16 bit patterns are copied as is. */
void o_scales_to_tile_order(const uint16_t *scales, int64_t M, int64_t K, uint16_t *tiled)
{
    int64_t G = K / O_GROUP, Mp = o_padded_rows(M);
    memset(tiled, 0, (size_t)(Mp * G) * 2);
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < G; ++g)
            tiled[((m / O_ROWS) * G + g) * O_ROWS + m % O_ROWS] = scales[m * G + g];
}

/* ------------------------------------------------------------------------------------
 * Five-trit packing (Section I: five trits per byte since 3^5 = 243 <= 256; a block of 128
 * weights needs ceil(128/5) = 26 bytes, i.e. 1.625 bits per weight).  The paper gives no
 * digit order; reading taken here: byte j of a block = sum_{i=0..4} (t[5j+i] + 1) * 3^i for
 * j = 0..24; byte 25 carries trits 125..127 in digits 0..2 and the digit value 1 (a zero
 * trit) in digits 3 and 4.  A block is 128 consecutive k of one row.  A row's blocks are
 * concatenated (26 * K/128 bytes, zero padded to a multiple of 4), read as little-endian
 * 32-bit words, and the words of the 32 rows of a row block are interleaved: word q of row
 * r of block rb is at 32-bit index (rb * WPR + q) * 32 + r, WPR = words per row.
 * ---------------------------------------------------------------------------------- */
void o_trit5_block_encode(const int8_t t[128], uint8_t out[26])
{
    for (int j = 0; j < 26; ++j) {
        int v = 0, pw = 1;
        for (int i = 0; i < 5; ++i) {
            int idx = 5 * j + i;
            int digit = (idx < 128) ? (t[idx] + 1) : 1;
            v += digit * pw;
            pw *= 3;
        }
        out[j] = (uint8_t)v;
    }
}

int o_trit5_block_decode(const uint8_t in[26], int8_t t[128])
{
    for (int j = 0; j < 26; ++j) {
        int v = in[j];
        if (v > 242) return O_ERR_CODE;
        for (int i = 0; i < 5; ++i) {
            int idx = 5 * j + i;
            int digit = v % 3;
            v /= 3;
            if (idx < 128) t[idx] = (int8_t)(digit - 1);
            else if (digit != 1) return O_ERR_CODE;
        }
    }
    return O_OK;
}

int64_t o_trit5_words_per_row(int64_t K) { return (26 * (K / O_GROUP) + 3) / 4; }
int64_t o_trit5_total_words(int64_t M, int64_t K) { return o_padded_rows(M) * o_trit5_words_per_row(K); }

int o_trit5_pack(const int8_t *trits, int64_t M, int64_t K, uint32_t *words)
{
    if (M < 1 || K < O_GROUP || K % O_GROUP != 0) return O_ERR_SHAPE;
    int64_t G = K / O_GROUP, WPR = o_trit5_words_per_row(K), Mp = o_padded_rows(M);
    uint8_t *rowbytes = (uint8_t *)malloc((size_t)(WPR * 4));
    int8_t zero[128];
    memset(zero, 0, sizeof zero);
    for (int64_t m = 0; m < Mp; ++m) {
        memset(rowbytes, 0, (size_t)(WPR * 4));
        for (int64_t g = 0; g < G; ++g) {
            const int8_t *src = (m < M) ? trits + m * K + g * O_GROUP : zero;
            for (int i = 0; i < 128; ++i)
                if (src[i] < -1 || src[i] > 1) { free(rowbytes); return O_ERR_TRIT; }
            o_trit5_block_encode(src, rowbytes + 26 * g);
        }
        for (int64_t q = 0; q < WPR; ++q) {
            uint32_t w = (uint32_t)rowbytes[4 * q] | ((uint32_t)rowbytes[4 * q + 1] << 8) |
                         ((uint32_t)rowbytes[4 * q + 2] << 16) | ((uint32_t)rowbytes[4 * q + 3] << 24);
            words[((m / O_ROWS) * WPR + q) * O_ROWS + m % O_ROWS] = w;
        }
    }
    free(rowbytes);
    return O_OK;
}

int o_trit5_unpack(const uint32_t *words, int64_t M, int64_t K, int8_t *trits)
{
    if (M < 1 || K < O_GROUP || K % O_GROUP != 0) return O_ERR_SHAPE;
    int64_t G = K / O_GROUP, WPR = o_trit5_words_per_row(K);
    int rc = O_OK;
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        uint8_t *rowbytes = (uint8_t *)malloc((size_t)(WPR * 4));
        for (int64_t q = 0; q < WPR; ++q) {
            uint32_t w = words[((m / O_ROWS) * WPR + q) * O_ROWS + m % O_ROWS];
            rowbytes[4 * q] = (uint8_t)w; rowbytes[4 * q + 1] = (uint8_t)(w >> 8);
            rowbytes[4 * q + 2] = (uint8_t)(w >> 16); rowbytes[4 * q + 3] = (uint8_t)(w >> 24);
        }
        for (int64_t g = 0; g < G; ++g)
            if (o_trit5_block_decode(rowbytes + 26 * g, trits + m * K + g * O_GROUP) != O_OK) {
                #pragma omp atomic write
                rc = O_ERR_CODE;
            }
        free(rowbytes);
    }
    return rc;
}

/* ------------------------------------------------------------------------------------
 * 2-bit packing (the paper's baseline format: 2.000 bits per weight; code assignment not
 * given).  Reading taken here: code = t + 1 in {0, 1, 2}, code 3 invalid.  16 weights per
 * 32-bit word; weight i (0..15) of a word occupies bits [8*(i%4) + 2*(i/4), +2), i.e. byte
 * b of the word holds weights b, 4+b, 8+b, 12+b.  A row is K/16 words; rows of a row block
 * are interleaved in 16-byte chunks: word j (0..3) of chunk c of row r of block rb sits at
 * 32-bit index ((rb * C + c) * 32 + r) * 4 + j, C = K / 64.
 * ---------------------------------------------------------------------------------- */
int64_t o_bit2_total_words(int64_t M, int64_t K) { return o_padded_rows(M) * (K / 16); }

static uint64_t o_bit2_word_index(int64_t K, int64_t m, int64_t w_in_row)
{
    int64_t C = K / 64, c = w_in_row / 4, j = w_in_row % 4;
    return (uint64_t)((((m / O_ROWS) * C + c) * O_ROWS + m % O_ROWS) * 4 + j);
}

int o_bit2_pack(const int8_t *trits, int64_t M, int64_t K, uint32_t *words)
{
    if (M < 1 || K < O_GROUP || K % O_GROUP != 0) return O_ERR_SHAPE;
    int64_t Mp = o_padded_rows(M);
    for (int64_t m = 0; m < Mp; ++m) {
        for (int64_t w = 0; w < K / 16; ++w) {
            uint32_t word = 0;
            for (int i = 0; i < 16; ++i) {
                int t = (m < M) ? trits[m * K + 16 * w + i] : 0;
                if (t < -1 || t > 1) return O_ERR_TRIT;
                uint32_t code = (uint32_t)(t + 1);
                word |= code << (8 * (i % 4) + 2 * (i / 4));
            }
            words[o_bit2_word_index(K, m, w)] = word;
        }
    }
    return O_OK;
}

int o_bit2_unpack(const uint32_t *words, int64_t M, int64_t K, int8_t *trits)
{
    if (M < 1 || K < O_GROUP || K % O_GROUP != 0) return O_ERR_SHAPE;
    int rc = O_OK;
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t w = 0; w < K / 16; ++w) {
            uint32_t word = words[o_bit2_word_index(K, m, w)];
            for (int i = 0; i < 16; ++i) {
                uint32_t code = (word >> (8 * (i % 4) + 2 * (i / 4))) & 3u;
                if (code == 3u) {
                    #pragma omp atomic write
                    rc = O_ERR_CODE;
                }
                trits[m * K + 16 * w + i] = (int8_t)((int)code - 1);
            }
        }
    }
    return rc;
}

/* ------------------------------------------------------------------------------------
 * The product.  W in {-1,0,+1}^{M x K}, x int8 [B][K], group scale S[m][g] bf16 >= 0,
 * per-token activation scale xs[b]:
 *     acc[b][m][g] = sum_{k in group g} W[m][k] * x[b][k]                      (int32)
 *     y[b][m]      = xs[b] * sum_g float(S[m][g]) * acc[b][m][g]
 * (Section II-C: integer path, int32 accumulation, group scale applied once per group.)
 * y is evaluated in double; mag[b][m] = |xs[b]| * sum_g |S * acc| is the magnitude the
 * fp32 tolerance is relative to.
 * ---------------------------------------------------------------------------------- */
static double o_bf16_to_double(uint16_t bits)
{
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

void o_dense_acc(const int8_t *W, const int8_t *x, int64_t M, int64_t K, int64_t B, int32_t *acc)
{
    int64_t G = K / O_GROUP;
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t b = 0; b < B; ++b)
            for (int64_t g = 0; g < G; ++g) {
                int32_t s = 0;
                for (int64_t k = g * O_GROUP; k < (g + 1) * O_GROUP; ++k)
                    s += (int32_t)W[m * K + k] * (int32_t)x[b * K + k];
                acc[(b * M + m) * G + g] = s;
            }
}

void o_dense_y(const int32_t *acc, const uint16_t *scales /* [M][G] bf16 */, const float *xs,
               int64_t M, int64_t K, int64_t B, double *y, double *mag)
{
    int64_t G = K / O_GROUP;
    for (int64_t b = 0; b < B; ++b)
        for (int64_t m = 0; m < M; ++m) {
            double s = 0.0, a = 0.0;
            for (int64_t g = 0; g < G; ++g) {
                double term = o_bf16_to_double(scales[m * G + g]) * (double)acc[(b * M + m) * G + g];
                s += term;
                a += fabs(term);
            }
            y[b * M + m] = (double)xs[b] * s;
            mag[b * M + m] = fabs((double)xs[b]) * a;
        }
}

/* Packed GEMV = decode the packed matrix back to dense trits, then the dense definition.
 * format: 0 = BITCOS (tile entry offsets), 1 = five-trit, 2 = 2-bit.  scales are [M][G]
 * row major.  Work buffers are allocated here. */
int o_gemv_packed(int format, const uint32_t *payload, const uint32_t *signs, const uint32_t *tile_off,
                  const uint16_t *scales, const int8_t *x, const float *xs, int64_t M, int64_t K,
                  int64_t B, int32_t *acc, double *y, double *mag)
{
    int8_t *W = (int8_t *)malloc((size_t)(M * K));
    if (!W) return O_ERR_CAPACITY;
    int rc;
    if (format == 0) rc = o_bitcos_unpack(payload, signs, tile_off, M, K, 3, W);
    else if (format == 1) rc = o_trit5_unpack(payload, M, K, W);
    else rc = o_bit2_unpack(payload, M, K, W);
    if (rc == O_OK) {
        o_dense_acc(W, x, M, K, B, acc);
        o_dense_y(acc, scales, xs, M, K, B, y, mag);
    }
    free(W);
    return rc;
}

int o_threads(void)
{
    int n = 1;
#ifdef _OPENMP
    #pragma omp parallel
    {
        #pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* Timing aid only (no arithmetic): limits the number of threads the loops above may use, so that
 * the same code can be timed on one core and on all of them.  n < 1 is ignored. */
void o_set_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
