// Host-side packers of the BITCOS library: dense trits + bf16 group scales -> the three
// device layouts declared in bitcos.h (and back).  Plain C++17, no CUDA.
//
// BITCOS (paper Section II-A): a presence bitmap with one bit per weight and a sign vector
// with one bit per non-zero weight in the same order.  The order used here interleaves 32
// output rows per block, as the paper's own kernels do (Fig. 2; Section II-D), and records
// where each (row block, group) tile enters the sign vector.
#include "bitcos.h"

#include <cmath>
#include <cstring>
#include <vector>

namespace {

constexpr int64_t kGroup = BITCOS_GROUP;
constexpr int64_t kRows = BITCOS_TILE_ROWS;

inline int64_t padded_rows(int64_t M) { return (M + kRows - 1) / kRows * kRows; }
inline bool shape_ok(int64_t M, int64_t K) { return M >= 1 && K >= kGroup && K % kGroup == 0; }

inline size_t sign_bytes_for(uint64_t nnz) {
    uint64_t b = (nnz + 7) / 8;
    b = (b + 15) / 16 * 16 + 32;
    return static_cast<size_t>(b);
}

// Appends `count` bits (the low bits of `bits`, count <= 32) to a little-endian bit stream.
struct BitWriter {
    uint32_t *words;
    uint64_t pos = 0;
    void put(uint32_t bits, int count) {
        if (count == 0) return;
        const uint64_t w = pos >> 5;
        const int sh = static_cast<int>(pos & 31);
        const uint64_t v = static_cast<uint64_t>(bits) << sh;
        words[w] |= static_cast<uint32_t>(v);
        if (sh + count > 32) words[w + 1] |= static_cast<uint32_t>(v >> 32);
        pos += static_cast<uint64_t>(count);
    }
};

// Presence word and negative word (lane order) of 32 consecutive trits; false on a bad value.
inline bool masks_of(const int8_t *t, uint32_t &present, uint32_t &negative) {
    uint32_t p = 0, n = 0;
    for (int i = 0; i < 32; ++i) {
        const int v = t[i];
        if (v < -1 || v > 1) return false;
        p |= static_cast<uint32_t>(v != 0) << i;
        n |= static_cast<uint32_t>(v < 0) << i;
    }
    present = p;
    negative = n;
    return true;
}

// Gathers the bits of `src` selected by `mask` into the low bits of the result (compaction
// of the negative mask into sign-vector order).
inline uint32_t compact_bits(uint32_t src, uint32_t mask) {
    uint32_t out = 0;
    int k = 0;
    while (mask) {
        const uint32_t low = mask & (0u - mask);
        out |= static_cast<uint32_t>((src & low) != 0) << k;
        ++k;
        mask &= mask - 1;
    }
    return out;
}

// Spreads the low bits of `src` onto the set positions of `mask` (Fig. 4).
inline uint32_t deposit_bits(uint32_t src, uint32_t mask) {
    uint32_t out = 0;
    while (mask) {
        const uint32_t low = mask & (0u - mask);
        if (src & 1u) out |= low;
        src >>= 1;
        mask &= mask - 1;
    }
    return out;
}

inline bool scale_ok(uint16_t bits) {
    if (bits & 0x8000u) return false;                 // negative (or -0)
    return (bits & 0x7F80u) != 0x7F80u;               // exponent all ones: Inf / NaN
}

}  // namespace

extern "C" {

const char *bitcos_status_string(int status) {
    switch (status) {
        case BITCOS_OK: return "ok";
        case BITCOS_ERR_NULL: return "null pointer";
        case BITCOS_ERR_SHAPE: return "bad shape";
        case BITCOS_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case BITCOS_ERR_TRIT: return "weight or packed code out of range";
        case BITCOS_ERR_SCALE: return "scale is negative or not finite";
        case BITCOS_ERR_CAPACITY: return "buffer too small";
        case BITCOS_ERR_OVERFLOW: return "too many non-zero weights";
        case BITCOS_ERR_CUDA: return "CUDA error";
        default: return "unknown status";
    }
}

int bitcos_pack_sizes(int64_t M, int64_t K, uint64_t nnz, size_t *bitmap_bytes, size_t *sign_bytes,
                      size_t *tile_off_bytes, size_t *scale_bytes) {
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t Mp = padded_rows(M), G = K / kGroup;
    if (nnz > static_cast<uint64_t>(Mp) * static_cast<uint64_t>(K)) return BITCOS_ERR_SHAPE;
    if (nnz > 0xFFFFFFFFull) return BITCOS_ERR_OVERFLOW;
    if (bitmap_bytes) *bitmap_bytes = static_cast<size_t>(Mp * K / 8);
    if (sign_bytes) *sign_bytes = sign_bytes_for(nnz);
    if (tile_off_bytes) *tile_off_bytes = (static_cast<size_t>((Mp / kRows) * G + 1) * 4 + 15) / 16 * 16;
    if (scale_bytes) *scale_bytes = static_cast<size_t>(Mp * G) * 2;
    return BITCOS_OK;
}

int bitcos_choose_format(int64_t M, int64_t K, uint64_t nnz, int *format, size_t *bitcos_bytes, size_t *trit5_bytes) {
    if (!format) return BITCOS_ERR_NULL;
    size_t bm = 0, sg = 0, off = 0, t5 = 0;
    int rc = bitcos_pack_sizes(M, K, nnz, &bm, &sg, &off, nullptr);
    if (rc) return rc;
    rc = trit5_pack_sizes(M, K, &t5);
    if (rc) return rc;
    // what a product reads: the sign bits themselves (not the vector's alignment slack) and the
    // entry offsets without their padding; the scales are the same in both formats
    const size_t n_tiles = static_cast<size_t>(padded_rows(M) / kRows) * static_cast<size_t>(K / kGroup);
    const size_t bc = bm + static_cast<size_t>((nnz + 7) / 8) + (n_tiles + 1) * 4;
    (void)sg;
    (void)off;
    *format = bc <= t5 ? 0 : 1;
    if (bitcos_bytes) *bitcos_bytes = bc;
    if (trit5_bytes) *trit5_bytes = t5;
    return BITCOS_OK;
}

int bitcos_count_nnz(const int8_t *trits, int64_t M, int64_t K, uint64_t *nnz) {
    if (!trits || !nnz) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    uint64_t c = 0;
    bool bad = false;
    const int64_t n = M * K;
#pragma omp parallel for reduction(+ : c) reduction(|| : bad) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        const int v = trits[i];
        bad = bad || v < -1 || v > 1;
        c += (v != 0);
    }
    if (bad) return BITCOS_ERR_TRIT;
    *nnz = c;
    return BITCOS_OK;
}

int bitcos_scales_tile(const uint16_t *scales, int64_t M, int64_t K, uint16_t *tiled) {
    if (!scales || !tiled) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t Mp = padded_rows(M), G = K / kGroup;
    for (int64_t i = 0; i < M * G; ++i)
        if (!scale_ok(scales[i])) return BITCOS_ERR_SCALE;
    std::memset(tiled, 0, static_cast<size_t>(Mp * G) * 2);
    for (int64_t rb = 0; rb < Mp / kRows; ++rb)
        for (int64_t g = 0; g < G; ++g)
            for (int64_t r = 0; r < kRows; ++r) {
                const int64_t m = rb * kRows + r;
                if (m < M) tiled[(rb * G + g) * kRows + r] = scales[m * G + g];
            }
    return BITCOS_OK;
}

int bitcos_scales_untile(const uint16_t *tiled, int64_t M, int64_t K, uint16_t *scales) {
    if (!scales || !tiled) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t G = K / kGroup;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < G; ++g)
            scales[m * G + g] = tiled[((m / kRows) * G + g) * kRows + m % kRows];
    return BITCOS_OK;
}

int bitcos_pack(const int8_t *trits, const uint16_t *scales_bf16, int64_t M, int64_t K, uint32_t *bitmap,
                uint32_t *signs, size_t sign_capacity_bytes, uint32_t *tile_off, uint16_t *scales_tiled,
                uint64_t *nnz_out) {
    if (!trits || !scales_bf16 || !bitmap || !signs || !tile_off || !scales_tiled) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t Mp = padded_rows(M), G = K / kGroup, RB = Mp / kRows, T = RB * G;

    int rc = bitcos_scales_tile(scales_bf16, M, K, scales_tiled);
    if (rc != BITCOS_OK) return rc;

    // Pass 1: bitmap words, and per tile the number of non-zeros.
    std::vector<uint32_t> tile_count(static_cast<size_t>(T), 0);
    bool bad = false;
#pragma omp parallel for schedule(static) reduction(|| : bad)
    for (int64_t t = 0; t < T; ++t) {
        const int64_t rb = t / G, g = t % G;
        uint32_t count = 0;
        for (int64_t r = 0; r < kRows; ++r) {
            const int64_t m = rb * kRows + r;
            uint32_t *dst = bitmap + (t * kRows + r) * 4;
            for (int j = 0; j < 4; ++j) {
                uint32_t p = 0, n = 0;
                if (m < M && !masks_of(trits + m * K + g * kGroup + 32 * j, p, n)) bad = true;
                dst[j] = p;
                count += static_cast<uint32_t>(__builtin_popcount(p));
            }
        }
        tile_count[static_cast<size_t>(t)] = count;
    }
    if (bad) return BITCOS_ERR_TRIT;

    uint64_t run = 0;
    for (int64_t t = 0; t < T; ++t) {
        tile_off[t] = static_cast<uint32_t>(run);
        run += tile_count[static_cast<size_t>(t)];
        if (run > 0xFFFFFFFFull) return BITCOS_ERR_OVERFLOW;
    }
    tile_off[T] = static_cast<uint32_t>(run);
    for (int64_t t = T + 1; t < (T + 1 + 3) / 4 * 4; ++t) tile_off[t] = 0;     // padding to 16 bytes
    const size_t need = sign_bytes_for(run);
    if (sign_capacity_bytes < need) return BITCOS_ERR_CAPACITY;
    std::memset(signs, 0, need);

    // Pass 2: the sign bits of every non-zero, in tile order.
    BitWriter bw{signs};
    for (int64_t t = 0; t < T; ++t) {
        const int64_t rb = t / G, g = t % G;
        for (int64_t r = 0; r < kRows; ++r) {
            const int64_t m = rb * kRows + r;
            if (m >= M) break;
            for (int j = 0; j < 4; ++j) {
                uint32_t p = 0, n = 0;
                masks_of(trits + m * K + g * kGroup + 32 * j, p, n);
                bw.put(compact_bits(n, p), __builtin_popcount(p));
            }
        }
    }
    if (nnz_out) *nnz_out = run;
    return BITCOS_OK;
}

int bitcos_unpack(const uint32_t *bitmap, const uint32_t *signs, const uint32_t *tile_off, int64_t M, int64_t K,
                  int8_t *trits_out) {
    if (!bitmap || !signs || !tile_off || !trits_out) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t Mp = padded_rows(M), G = K / kGroup, T = (Mp / kRows) * G;
    bool bad = false;
#pragma omp parallel for schedule(static) reduction(|| : bad)
    for (int64_t t = 0; t < T; ++t) {
        const int64_t rb = t / G, g = t % G;
        uint64_t cursor = tile_off[t];
        for (int64_t r = 0; r < kRows; ++r) {
            const int64_t m = rb * kRows + r;
            for (int j = 0; j < 4; ++j) {
                const uint32_t p = bitmap[(t * kRows + r) * 4 + j];
                const uint64_t w = cursor >> 5;
                const uint64_t win = (static_cast<uint64_t>(signs[w]) | (static_cast<uint64_t>(signs[w + 1]) << 32)) >>
                                     (cursor & 31);
                const uint32_t n = deposit_bits(static_cast<uint32_t>(win), p);
                cursor += static_cast<uint64_t>(__builtin_popcount(p));
                if (m < M) {
                    int8_t *dst = trits_out + m * K + g * kGroup + 32 * j;
                    for (int i = 0; i < 32; ++i)
                        dst[i] = static_cast<int8_t>(static_cast<int>((p >> i) & 1u) - 2 * static_cast<int>((n >> i) & 1u));
                } else if (p != 0) {
                    bad = true;
                }
            }
        }
        if (cursor != tile_off[t + 1]) bad = true;
    }
    return bad ? BITCOS_ERR_TRIT : BITCOS_OK;
}

// ---- five-trit --------------------------------------------------------------------------------
static inline int64_t trit5_wpr(int64_t K) { return (26 * (K / kGroup) + 3) / 4; }

int trit5_pack_sizes(int64_t M, int64_t K, size_t *bytes) {
    if (!bytes) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    *bytes = static_cast<size_t>(padded_rows(M) * trit5_wpr(K)) * 4;
    return BITCOS_OK;
}

int trit5_pack(const int8_t *trits, int64_t M, int64_t K, uint32_t *words) {
    if (!trits || !words) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t Mp = padded_rows(M), G = K / kGroup, WPR = trit5_wpr(K);
    bool bad = false;
#pragma omp parallel for schedule(static) reduction(|| : bad)
    for (int64_t m = 0; m < Mp; ++m) {
        std::vector<uint8_t> row(static_cast<size_t>(WPR) * 4, 0);
        for (int64_t g = 0; g < G; ++g) {
            uint8_t *blk = row.data() + 26 * g;
            for (int j = 0; j < 26; ++j) {
                int v = 0;
                for (int i = 4; i >= 0; --i) {          // Horner, most significant digit first
                    const int idx = 5 * j + i;
                    int t = 0;
                    if (idx < 128 && m < M) {
                        t = trits[m * K + g * kGroup + idx];
                        if (t < -1 || t > 1) { bad = true; t = 0; }
                    }
                    v = v * 3 + (t + 1);
                }
                blk[j] = static_cast<uint8_t>(v);
            }
        }
        for (int64_t q = 0; q < WPR; ++q) {
            uint32_t w;
            std::memcpy(&w, row.data() + 4 * q, 4);     // little-endian host
            words[((m / kRows) * WPR + q) * kRows + m % kRows] = w;
        }
    }
    return bad ? BITCOS_ERR_TRIT : BITCOS_OK;
}

int trit5_unpack(const uint32_t *words, int64_t M, int64_t K, int8_t *trits_out) {
    if (!trits_out || !words) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t G = K / kGroup, WPR = trit5_wpr(K);
    bool bad = false;
#pragma omp parallel for schedule(static) reduction(|| : bad)
    for (int64_t m = 0; m < M; ++m) {
        std::vector<uint8_t> row(static_cast<size_t>(WPR) * 4, 0);
        for (int64_t q = 0; q < WPR; ++q) {
            const uint32_t w = words[((m / kRows) * WPR + q) * kRows + m % kRows];
            std::memcpy(row.data() + 4 * q, &w, 4);
        }
        for (int64_t g = 0; g < G; ++g)
            for (int j = 0; j < 26; ++j) {
                int v = row[static_cast<size_t>(26 * g + j)];
                if (v > 242) bad = true;
                for (int i = 0; i < 5; ++i) {
                    const int idx = 5 * j + i, d = v % 3;
                    v /= 3;
                    if (idx < 128) trits_out[m * K + g * kGroup + idx] = static_cast<int8_t>(d - 1);
                    else if (d != 1) bad = true;
                }
            }
    }
    return bad ? BITCOS_ERR_TRIT : BITCOS_OK;
}

// ---- 2-bit ---------------------------------------------------------------------------------------
int bit2_pack_sizes(int64_t M, int64_t K, size_t *bytes) {
    if (!bytes) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    *bytes = static_cast<size_t>(padded_rows(M) * K / 4);
    return BITCOS_OK;
}

static inline int64_t bit2_index(int64_t K, int64_t m, int64_t w) {
    return (((m / kRows) * (K / 64) + w / 4) * kRows + m % kRows) * 4 + w % 4;
}

int bit2_pack(const int8_t *trits, int64_t M, int64_t K, uint32_t *words) {
    if (!trits || !words) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    const int64_t Mp = padded_rows(M);
    bool bad = false;
#pragma omp parallel for schedule(static) reduction(|| : bad)
    for (int64_t m = 0; m < Mp; ++m)
        for (int64_t w = 0; w < K / 16; ++w) {
            uint32_t word = 0;
            for (int byte = 0; byte < 4; ++byte)
                for (int pair = 0; pair < 4; ++pair) {
                    int t = 0;
                    if (m < M) {
                        t = trits[m * K + 16 * w + 4 * pair + byte];
                        if (t < -1 || t > 1) { bad = true; t = 0; }
                    }
                    word |= static_cast<uint32_t>(t + 1) << (8 * byte + 2 * pair);
                }
            words[bit2_index(K, m, w)] = word;
        }
    return bad ? BITCOS_ERR_TRIT : BITCOS_OK;
}

int bit2_unpack(const uint32_t *words, int64_t M, int64_t K, int8_t *trits_out) {
    if (!trits_out || !words) return BITCOS_ERR_NULL;
    if (!shape_ok(M, K)) return BITCOS_ERR_SHAPE;
    bool bad = false;
#pragma omp parallel for schedule(static) reduction(|| : bad)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t w = 0; w < K / 16; ++w) {
            const uint32_t word = words[bit2_index(K, m, w)];
            for (int byte = 0; byte < 4; ++byte)
                for (int pair = 0; pair < 4; ++pair) {
                    const uint32_t code = (word >> (8 * byte + 2 * pair)) & 3u;
                    if (code == 3u) bad = true;
                    trits_out[m * K + 16 * w + 4 * pair + byte] = static_cast<int8_t>(static_cast<int>(code) - 1);
                }
        }
    return bad ? BITCOS_ERR_TRIT : BITCOS_OK;
}

}  // extern "C"
