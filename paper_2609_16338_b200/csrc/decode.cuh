// Tile decoders of the BITCOS library, shared by the GEMV kernels and the decode-rate probe.
//
// A lane owns one row of a 32 x 128 tile: four 32-bit presence words and the row's sign bits,
// which start at a bit cursor inside the tile's piece of the sign vector (paper Section II-A).
// The GPU has no bit-deposit instruction (Fig. 4), so the scatter of the compacted signs onto the
// present positions is done in software.  Several structurally different ways of doing it live
// here, so that their on-chip cost (the gamma of the paper's two-term roofline, Eq. 6) can be
// measured side by side; the GEMV kernels use the cheapest one.
#ifndef BITCOS_DECODE_CUH
#define BITCOS_DECODE_CUH

#include <cuda_runtime.h>

#include <cstdint>

namespace bitcos_dev {

constexpr int kLutBytes = 64 * 1024;      // a 256-entry table of 32-bit words, one copy per lane

// ---------------------------------------------------------------------------------------------
// Lookup tables, generated at compile time.
// ---------------------------------------------------------------------------------------------
struct Lut256 {
    uint32_t v[256];
};
struct Lut256x2 {
    uint32_t lo[256];
    uint32_t hi[256];
};

// Entry (m, s) of Eq. 4 as four int8: byte i = 0 if bit i of m is clear, else +1 / -1 by the
// sign bit whose index is the rank of i among the set bits of m.  Index = (s << 4) | m.
constexpr Lut256 make_nibble_lut() {
    Lut256 t{};
    for (int key = 0; key < 256; ++key) {
        const int m = key & 15, s = key >> 4;
        uint32_t e = 0;
        int r = 0;
        for (int i = 0; i < 4; ++i) {
            if ((m >> i) & 1) {
                e |= (((s >> r) & 1) ? 0xFFu : 0x01u) << (8 * i);
                ++r;
            }
        }
        t.v[key] = e;
    }
    return t;
}

// Five-trit byte -> digits t0..t4 (value - 1 each) as int8: lo = (t0,t1,t2,t3), hi = (t1,t2,t3,t4).
constexpr Lut256x2 make_trit5_lut() {
    Lut256x2 t{};
    for (int b = 0; b < 256; ++b) {
        int v = b;
        uint32_t d[5] = {0, 0, 0, 0, 0};
        for (int i = 0; i < 5; ++i) {
            d[i] = static_cast<uint32_t>((v % 3) - 1) & 0xFFu;
            v /= 3;
        }
        t.lo[b] = d[0] | (d[1] << 8) | (d[2] << 16) | (d[3] << 24);
        t.hi[b] = d[1] | (d[2] << 8) | (d[3] << 16) | (d[4] << 24);
    }
    return t;
}

// The tables as they sit in shared memory, replicated once per lane (32 copies) so that a warp's
// 32 lookups always fall into 32 different banks.
struct LutBig {
    uint32_t v[kLutBytes / 4];
};

// BITCOS: byte address = key * 256 + sub * 128 + lane * 4;
//   sub 0 ("even" nibbles): key = (s << 4) | m;  sub 1 ("odd" nibbles): key = (m << 4) | s,
// so that a presence BYTE placed in address bits 8..15 needs only its other nibble replaced
// by the four sign bits.
constexpr LutBig make_bitcos_lut() {
    const Lut256 base = make_nibble_lut();
    LutBig t{};
    for (int idx = 0; idx < kLutBytes / 4; ++idx) {
        const int key = idx >> 6, sub = (idx >> 5) & 1;
        const int src = sub ? (((key & 15) << 4) | (key >> 4)) : key;
        t.v[idx] = base.v[src];
    }
    return t;
}

// Five-trit: byte address = byte value * 256 + lane * 8 (lo word, hi word).
constexpr LutBig make_trit5_big() {
    const Lut256x2 base = make_trit5_lut();
    LutBig t{};
    for (int idx = 0; idx < kLutBytes / 4; ++idx) {
        const int key = idx >> 6;
        t.v[idx] = (idx & 1) ? base.hi[key] : base.lo[key];
    }
    return t;
}

// ---------------------------------------------------------------------------------------------
// Primitives.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t lds32(const uint8_t *base, uint32_t off) {
    return *reinterpret_cast<const uint32_t *>(base + off);
}
__device__ __forceinline__ uint2 lds64(const uint8_t *base, uint32_t off) {
    return *reinterpret_cast<const uint2 *>(base + off);
}
// dot product of four unsigned bytes of a with four signed bytes of b, plus c
__device__ __forceinline__ int dp4a_us(uint32_t a, int b, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// d = (a & c) | (b & ~c): one LOP3
__device__ __forceinline__ uint32_t bit_select(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xE4;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// d = a | (b & c): one LOP3
__device__ __forceinline__ uint32_t or_and(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xF8;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

// The 32-bit sign windows of a row's four presence words: S[j] holds, from bit 0 on, the sign bits
// of the non-zero weights of word j.  sp = the sign words at the word holding the row's first sign
// bit, sh = bit offset inside that word; a row consumes at most 128 sign bits, so five words
// starting there cover it (31 + 128 <= 160).
__device__ __forceinline__ void sign_windows(const uint4 bm, const uint32_t *sp, uint32_t sh, uint32_t (&S)[4]) {
    const int c0 = __popc(bm.x), c1 = __popc(bm.y), c2 = __popc(bm.z);
    const uint32_t s0 = sp[0], s1 = sp[1], s2 = sp[2], s3 = sp[3], s4 = sp[4];
    uint32_t a0 = __funnelshift_r(s0, s1, sh), a1 = __funnelshift_r(s1, s2, sh);
    uint32_t a2 = __funnelshift_r(s2, s3, sh), a3 = __funnelshift_r(s3, s4, sh);
    S[0] = a0;
    a0 = __funnelshift_rc(a0, a1, c0);
    a1 = __funnelshift_rc(a1, a2, c0);
    a2 = __funnelshift_rc(a2, a3, c0);
    S[1] = a0;
    a0 = __funnelshift_rc(a0, a1, c1);
    a1 = __funnelshift_rc(a1, a2, c1);
    S[2] = a0;
    S[3] = __funnelshift_rc(a0, a1, c2);
}

// ---------------------------------------------------------------------------------------------
// Decoder A ("shifted window"): the 256-entry (presence nibble, sign nibble) table of Eq. 4; every
// word keeps its sign window in a register and shifts it by the number of sign bits a nibble
// consumed (dp4a(e, e) of the looked-up entry).  Produces the row's 32 int8x4 words; the
// contraction follows as a separate step.  Five instructions per nibble besides the contraction:
// shift-left, bit-select, table load, dp4a popcount, shift-right.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void bitcos_decode_row(const uint4 bm, const uint32_t *sp, uint32_t sh, const uint8_t *lut,
                                                  uint32_t lane4, int (&w)[32]) {
    uint32_t S[4];
    sign_windows(bm, sp, sh, S);
    const uint32_t P[4] = {bm.x, bm.y, bm.z, bm.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // address bits 0..6 = lane * 4, bits 8..15 = presence byte k of word j (bits 16.. are 0)
            const uint32_t R = __byte_perm(P[j], lane4, 0x6504 | (k << 4));
            uint32_t off = bit_select(S[j] << 12, R, 0xF000u);     // sign nibble over the odd presence nibble
            int e = static_cast<int>(lds32(lut, off));
            w[8 * j + 2 * k] = e;
            S[j] >>= __dp4a(e, e, 0);                    // non-zeros in the nibble = sign bits consumed
            off = bit_select(S[j] << 8, R, 0x0F00u);               // sign nibble over the even presence nibble
            e = static_cast<int>(lds32(lut + 128, off));
            w[8 * j + 2 * k + 1] = e;
            S[j] >>= __dp4a(e, e, 0);
        }
    }
}

// int32 accumulator of a decoded row against one token's group activations xg[0..7] (shared memory).
__device__ __forceinline__ int row_contract(const int (&w)[32], const int4 *xg) {
    int a0 = 0, a1 = 0, a2 = 0, a3 = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int4 xq = xg[q];
        a0 = __dp4a(w[4 * q + 0], xq.x, a0);
        a1 = __dp4a(w[4 * q + 1], xq.y, a1);
        a2 = __dp4a(w[4 * q + 2], xq.z, a2);
        a3 = __dp4a(w[4 * q + 3], xq.w, a3);
    }
    return (a0 + a1) + (a2 + a3);
}

// ---------------------------------------------------------------------------------------------
// Decoder B ("running position"): the same table, but the window of a word is never shifted.
// Each word keeps a running bit position pos; dp4a(e, e, pos) adds a nibble's population count to
// it in the instruction that computes the count, and one rotate of a pre-rotated copy of the
// window puts the next four sign bits where the table key wants them (bits 12..15 for even
// nibbles, 8..11 for odd ones).  Four instructions per nibble besides the contraction: rotate,
// bit-select, table load, dp4a position; the contraction (one dp4a per token) is fused in, so the
// row never sits in 32 registers.  acc[b] receives the row's int32 group accumulator of token b.
//   xs          the group's activations of token 0 in shared memory (128 bytes, 16-byte aligned)
//   x_stride    bytes from one token's activations to the next
// ---------------------------------------------------------------------------------------------
template <int NB>
__device__ __forceinline__ void bitcos_row_dot(const uint4 bm, const uint32_t *sp, uint32_t sh, const uint8_t *lut,
                                               uint32_t lane4, const uint8_t *xs, uint32_t x_stride, int nb, int (&acc)[NB]) {
    uint32_t S[4];
    sign_windows(bm, sp, sh, S);
    const uint32_t P[4] = {bm.x, bm.y, bm.z, bm.w};
    uint32_t A[4], B[4];
    int pos[4];
    int a[NB][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        A[j] = __funnelshift_l(S[j], S[j], 12);     // sign bit pos lands on bit 12 after a right rotate by pos
        B[j] = __funnelshift_l(S[j], S[j], 8);      // ... on bit 8
        pos[j] = 0;
#pragma unroll
        for (int b = 0; b < NB; ++b) a[b][j] = 0;
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // activation words 8 j + 4 h .. + 3 of every token
            int4 xq[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b)
                xq[b] = (NB == 1 || b < nb) ? reinterpret_cast<const int4 *>(xs + static_cast<uint32_t>(b) * x_stride)[2 * j + h]
                                            : make_int4(0, 0, 0, 0);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                const int k = 2 * h + kk;
                const uint32_t R = __byte_perm(P[j], lane4, 0x6504 | (k << 4));
                uint32_t t = __funnelshift_r(A[j], A[j], pos[j]);
                int e = static_cast<int>(lds32(lut, bit_select(t, R, 0xF000u)));
                pos[j] = __dp4a(e, e, pos[j]);
#pragma unroll
                for (int b = 0; b < NB; ++b) a[b][j] = __dp4a(e, kk ? xq[b].z : xq[b].x, a[b][j]);
                t = __funnelshift_r(B[j], B[j], pos[j]);
                e = static_cast<int>(lds32(lut + 128, bit_select(t, R, 0x0F00u)));
                pos[j] = __dp4a(e, e, pos[j]);
#pragma unroll
                for (int b = 0; b < NB; ++b) a[b][j] = __dp4a(e, kk ? xq[b].w : xq[b].y, a[b][j]);
            }
        }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[b] = (a[b][0] + a[b][1]) + (a[b][2] + a[b][3]);
}

// ---------------------------------------------------------------------------------------------
// Decoder C ("byte table"): eight weights per step.  A first table, indexed by the presence byte,
// gives the place of that byte's block in a second table that holds, for every presence byte m,
// the 2^popcount(m) possible sign patterns (3^8 = 6561 entries of eight int8 weights, 52 KB, each
// block aligned to its own size), and the mask that keeps popcount(m) sign bits.  Two dependent
// loads per eight weights instead of two independent ones per four; the second table cannot be
// replicated per lane, so its loads collide on banks.
//   first table:  byte address = m * 256 + lane * 4; entry = block offset | (((8 << c) - 8) << 16)
//   second table: byte address = block offset + 8 * (the c sign bits); entry = two int8x4 words
// ---------------------------------------------------------------------------------------------
constexpr int kByteTableEntries = 6561;
constexpr int kByteTableBytes = kByteTableEntries * 8;

__device__ __forceinline__ int byte_block_offset(int m) {
    // blocks in order of falling size (so that each is aligned to its size), ties by m
    const int c = __popc(m);
    int off = 0;
    for (int o = 0; o < 256; ++o) {
        const int co = __popc(o);
        if (co > c || (co == c && o < m)) off += 8 << co;
    }
    return off;
}

// Fills both tables (all threads of the block take part; no barrier inside).
__device__ inline void build_byte_tables(uint8_t *first, uint8_t *second) {
    for (int i = threadIdx.x; i < 256 * 32; i += blockDim.x) {
        const int m = i >> 5, lane = i & 31;
        const uint32_t c = static_cast<uint32_t>(__popc(m));
        reinterpret_cast<uint32_t *>(first)[m * 64 + lane] = static_cast<uint32_t>(byte_block_offset(m)) | (((8u << c) - 8u) << 16);
    }
    for (int m = threadIdx.x; m < 256; m += blockDim.x) {
        const int c = __popc(m);
        uint32_t *blk = reinterpret_cast<uint32_t *>(second + byte_block_offset(m));
        for (int s = 0; s < (1 << c); ++s) {
            uint32_t lo = 0, hi = 0;
            int r = 0;
            for (int i = 0; i < 8; ++i) {
                if (!((m >> i) & 1)) continue;
                const uint32_t v = ((s >> r) & 1) ? 0xFFu : 0x01u;
                if (i < 4) lo |= v << (8 * i);
                else hi |= v << (8 * (i - 4));
                ++r;
            }
            blk[2 * s] = lo;
            blk[2 * s + 1] = hi;
        }
    }
}

__device__ __forceinline__ int bitcos_row_dot_bytes(const uint4 bm, const uint32_t *sp, uint32_t sh, const uint8_t *first,
                                                    const uint8_t *second, uint32_t lane4, const uint8_t *xs) {
    uint32_t S[4];
    sign_windows(bm, sp, sh, S);
    const uint32_t P[4] = {bm.x, bm.y, bm.z, bm.w};
    uint32_t A[4];
    int pos[4], a[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        A[j] = __funnelshift_l(S[j], S[j], 3);      // sign bit pos lands on bit 3 (entries are 8 bytes)
        pos[j] = 0;
        a[j] = 0;
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int4 xq = reinterpret_cast<const int4 *>(xs)[2 * j + h];
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                const int k = 2 * h + kk;
                const uint32_t e = lds32(first, __byte_perm(P[j], lane4, 0x6504 | (k << 4)));
                const uint32_t t = __funnelshift_r(A[j], A[j], pos[j]) & (e >> 16);
                const uint2 wv = lds64(second, or_and(t, e, 0xFFFFu));
                pos[j] = __dp4a(static_cast<int>(wv.x), static_cast<int>(wv.x), pos[j]);
                pos[j] = __dp4a(static_cast<int>(wv.y), static_cast<int>(wv.y), pos[j]);
                a[j] = __dp4a(static_cast<int>(wv.x), kk ? xq.z : xq.x, a[j]);
                a[j] = __dp4a(static_cast<int>(wv.y), kk ? xq.w : xq.y, a[j]);
            }
        }
    }
    return (a[0] + a[1]) + (a[2] + a[3]);
}

// ---------------------------------------------------------------------------------------------
// Decoder D ("no table"): the deposit of Fig. 4 carried out with shifts and masks on whole 32-bit
// words (five rounds that move the sign bits up by 16, 8, 4, 2 and 1 places under masks derived
// from the presence word by a parallel-prefix count of its zeros), then the contraction on bit
// planes: a presence (or negative) word masked with 0x01010101 << i holds bits 8 b + i as bytes of
// value 2^i, which an unsigned-by-signed dp4a multiplies with the four activations of those
// positions; acc = sum(p * x) - 2 sum(n * x), Eq. 2.  No shared-memory table at all.
//   xp   the group's activations re-ordered for the bit planes: word 8 j + i = bytes
//        x[32 j + i], x[32 j + 8 + i], x[32 j + 16 + i], x[32 j + 24 + i]
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t deposit32(uint32_t src, uint32_t mask) {
    uint32_t mv[5];
    uint32_t m = mask, mk = ~mask << 1;           // mk: positions with a zero just below them
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        uint32_t mp = mk ^ (mk << 1);             // parity of the zeros below each position
        mp ^= mp << 2;
        mp ^= mp << 4;
        mp ^= mp << 8;
        mp ^= mp << 16;
        mv[i] = mp & m;                           // mask bits that move by 2^i in this round
        m = (m ^ mv[i]) | (mv[i] >> (1 << i));
        mk &= ~mp;
    }
    uint32_t v = src;
#pragma unroll
    for (int i = 4; i >= 0; --i) {
        const uint32_t t = v << (1 << i);
        v = (v & ~mv[i]) | (t & mv[i]);
    }
    return v & mask;
}

__device__ __forceinline__ int bitcos_row_dot_planes(const uint4 bm, const uint32_t *sp, uint32_t sh, const uint8_t *xp) {
    uint32_t S[4];
    sign_windows(bm, sp, sh, S);
    const uint32_t P[4] = {bm.x, bm.y, bm.z, bm.w};
    // plane i of a word multiplies with byte value 2^i, so every plane keeps its own pair of sums
    // (each an exact multiple of 2^i) and is scaled back at the end
    int ap[8], an[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) ap[i] = an[i] = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t N = deposit32(S[j], P[j]);
        const int4 x0 = reinterpret_cast<const int4 *>(xp)[2 * j], x1 = reinterpret_cast<const int4 *>(xp)[2 * j + 1];
        const int xw[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            ap[i] = dp4a_us(P[j] & (0x01010101u << i), xw[i], ap[i]);
            an[i] = dp4a_us(N & (0x01010101u << i), xw[i], an[i]);
        }
    }
    int acc = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc += (ap[i] - 2 * an[i]) >> i;
    return acc;
}

// ---------------------------------------------------------------------------------------------
// Decoder F ("split row"): the first NL presence words of a row through the table with running
// positions (decoder B), the others through the table-free deposit and bit planes (decoder D).
// The table path is bound by shared-memory wavefronts, the table-free path by the integer ALU;
// splitting a row between them loads both pipes.
//   xs   the group's activations in natural order, xp the same in bit-plane order (decoder D)
// ---------------------------------------------------------------------------------------------
template <int NL>
__device__ __forceinline__ int bitcos_row_dot_split(const uint4 bm, const uint32_t *sp, uint32_t sh, const uint8_t *lut,
                                                    uint32_t lane4, const uint8_t *xs, const uint8_t *xp) {
    uint32_t S[4];
    sign_windows(bm, sp, sh, S);
    const uint32_t P[4] = {bm.x, bm.y, bm.z, bm.w};
    int acc = 0;
    // table part
    uint32_t A[NL > 0 ? NL : 1], B[NL > 0 ? NL : 1];
    int pos[NL > 0 ? NL : 1], a[NL > 0 ? NL : 1];
#pragma unroll
    for (int j = 0; j < NL; ++j) {
        A[j] = __funnelshift_l(S[j], S[j], 12);
        B[j] = __funnelshift_l(S[j], S[j], 8);
        pos[j] = 0;
        a[j] = 0;
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int j = 0; j < NL; ++j) {
            const int4 xq = reinterpret_cast<const int4 *>(xs)[2 * j + h];
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                const int k = 2 * h + kk;
                const uint32_t R = __byte_perm(P[j], lane4, 0x6504 | (k << 4));
                uint32_t t = __funnelshift_r(A[j], A[j], pos[j]);
                int e = static_cast<int>(lds32(lut, bit_select(t, R, 0xF000u)));
                pos[j] = __dp4a(e, e, pos[j]);
                a[j] = __dp4a(e, kk ? xq.z : xq.x, a[j]);
                t = __funnelshift_r(B[j], B[j], pos[j]);
                e = static_cast<int>(lds32(lut + 128, bit_select(t, R, 0x0F00u)));
                pos[j] = __dp4a(e, e, pos[j]);
                a[j] = __dp4a(e, kk ? xq.w : xq.y, a[j]);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < NL; ++j) acc += a[j];
    // table-free part
    if (NL < 4) {
        int ap[8], an[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) ap[i] = an[i] = 0;
#pragma unroll
        for (int j = NL; j < 4; ++j) {
            const uint32_t N = deposit32(S[j], P[j]);
            const int4 x0 = reinterpret_cast<const int4 *>(xp)[2 * j], x1 = reinterpret_cast<const int4 *>(xp)[2 * j + 1];
            const int xw[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                ap[i] = dp4a_us(P[j] & (0x01010101u << i), xw[i], ap[i]);
                an[i] = dp4a_us(N & (0x01010101u << i), xw[i], an[i]);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) acc += (ap[i] - 2 * an[i]) >> i;
    }
    return acc;
}

// ---------------------------------------------------------------------------------------------
// Decoder E ("lane = bit"): the whole warp works on one presence word at a time, lane i on bit i:
// a weight's sign slot is the population count of the word's lower bits, its sign is that bit of
// the window at the warp's running cursor, and the 32 products are added across the warp.  Rows
// are taken one after the other.  `bitmap` = the tile's 128 presence words (row major), `sg` =
// the tile's sign words from the word of its first sign bit, `cur` = bit offset of that first
// bit; lane r returns row r's accumulator.
//   xl   this lane's activations: xl[j] = x[32 j + lane]
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int bitcos_tile_dot_lanes(const uint32_t *bitmap, const uint32_t *sg, uint32_t cur, const int (&xl)[4],
                                                     int lane) {
    const uint32_t below = (1u << lane) - 1u;
    int mine = 0;
    for (int r = 0; r < 32; ++r) {
        const uint4 bm = reinterpret_cast<const uint4 *>(bitmap)[r];
        const uint32_t P[4] = {bm.x, bm.y, bm.z, bm.w};
        int a = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t w = cur >> 5;
            const uint32_t win = __funnelshift_r(sg[w], sg[w + 1], cur);
            const int p = static_cast<int>((P[j] >> lane) & 1u);
            const int n = static_cast<int>((win >> __popc(P[j] & below)) & 1u);
            a += (p - 2 * (p & n)) * xl[j];
            cur += static_cast<uint32_t>(__popc(P[j]));
        }
        a = __reduce_add_sync(0xFFFFFFFFu, a);
        if (lane == r) mine = a;
    }
    return mine;
}

// ---------------------------------------------------------------------------------------------
// Five-trit and 2-bit rows.
// ---------------------------------------------------------------------------------------------

// Five-trit: wd = the seven words that hold the row's 26 bytes, odd = byte offset 2 (odd group).
__device__ __forceinline__ void trit5_decode_row(const uint32_t (&wd)[7], int odd, const uint8_t *lut, uint32_t lane8,
                                                 int (&w)[32]) {
    uint32_t lo[26], hi[26];
#pragma unroll
    for (int j = 0; j < 26; ++j) {
        const int be = j, bo = j + 2;
        const uint32_t word = odd ? wd[bo >> 2] : wd[be >> 2];
        const uint32_t sel = odd ? (0x6504u | ((bo & 3) << 4)) : (0x6504u | ((be & 3) << 4));
        const uint32_t off = __byte_perm(word, lane8, sel);    // byte * 256 + lane * 8
        const uint2 e = lds64(lut, off);
        lo[j] = e.x;
        hi[j] = e.y;
    }
#pragma unroll
    for (int q = 0; q < 6; ++q) {
        w[5 * q + 0] = static_cast<int>(lo[4 * q]);
        w[5 * q + 1] = static_cast<int>(__byte_perm(hi[4 * q], lo[4 * q + 1], 0x6543));
        w[5 * q + 2] = static_cast<int>(__byte_perm(hi[4 * q + 1], lo[4 * q + 2], 0x5432));
        w[5 * q + 3] = static_cast<int>(__byte_perm(hi[4 * q + 2], lo[4 * q + 3], 0x4321));
        w[5 * q + 4] = static_cast<int>(hi[4 * q + 3]);
    }
    w[30] = static_cast<int>(lo[24]);
    w[31] = static_cast<int>(__byte_perm(hi[24], lo[25], 0x6543));
}

// 2-bit: w[4q + j] keeps pair j of every byte of word q in place (value = code * 4^j), to be
// multiplied with activation word 4q + j.
__device__ __forceinline__ void bit2_decode_row(const uint4 v0, const uint4 v1, int (&w)[32]) {
    const uint32_t wd[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
    for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int j = 0; j < 4; ++j) w[4 * q + j] = static_cast<int>(wd[q] & (0x03030303u << (2 * j)));
}

// 2-bit, as plain int8: w[4q + j] byte b = code - 1 of weight 16 q + 4 j + b.  Per byte,
// (code + 0x7F) ^ 0x80 maps 0, 1, 2 to -1, 0, +1 without a carry between bytes.
__device__ __forceinline__ void bit2_decode_row_s8(const uint4 v0, const uint4 v1, int (&w)[32]) {
    const uint32_t wd[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
    for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            w[4 * q + j] = static_cast<int>((((wd[q] >> (2 * j)) & 0x03030303u) + 0x7F7F7F7Fu) ^ 0x80808080u);
}

}  // namespace bitcos_dev

#endif  // BITCOS_DECODE_CUH
