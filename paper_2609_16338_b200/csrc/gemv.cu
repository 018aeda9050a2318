// Device side of the BITCOS library: ternary GEMV kernels for sm_100a and their C entry
// points (bitcos_gemv, trit5_gemv, bit2_gemv, bitcos_gemv_grouped).
//
// Work decomposition (all formats).  Rows are handled 32 at a time (a "row block"), one
// row per lane, so that the activations a warp needs are the same for all of its lanes
// and arrive by broadcast loads; the reduction is cut into groups of 128.  A warp runs over
// `gpw` consecutive groups of one row block, keeping one fp32 partial sum per lane and
// token.  The S = (K/128)/gpw runs of a row block are spread over SC warps of one thread
// block and, if S > SC, over CS thread blocks; partial sums are added in a fixed order
// (shared memory inside a block, then a scratch buffer and an arrival counter across
// blocks), so results do not depend on scheduling.
//
// BITCOS decode (paper Section II-D, Eq. 4, adapted): the GPU has no bit-deposit
// instruction, so four weights at a time are rebuilt from a (presence nibble, next four
// sign bits) key through a 256-entry table held in shared memory, replicated once per lane
// so that lookups never conflict.  Entries are the four weights as int8 (w = p - 2n, Eq. 2)
// and feed dp4a directly.  A lane's position in the sign vector is the tile's entry offset
// plus a warp prefix sum over the rows' population counts; inside a row the window is
// shifted by the number of sign bits each nibble consumed.
#include "bitcos.h"

#include <cuda_runtime.h>

#include <cstdint>

namespace {

constexpr int kGroup = BITCOS_GROUP;
constexpr int kRows = BITCOS_TILE_ROWS;
constexpr int kMaxWarps = 16;           // warps per thread block
constexpr int kLutBytes = 64 * 1024;    // replicated lookup tables (BITCOS, five-trit)

enum Format { kBitcos = 0, kTrit5 = 1, kBit2 = 2 };

thread_local int g_last_cuda_error = 0;

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

__constant__ Lut256 c_nibble_lut = make_nibble_lut();
__constant__ Lut256x2 c_trit5_lut = make_trit5_lut();

// ---------------------------------------------------------------------------------------------
// Launch plan.
// ---------------------------------------------------------------------------------------------
struct Plan {
    int gpw;        // groups per warp run
    int S;          // runs per row block
    int SC;         // runs of a row block inside one thread block
    int CS;         // thread blocks per row block
    int RBC;        // row blocks per thread block (> 1 only if CS == 1)
    int NW;         // warps per thread block
    int64_t units;  // work units
};

struct Problem {
    const uint32_t *payload;   // bitmap / five-trit words / 2-bit words
    const uint32_t *signs;
    const uint32_t *tile_off;
    const uint16_t *scales;    // tile order
    const int8_t *x;
    const float *x_scale;
    const int32_t *xrow;       // NULL: token b reads row b of x
    float *y;
    int32_t *acc_debug;
    float *partial;
    unsigned int *counters;
    int64_t M, K;
    int G, RB;
    int nb;                    // tokens in this call / group
    int64_t out_row0;          // first output row of y / acc_debug for token 0
};

struct GroupedArgs {
    const bitcos_weights *experts;
    const int32_t *group_expert;
    const int32_t *group_begin;
    size_t ws_stride;          // workspace bytes per group
    int n_experts;
};

inline int64_t padded_rows(int64_t M) { return (M + kRows - 1) / kRows * kRows; }

Plan make_plan(int64_t M, int64_t K) {
    const int G = static_cast<int>(K / kGroup);
    const int64_t RB = padded_rows(M) / kRows;
    const int64_t target = 148 * 32;
    // Longest run that still yields enough warps to fill the machine; else one group per warp.
    int best = 1;
    for (int d = 1; d <= G; ++d) {
        if (G % d) continue;
        if (RB * (G / d) >= target) best = d;
    }
    Plan p{};
    auto derive = [&](int d) {
        p.gpw = d;
        p.S = G / d;
        if (p.S <= kMaxWarps) {
            p.SC = p.S;
            p.CS = 1;
            int64_t r = kMaxWarps / p.S;
            if (r > RB) r = RB;
            if (r < 1) r = 1;
            p.RBC = static_cast<int>(r);
        } else {
            int sc = 1;
            for (int c = 1; c <= kMaxWarps; ++c)
                if (p.S % c == 0) sc = c;
            p.SC = sc;
            p.CS = p.S / sc;
            p.RBC = 1;
        }
        p.NW = p.SC * p.RBC;
    };
    derive(best);
    if (p.NW < 4) {
        // S has no useful divisor: fall back to the divisor of G giving the fullest block
        int pick = best, pick_nw = p.NW;
        for (int d = 1; d <= G; ++d) {
            if (G % d) continue;
            derive(d);
            if (p.NW > pick_nw) { pick = d; pick_nw = p.NW; }
        }
        derive(pick);
    }
    p.units = ((RB + p.RBC - 1) / p.RBC) * p.CS;
    return p;
}

size_t counters_bytes(int64_t RB) { return static_cast<size_t>((RB * 4 + 255) / 256 * 256); }

size_t workspace_bytes_for(int64_t M, int64_t K) {
    const Plan p = make_plan(M, K);
    const int64_t RB = padded_rows(M) / kRows;
    size_t b = counters_bytes(RB);
    if (p.CS > 1) b += static_cast<size_t>(RB) * p.CS * BITCOS_MAX_BATCH * kRows * sizeof(float);
    return b;
}

// ---------------------------------------------------------------------------------------------
// Device helpers.
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
__device__ __forceinline__ float bf16_to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// Replicated table layout, byte address = key * 256 + sub * 128 + lane * 4:
//   sub 0 ("even" nibbles): key = (s << 4) | m;  sub 1 ("odd" nibbles): key = (m << 4) | s.
// so that a presence BYTE placed in address bits 8..15 needs only its other nibble replaced
// by the four sign bits.
__device__ __forceinline__ void build_bitcos_lut(uint8_t *smem) {
    uint32_t *lut = reinterpret_cast<uint32_t *>(smem);
    for (int idx = threadIdx.x; idx < kLutBytes / 4; idx += blockDim.x) {
        const int key = idx >> 6, sub = (idx >> 5) & 1;
        const int src = sub ? (((key & 15) << 4) | (key >> 4)) : key;
        lut[idx] = c_nibble_lut.v[src];
    }
}

// byte address = byte value * 256 + lane * 8 (lo, hi)
__device__ __forceinline__ void build_trit5_lut(uint8_t *smem) {
    uint32_t *lut = reinterpret_cast<uint32_t *>(smem);
    for (int idx = threadIdx.x; idx < kLutBytes / 4; idx += blockDim.x) {
        const int key = idx >> 6;
        lut[idx] = (idx & 1) ? c_trit5_lut.hi[key] : c_trit5_lut.lo[key];
    }
}

// One 32-bit presence word: eight (nibble, sign window) lookups.  `sw` holds the sign bits
// of this word's non-zeros from bit 0 upwards.  lane4 = lane * 4.
__device__ __forceinline__ void bitcos_decode_word(uint32_t P, uint32_t sw, const uint8_t *lut, uint32_t lane4,
                                                   int *w) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        // address bits 0..6 = lane * 4, bits 8..15 = presence byte k
        const uint32_t R = __byte_perm(P, lane4, 0x6504 | (k << 4));
        uint32_t off = ((sw << 12) & 0xF000u) | (R & 0x0FFFu);
        int e = static_cast<int>(lds32(lut, off));
        w[2 * k] = e;
        sw >>= __dp4a(e, e, 0);                      // number of non-zeros = sign bits consumed
        off = ((sw << 8) & 0x0F00u) | (R & 0xF0FFu);
        e = static_cast<int>(lds32(lut + 128, off));
        w[2 * k + 1] = e;
        sw >>= __dp4a(e, e, 0);
    }
}

// Decodes tile t (32 rows x 128 k) of a BITCOS matrix: lane = row.  w[i] = weights 4i..4i+3 as int8.
__device__ __forceinline__ void bitcos_decode_tile(const Problem &pr, int64_t t, int lane, const uint8_t *lut,
                                                   int (&w)[32]) {
    const uint4 bm = __ldcs(reinterpret_cast<const uint4 *>(pr.payload) + t * kRows + lane);
    const int c0 = __popc(bm.x), c1 = __popc(bm.y), c2 = __popc(bm.z), c3 = __popc(bm.w);
    const int c = c0 + c1 + c2 + c3;
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += v;
    }
    const uint32_t cursor = __ldg(pr.tile_off + t) + static_cast<uint32_t>(incl - c);
    const uint32_t *sp = pr.signs + (cursor >> 5);
    const uint32_t s0 = __ldg(sp), s1 = __ldg(sp + 1), s2 = __ldg(sp + 2), s3 = __ldg(sp + 3), s4 = __ldg(sp + 4);
    const uint32_t sh = cursor & 31u;
    uint32_t a0 = __funnelshift_r(s0, s1, sh), a1 = __funnelshift_r(s1, s2, sh);
    uint32_t a2 = __funnelshift_r(s2, s3, sh), a3 = __funnelshift_r(s3, s4, sh);
    const uint32_t lane4 = static_cast<uint32_t>(lane) * 4u;
    bitcos_decode_word(bm.x, a0, lut, lane4, w);
    a0 = __funnelshift_rc(a0, a1, c0);
    a1 = __funnelshift_rc(a1, a2, c0);
    a2 = __funnelshift_rc(a2, a3, c0);
    bitcos_decode_word(bm.y, a0, lut, lane4, w + 8);
    a0 = __funnelshift_rc(a0, a1, c1);
    a1 = __funnelshift_rc(a1, a2, c1);
    bitcos_decode_word(bm.z, a0, lut, lane4, w + 16);
    a0 = __funnelshift_rc(a0, a1, c2);
    bitcos_decode_word(bm.w, a0, lut, lane4, w + 24);
}

// Five-trit tile: the 26 bytes of group g of the lane's row start at byte 26g of the row
// string, i.e. at word (26g)/4 with byte offset 0 (g even) or 2 (g odd): seven words.
__device__ __forceinline__ void trit5_decode_tile(const Problem &pr, int64_t rb, int g, int lane, const uint8_t *lut,
                                                  int (&w)[32]) {
    const int64_t WPR = (26 * static_cast<int64_t>(pr.G) + 3) / 4;
    const int q0 = (26 * g) >> 2;
    const uint32_t *src = pr.payload + (rb * WPR + q0) * kRows + lane;
    uint32_t wd[7];
#pragma unroll
    for (int i = 0; i < 7; ++i) {
        // row strings are padded to whole words, so word q0 + 6 always exists
        wd[i] = __ldcs(src + static_cast<int64_t>(i) * kRows);
    }
    const uint32_t lane8 = static_cast<uint32_t>(lane) * 8u;
    const int odd = g & 1;
    uint32_t lo[26], hi[26];
#pragma unroll
    for (int j = 0; j < 26; ++j) {
        // byte j of the block = byte (j + 2*odd) of the seven loaded words
        const int be = j, bo = j + 2;
        const uint32_t we = wd[be >> 2], wo = wd[bo >> 2];
        const uint32_t word = odd ? wo : we;
        const uint32_t sel = odd ? (0x6504u | ((bo & 3) << 4)) : (0x6504u | ((be & 3) << 4));
        const uint32_t off = __byte_perm(word, lane8, sel);   // byte * 256 + lane * 8
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

// 2-bit tile: eight words per lane; w[4q + j] keeps pair j of every byte of word q in place
// (value = code * 4^j), to be multiplied with activation word 4q + j.
__device__ __forceinline__ void bit2_decode_tile(const Problem &pr, int64_t t, int lane, int (&w)[32]) {
    const uint4 *src = reinterpret_cast<const uint4 *>(pr.payload) + (t * 2) * kRows + lane;
    const uint4 v0 = __ldcs(src), v1 = __ldcs(src + kRows);
    const uint32_t wd[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
    for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int j = 0; j < 4; ++j) w[4 * q + j] = static_cast<int>(wd[q] & (0x03030303u << (2 * j)));
}

// int32 accumulator of one row (lane) and group against token activations xg[0..127].
template <int FMT>
__device__ __forceinline__ int contract(const int (&w)[32], const int8_t *xg, int lane) {
    const int4 *xv = reinterpret_cast<const int4 *>(xg);
    if (FMT == kBit2) {
        int a0 = 0, a1 = 0, a2 = 0, a3 = 0;
        // sum of the group's activations, needed because the stored code is weight + 1
        int sx = __dp4a(0x01010101, __ldg(reinterpret_cast<const int *>(xg) + lane), 0);
        sx = __reduce_add_sync(0xFFFFFFFFu, sx);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int4 xq = __ldg(xv + q);
            a0 = dp4a_us(static_cast<uint32_t>(w[4 * q + 0]), xq.x, a0);
            a1 = dp4a_us(static_cast<uint32_t>(w[4 * q + 1]), xq.y, a1);
            a2 = dp4a_us(static_cast<uint32_t>(w[4 * q + 2]), xq.z, a2);
            a3 = dp4a_us(static_cast<uint32_t>(w[4 * q + 3]), xq.w, a3);
        }
        return a0 + (a1 >> 2) + (a2 >> 4) + (a3 >> 6) - sx;
    } else {
        int a = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int4 xq = __ldg(xv + q);
            a = __dp4a(w[4 * q + 0], xq.x, a);
            a = __dp4a(w[4 * q + 1], xq.y, a);
            a = __dp4a(w[4 * q + 2], xq.z, a);
            a = __dp4a(w[4 * q + 3], xq.w, a);
        }
        return a;
    }
}

template <int FMT, int NB>
__device__ __forceinline__ void run_problem(const Problem &pr, const Plan &pl, uint8_t *smem) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint8_t *lut = smem;
    float *red = reinterpret_cast<float *>(smem + (FMT == kBit2 ? 0 : kLutBytes));
    __shared__ int s_last;

    int xr[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        const int bb = b < pr.nb ? b : 0;
        xr[b] = pr.xrow ? __ldg(pr.xrow + bb) : bb;
    }

    for (int64_t u = blockIdx.x; u < pl.units; u += gridDim.x) {
        const int64_t rbg = u / pl.CS;
        const int cs = static_cast<int>(u % pl.CS);
        const int rbl = warp / pl.SC, run_local = warp % pl.SC;
        const int64_t rb = rbg * pl.RBC + rbl;
        const int run = cs * pl.SC + run_local;
        const bool active = rb < pr.RB;
        const int64_t m = rb * kRows + lane;

        float ysum[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) ysum[b] = 0.f;

        if (active) {
            for (int g = run * pl.gpw; g < (run + 1) * pl.gpw; ++g) {
                const int64_t t = rb * pr.G + g;
                int w[32];
                if (FMT == kBitcos) bitcos_decode_tile(pr, t, lane, lut, w);
                else if (FMT == kTrit5) trit5_decode_tile(pr, rb, g, lane, lut, w);
                else bit2_decode_tile(pr, t, lane, w);
                const float s = bf16_to_float(__ldg(pr.scales + t * kRows + lane));
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (b < pr.nb) {
                        const int a = contract<FMT>(w, pr.x + static_cast<int64_t>(xr[b]) * pr.K + g * kGroup, lane);
                        ysum[b] = fmaf(s, static_cast<float>(a), ysum[b]);
                        if (pr.acc_debug && m < pr.M)
                            pr.acc_debug[((pr.out_row0 + b) * pr.M + m) * pr.G + g] = a;
                    }
                }
            }
        }

        // ---- reduce the runs of each row block inside the thread block, in run order ----
        if (pl.SC > 1) {
#pragma unroll
            for (int b = 0; b < NB; ++b) red[(warp * NB + b) * kRows + lane] = ysum[b];
            __syncthreads();
            if (run_local == 0) {
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    float tot = 0.f;
                    for (int s2 = 0; s2 < pl.SC; ++s2) tot += red[((warp + s2) * NB + b) * kRows + lane];
                    ysum[b] = tot;
                }
            }
        }
        if (pl.CS == 1) {
            if (run_local == 0 && active && m < pr.M) {
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    if (b < pr.nb) pr.y[(pr.out_row0 + b) * pr.M + m] = __ldg(pr.x_scale + xr[b]) * ysum[b];
            }
        } else {
            // ---- several thread blocks per row block: scratch partials + arrival counter ----
            if (run_local == 0) {
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    if (b < pr.nb) pr.partial[((rb * pl.CS + cs) * pr.nb + b) * kRows + lane] = ysum[b];
                __threadfence();
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                const unsigned int old = atomicAdd(pr.counters + rb, 1u);
                s_last = (old == static_cast<unsigned int>(pl.CS - 1));
            }
            __syncthreads();
            if (s_last && warp == 0) {
                __threadfence();
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (b < pr.nb) {
                        float tot = 0.f;
                        for (int c = 0; c < pl.CS; ++c)
                            tot += __ldcg(pr.partial + ((rb * pl.CS + c) * pr.nb + b) * kRows + lane);
                        if (m < pr.M) pr.y[(pr.out_row0 + b) * pr.M + m] = __ldg(pr.x_scale + xr[b]) * tot;
                    }
                }
                if (lane == 0) pr.counters[rb] = 0u;   // leave the counter ready for the next call
            }
        }
        __syncthreads();
    }
}

template <int FMT, int NB>
__global__ void __launch_bounds__(kMaxWarps * 32) gemv_kernel(const Problem pr, const Plan pl) {
    extern __shared__ __align__(16) uint8_t smem[];
    if (FMT == kBitcos) build_bitcos_lut(smem);
    if (FMT == kTrit5) build_trit5_lut(smem);
    if (FMT != kBit2) __syncthreads();
    run_problem<FMT, NB>(pr, pl, smem);
}

template <int NB>
__global__ void __launch_bounds__(kMaxWarps * 32) gemv_grouped_kernel(Problem pr, const Plan pl, const GroupedArgs ga) {
    extern __shared__ __align__(16) uint8_t smem[];
    build_bitcos_lut(smem);
    __syncthreads();
    const int grp = blockIdx.y;
    const int e = __ldg(ga.group_expert + grp);
    const int begin = __ldg(ga.group_begin + grp), end = __ldg(ga.group_begin + grp + 1);
    if (e < 0 || e >= ga.n_experts || end <= begin) return;
    const bitcos_weights wdesc = ga.experts[e];
    pr.payload = wdesc.bitmap;
    pr.signs = wdesc.signs;
    pr.tile_off = wdesc.tile_off;
    pr.scales = wdesc.scales;
    pr.nb = min(end - begin, NB);
    pr.xrow = pr.xrow + begin;
    pr.out_row0 = begin;
    uint8_t *ws = reinterpret_cast<uint8_t *>(pr.counters) + static_cast<size_t>(grp) * ga.ws_stride;
    pr.counters = reinterpret_cast<unsigned int *>(ws);
    pr.partial = reinterpret_cast<float *>(ws + ((static_cast<size_t>(pr.RB) * 4 + 255) / 256 * 256));
    run_problem<kBitcos, NB>(pr, pl, smem);
}

// ---------------------------------------------------------------------------------------------
// Host side of the device entry points.
// ---------------------------------------------------------------------------------------------
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int check_cuda(cudaError_t e) {
    if (e == cudaSuccess) return BITCOS_OK;
    g_last_cuda_error = static_cast<int>(e);
    return BITCOS_ERR_CUDA;
}

size_t smem_bytes(int fmt, int nw, int nb) {
    return (fmt == kBit2 ? 0 : kLutBytes) + static_cast<size_t>(nw) * nb * kRows * sizeof(float);
}

// Number of thread blocks to launch: min(units, SMs x resident blocks per SM).  The
// occupancy query and the opt-in to large dynamic shared memory are done on the first call
// for a given kernel (one cache per kernel instantiation), block size and device, and remembered (so that first call must not
// happen during stream capture; later calls only read the cache).
template <auto kernel>
int grid_for(int threads, size_t smem, int64_t units, int *grid) {
    constexpr int kMaxDev = 32;
    static int cache[kMaxDev][kMaxWarps + 1][2];      // [device][warps][0: blocks per SM, 1: SMs]; 0 = unknown
    int dev = 0;
    int rc = check_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    const int nw = threads / 32;
    int per_sm = 0, sms = 0;
    if (dev < kMaxDev && cache[dev][nw][0] > 0) {
        per_sm = cache[dev][nw][0];
        sms = cache[dev][nw][1];
    } else {
        rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (rc) return rc;
        rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLutBytes + 32 * 1024));
        if (rc) return rc;
        rc = check_cuda(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem));
        if (rc) return rc;
        if (per_sm < 1) per_sm = 1;
        if (dev < kMaxDev) {
            cache[dev][nw][1] = sms;
            cache[dev][nw][0] = per_sm;
        }
    }
    const int64_t cap = static_cast<int64_t>(sms) * per_sm;
    *grid = static_cast<int>(units < cap ? units : cap);
    return BITCOS_OK;
}

template <int FMT, int NB>
int launch(const Problem &pr, const Plan &pl, cudaStream_t stream) {
    const size_t smem = smem_bytes(FMT, pl.NW, NB);
    int grid = 1;
    int rc = grid_for<gemv_kernel<FMT, NB>>(pl.NW * 32, smem, pl.units, &grid);
    if (rc) return rc;
    gemv_kernel<FMT, NB><<<grid, pl.NW * 32, smem, stream>>>(pr, pl);
    return check_cuda(cudaGetLastError());
}

template <int FMT>
int launch_nb(const Problem &pr, const Plan &pl, cudaStream_t stream) {
    if (pr.nb <= 1) return launch<FMT, 1>(pr, pl, stream);
    if (pr.nb <= 2) return launch<FMT, 2>(pr, pl, stream);
    if (pr.nb <= 4) return launch<FMT, 4>(pr, pl, stream);
    if (pr.nb <= 8) return launch<FMT, 8>(pr, pl, stream);
    return launch<FMT, 16>(pr, pl, stream);
}

template <int NB>
int launch_grouped(const Problem &pr, const Plan &pl, const GroupedArgs &ga, int n_groups, cudaStream_t stream) {
    const size_t smem = smem_bytes(kBitcos, pl.NW, NB);
    int grid = 1;
    int rc = grid_for<gemv_grouped_kernel<NB>>(pl.NW * 32, smem, pl.units, &grid);
    if (rc) return rc;
    // the grid's x extent is shared by all groups: spread the machine over them
    int gx = (grid + n_groups - 1) / n_groups;
    if (gx < 1) gx = 1;
    if (gx > pl.units) gx = static_cast<int>(pl.units);
    gemv_grouped_kernel<NB><<<dim3(gx, n_groups), pl.NW * 32, smem, stream>>>(pr, pl, ga);
    return check_cuda(cudaGetLastError());
}

int gemv_common(int fmt, const uint32_t *payload, const uint32_t *signs, const uint32_t *tile_off,
                const uint16_t *scales, int64_t M, int64_t K, const int8_t *x, const float *x_scale, int batch,
                float *y, int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!payload || !scales || !x || !x_scale || !y || !workspace) return BITCOS_ERR_NULL;
    if (fmt == kBitcos && (!signs || !tile_off)) return BITCOS_ERR_NULL;
    if (M < 1 || K < kGroup || K % kGroup != 0 || batch < 1 || batch > BITCOS_MAX_BATCH) return BITCOS_ERR_SHAPE;
    if (K / kGroup > 0x7FFFFF || padded_rows(M) / kRows > 0x7FFFFFFF) return BITCOS_ERR_SHAPE;
    if (!aligned16(payload) || !aligned16(scales) || !aligned16(x) || !aligned16(y) || !aligned16(workspace) ||
        (signs && !aligned16(signs)) || (tile_off && !aligned16(tile_off)) || (acc_debug && !aligned16(acc_debug)))
        return BITCOS_ERR_ALIGN;
    if (workspace_bytes < workspace_bytes_for(M, K)) return BITCOS_ERR_CAPACITY;

    const Plan pl = make_plan(M, K);
    Problem pr{};
    pr.payload = payload;
    pr.signs = signs;
    pr.tile_off = tile_off;
    pr.scales = scales;
    pr.x = x;
    pr.x_scale = x_scale;
    pr.xrow = nullptr;
    pr.y = y;
    pr.acc_debug = acc_debug;
    pr.M = M;
    pr.K = K;
    pr.G = static_cast<int>(K / kGroup);
    pr.RB = static_cast<int>(padded_rows(M) / kRows);
    pr.nb = batch;
    pr.out_row0 = 0;
    pr.counters = static_cast<unsigned int *>(workspace);
    pr.partial = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + counters_bytes(pr.RB));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (fmt == kBitcos) return launch_nb<kBitcos>(pr, pl, stream);
    if (fmt == kTrit5) return launch_nb<kTrit5>(pr, pl, stream);
    return launch_nb<kBit2>(pr, pl, stream);
}

}  // namespace

extern "C" {

int bitcos_last_cuda_error(void) { return g_last_cuda_error; }

size_t bitcos_gemv_workspace_bytes(int64_t M, int64_t K) {
    if (M < 1 || K < kGroup || K % kGroup != 0) return 0;
    return workspace_bytes_for(M, K);
}

int bitcos_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!workspace) return BITCOS_ERR_NULL;
    return check_cuda(cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(cuda_stream)));
}

int bitcos_gemv(const bitcos_weights *W, const int8_t *x, const float *x_scale, int batch, float *y,
                int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!W) return BITCOS_ERR_NULL;
    return gemv_common(kBitcos, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x, x_scale, batch, y,
                       acc_debug, workspace, workspace_bytes, cuda_stream);
}

size_t bitcos_gemv_host_staging_bytes(int64_t M, int64_t K, int batch) {
    if (M < 1 || K < kGroup || K % kGroup != 0 || batch < 1 || batch > BITCOS_MAX_BATCH) return 0;
    const size_t xb = (static_cast<size_t>(batch) * K + 255) / 256 * 256;
    return xb + 256 + static_cast<size_t>(batch) * M * sizeof(float);
}

int bitcos_gemv_host(const bitcos_weights *W, const int8_t *x_host, const float *x_scale_host, int batch,
                     float *y_host, void *staging, size_t staging_bytes, void *workspace,
                     size_t workspace_bytes, void *cuda_stream) {
    if (!W || !x_host || !x_scale_host || !y_host || !staging) return BITCOS_ERR_NULL;
    const size_t need = bitcos_gemv_host_staging_bytes(W->M, W->K, batch);
    if (need == 0) return BITCOS_ERR_SHAPE;
    if (staging_bytes < need) return BITCOS_ERR_CAPACITY;
    if (!aligned16(staging)) return BITCOS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint8_t *base = static_cast<uint8_t *>(staging);
    const size_t xb = (static_cast<size_t>(batch) * W->K + 255) / 256 * 256;
    int8_t *x_dev = reinterpret_cast<int8_t *>(base);
    float *xs_dev = reinterpret_cast<float *>(base + xb);
    float *y_dev = reinterpret_cast<float *>(base + xb + 256);
    int rc = check_cuda(cudaMemcpyAsync(x_dev, x_host, static_cast<size_t>(batch) * W->K, cudaMemcpyHostToDevice, stream));
    if (rc) return rc;
    rc = check_cuda(cudaMemcpyAsync(xs_dev, x_scale_host, static_cast<size_t>(batch) * sizeof(float),
                                    cudaMemcpyHostToDevice, stream));
    if (rc) return rc;
    rc = bitcos_gemv(W, x_dev, xs_dev, batch, y_dev, nullptr, workspace, workspace_bytes, cuda_stream);
    if (rc) return rc;
    rc = check_cuda(cudaMemcpyAsync(y_host, y_dev, static_cast<size_t>(batch) * W->M * sizeof(float),
                                    cudaMemcpyDeviceToHost, stream));
    if (rc) return rc;
    return check_cuda(cudaStreamSynchronize(stream));
}

int trit5_gemv(const uint32_t *words, const uint16_t *scales_tiled, int64_t M, int64_t K, const int8_t *x,
               const float *x_scale, int batch, float *y, int32_t *acc_debug, void *workspace,
               size_t workspace_bytes, void *cuda_stream) {
    return gemv_common(kTrit5, words, nullptr, nullptr, scales_tiled, M, K, x, x_scale, batch, y, acc_debug,
                       workspace, workspace_bytes, cuda_stream);
}

int bit2_gemv(const uint32_t *words, const uint16_t *scales_tiled, int64_t M, int64_t K, const int8_t *x,
              const float *x_scale, int batch, float *y, int32_t *acc_debug, void *workspace,
              size_t workspace_bytes, void *cuda_stream) {
    return gemv_common(kBit2, words, nullptr, nullptr, scales_tiled, M, K, x, x_scale, batch, y, acc_debug,
                       workspace, workspace_bytes, cuda_stream);
}

int bitcos_gemv_grouped(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K,
                        const int32_t *group_expert, const int32_t *group_begin, int n_groups,
                        const int32_t *pair_xrow, int n_pairs, int max_group_size, const int8_t *x,
                        const float *x_scale, float *y, int32_t *acc_debug, void *workspace,
                        size_t workspace_bytes, void *cuda_stream) {
    if (!experts || !group_expert || !group_begin || !pair_xrow || !x || !x_scale || !y || !workspace)
        return BITCOS_ERR_NULL;
    if (M < 1 || K < kGroup || K % kGroup != 0 || n_experts < 1 || n_groups < 1 || n_groups > 65535 ||
        n_pairs < n_groups || max_group_size < 1 || max_group_size > BITCOS_MAX_BATCH)
        return BITCOS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y) || !aligned16(workspace) || (acc_debug && !aligned16(acc_debug)))
        return BITCOS_ERR_ALIGN;
    const size_t stride = workspace_bytes_for(M, K);
    if (workspace_bytes < stride * static_cast<size_t>(n_groups)) return BITCOS_ERR_CAPACITY;

    const Plan pl = make_plan(M, K);
    Problem pr{};
    pr.x = x;
    pr.x_scale = x_scale;
    pr.xrow = pair_xrow;
    pr.y = y;
    pr.acc_debug = acc_debug;
    pr.M = M;
    pr.K = K;
    pr.G = static_cast<int>(K / kGroup);
    pr.RB = static_cast<int>(padded_rows(M) / kRows);
    pr.counters = static_cast<unsigned int *>(workspace);
    GroupedArgs ga{experts, group_expert, group_begin, stride, n_experts};
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (max_group_size <= 1) return launch_grouped<1>(pr, pl, ga, n_groups, stream);
    if (max_group_size <= 2) return launch_grouped<2>(pr, pl, ga, n_groups, stream);
    if (max_group_size <= 4) return launch_grouped<4>(pr, pl, ga, n_groups, stream);
    if (max_group_size <= 8) return launch_grouped<8>(pr, pl, ga, n_groups, stream);
    return launch_grouped<16>(pr, pl, ga, n_groups, stream);
}

}  // extern "C"
