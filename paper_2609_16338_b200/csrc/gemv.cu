// Device side of the BITCOS library: ternary GEMV kernels for sm_100a and their C entry
// points (bitcos_gemv, trit5_gemv, bit2_gemv, bitcos_gemv_grouped, bitcos_gemv_host).
//
// Work decomposition (all formats).  Rows are handled 32 at a time (a "row block"), one
// row per lane, so that the activations a warp needs are the same for all of its lanes
// and arrive by broadcast reads; the reduction is cut into groups of 128.  A tile is one
// group of one row block (32 x 128 weights); one warp decodes one tile at a time.  An
// "item" is a run of up to 20 consecutive tiles -- CG groups of one row block, or several
// whole row blocks when a row has few groups -- and is what one thread block processes per
// pipeline stage: because tiles are stored in that order, an item's bitmap words, sign bits,
// scales and entry offsets are four contiguous byte ranges, fetched with four bulk asynchronous
// copies (cp.async.bulk + mbarrier) into a ring of shared-memory stages while earlier stages are
// being decoded.  Thread blocks are persistent and take either a contiguous range of the item
// list or every n-th row-block chunk.  Row sums are formed in a fixed order (a fixed tree over the
// groups inside a block through shared memory; column blocks ascending through a scratch buffer
// and an arrival counter), so results do not depend on scheduling.
//
// Contraction.  One or two tokens: dp4a against activations kept in shared memory.  Four tokens
// and more: the decoded rows pass through a small shared-memory buffer to ldmatrix and
// mma.m16n8k32 (int8 in, int32 out), so that the decode is paid once per call whatever the batch.
//
// BITCOS decode (paper Section II-D, Eq. 4, adapted): the GPU has no bit-deposit
// instruction, so four weights at a time are rebuilt from a (presence nibble, next four
// sign bits) key through a 256-entry table held in shared memory, replicated once per lane
// so that lookups never conflict.  Entries are the four weights as int8 (w = p - 2n, Eq. 2)
// ready for dp4a or the tensor cores.  A lane's position in the sign vector is the tile's entry offset
// plus a warp prefix sum over the rows' population counts; the four 32-bit presence words of
// a lane's row are decoded as four independent chains, each shifting its own sign window by
// the number of sign bits a nibble consumed.
#include "bitcos.h"
#include "decode.cuh"

#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <algorithm>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <utility>
#include <vector>

namespace {

using namespace bitcos_dev;

constexpr int kGroup = BITCOS_GROUP;
constexpr int kRows = BITCOS_TILE_ROWS;
constexpr int kMaxWarps = 20;             // warps per thread block = tiles per item
constexpr int kWarps16 = 14;              // the same for more than 8 tokens (16 warps per block: 128 registers per thread)
constexpr int kMaxStages = 8;             // upper bound on the shared-memory ring depth (Plan::stages)
constexpr uint64_t kWaitLimitNs = 500ull * 1000 * 1000;   // an mbarrier wait gives up after half a second
constexpr int64_t kXResidentBytes = 48 * 1024;   // activations up to this size are kept in shared memory
constexpr int kMmaMinBatch = 4;           // from this many tokens on the contraction runs on the tensor cores
constexpr int kScrRowBytes = 48;          // a quarter of a decoded row (32 int8) + 16 bytes of padding against bank conflicts
constexpr int kScrBytes = kRows * kScrRowBytes;   // per decoder warp: the transposition buffer in front of ldmatrix

enum Format { kBitcos = 0, kTrit5 = 1, kBit2 = 2 };

thread_local int g_last_cuda_error = 0;

// The replicated lookup tables in their shared-memory form (decode.cuh); each thread block fetches
// its copy from global memory with one bulk asynchronous copy.
__device__ __align__(128) const LutBig g_bitcos_lut = make_bitcos_lut();
__device__ __align__(128) const LutBig g_trit5_lut = make_trit5_big();

// ---------------------------------------------------------------------------------------------
// Launch plan and problem description.
// ---------------------------------------------------------------------------------------------
struct Plan {
    int CG;          // groups per column block
    int CS;          // column blocks per row
    int RBC;         // row blocks per item (1 unless CS == 1)
    int NW;          // decoder warps per thread block = ceil(CG * RBC / tpw)
    int tpw;         // tiles of an item per decoder warp: 1, or 2 on large matrices (one or two tokens)
    int64_t items;   // ceil(RB / RBC) * CS
    int cyclic;      // 1: blocks take whole row-block chunks round robin; 0: contiguous balanced ranges
    int stages;      // depth of the shared-memory ring (2 .. kMaxStages), set at launch
    int x_in_stage;  // 1: every stage also receives the item's activation rows (grouped launch, 1-2 tokens)
    int wq, wrem;    // contiguous walk: blocks 0 .. wrem-1 own wq + 1 items, the others wq (set at launch)
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
    unsigned int *status;      // device word set to 1 if an mbarrier wait ran out
    int64_t M, K;
    int G, RB;
    int nb;                    // tokens in this call / group
    int64_t out_row0;          // first output row of y / acc_debug for token 0
};

// Entry offsets of every thread block's first item (sign-vector positions of its first tile and of
// the tile after its last), passed by value when the caller supplied a host copy of tile_off.
constexpr int kMaxGrid = 160;
struct FirstOff {
    uint32_t lo[kMaxGrid];
    uint32_t hi[kMaxGrid];
    int valid;
    // every block's share of the items, worked out on the host (no divisions at kernel start)
    int first[kMaxGrid];
    int count[kMaxGrid];
    int walks;                 // 1: first / count are filled in
};

// Arrays some LATER launch will read (the packed weights of the next products of a layer): every
// thread block asks for its 1 / gridDim.x share of each to be brought into L2 once its own first
// copies are on their way, so that the later launch starts from L2 instead of device memory.
constexpr int kMaxPrefetch = 28;
struct PrefetchList {
    const uint8_t *ptr[kMaxPrefetch];
    uint32_t bytes[kMaxPrefetch];     // multiples of 16
    int n;
#ifdef BITCOS_TIMELINE
    unsigned long long *tl;           // debug build: 16 time stamps per thread block of this launch
#endif
};
#ifdef BITCOS_TIMELINE
#define BITCOS_TLP(src, i)                                                                                              \
    do {                                                                                                                \
        if constexpr (Segs::kHetero)                                                                                    \
            if ((src).pa->tl) (src).pa->tl[static_cast<size_t>(blockIdx.x) * 32 + (src).phase * 6 + (i)] = global_timer_ns(); \
    } while (0)
#else
#define BITCOS_TLP(src, i) \
    do {                   \
    } while (0)
#endif
// What the producer warp needs to send a thread block's first copies on their way, worked out on
// the host for every block of a multi launch: with it the block's first tiles and its lookup table
// are requested a few hundred cycles after the block starts, before any of the block's own address
// arithmetic (arguments, layout, walk, item ranges), which then runs while the data is in flight.
struct FirstCopies {
    const void *src[4];      // entry offsets, bitmap, sign bits, scales of the block's first item
    uint32_t bytes[4];       // (bytes[2] may be 0: an item without a nonzero weight)
    uint32_t dst[4];         // byte offsets inside the block's shared memory
    uint32_t desc[4];        // the item's descriptor for the decoder warps (see issue_item)
    uint32_t desc_off;       // where it goes
    uint32_t bar;            // byte offset of the barrier region
};
struct FirstCopiesTable {
    FirstCopies c[kMaxGrid];
    int valid;
};
// (the table is 14 KB of kernel arguments: free when the launch is recorded into a CUDA graph, whose
// arguments are staged once, but about 4 us of launch latency on a plain stream launch, which therefore
// goes without it)
struct NoFirstCopies {
    int valid;
};
template <typename T>
struct first_copy {
    __device__ static bool sent(const T &, int) { return false; }
};
template <>
struct first_copy<FirstCopiesTable> {
    __device__ static bool sent(const FirstCopiesTable &t, int b) { return t.valid != 0 && t.c[b].bytes[1] != 0; }
};

// Debug build (-DBITCOS_TIMELINE): where a thread block of the multi launch spends its time.
#ifdef BITCOS_TIMELINE
#define BITCOS_TL(i, v)                                                                   \
    do {                                                                                  \
        if (pf && pf->tl) pf->tl[static_cast<size_t>(blockIdx.x) * 32 + (i)] = (v);      \
    } while (0)
#else
#define BITCOS_TL(i, v) \
    do {                \
    } while (0)
#endif

struct GroupedArgs {
    const bitcos_weights *experts;
    const int32_t *group_expert;
    const int32_t *group_begin;
    size_t ws_stride;          // workspace bytes per group
    int n_experts;
    int n_groups;
    int flat;                  // 1: one list of all groups' items, split evenly over the thread blocks
    int n_pairs;               // length of the pair list (outputs, pair_xrow)
    int n_xrows;               // rows of x
    const int32_t *n_groups_dev;   // NULL, or device word holding the number of groups (n_groups is then its upper bound)
};

// A group of a grouped product as its routing lists describe it; ok = false if the lists are
// malformed for it (its pairs outside the pair list, more tokens than the launch was sized for, an
// activation row outside x).  Such a group is skipped -- nothing of it is read or written -- and its
// status word and the launch's (word 0 of the first group's workspace) are set to 2.
struct GroupDesc {
    int e, begin, end;
    bool ok, empty;
};
__device__ __forceinline__ GroupDesc read_group(const GroupedArgs &ga, const int32_t *pair_xrow, unsigned int *status0, int grp,
                                                int nb_max) {
    GroupDesc d;
    d.e = __ldg(ga.group_expert + grp);
    d.begin = __ldg(ga.group_begin + grp);
    d.end = __ldg(ga.group_begin + grp + 1);
    d.empty = d.end <= d.begin;
    d.ok = d.e >= 0 && d.e < ga.n_experts && d.begin >= 0 && d.end <= ga.n_pairs && d.end - d.begin <= nb_max;
    if (d.ok && !d.empty)
        for (int i = d.begin; i < d.end; ++i) {
            const int r = __ldg(pair_xrow + i);
            if (r < 0 || r >= ga.n_xrows) d.ok = false;
        }
    if (!d.ok && !d.empty) {
        *reinterpret_cast<unsigned int *>(reinterpret_cast<uint8_t *>(status0) + static_cast<size_t>(grp) * ga.ws_stride) = 2u;
        *status0 = 2u;
    }
    return d;
}

inline int64_t padded_rows(int64_t M) { return (M + kRows - 1) / kRows * kRows; }

// Decoder warps per thread block: 20, or 14 for more than 8 tokens (the tensor-core path then holds
// 16 accumulators and 16 activation fragments per lane; with 20 warps it spills).
__host__ __device__ constexpr int decoder_warps(int batch) { return batch > 8 ? kWarps16 : kMaxWarps; }
// Threads of the widest block an instantiation for up to nb tokens is launched with.
__host__ __device__ constexpr int max_block_threads(int nb) { return (decoder_warps(nb) + 2) * 32; }

Plan make_plan(int64_t M, int64_t K, int max_warps_per_block, int tpw = 1) {
    const int G = static_cast<int>(K / kGroup);
    const int64_t RB = padded_rows(M) / kRows;
    Plan p{};
    p.tpw = tpw;
    const int max_warps = max_warps_per_block * tpw;       // tiles an item may hold
    const int blocks = (G + max_warps - 1) / max_warps;
    p.CG = (G + blocks - 1) / blocks;
    p.CS = (G + p.CG - 1) / p.CG;
    p.RBC = 1;
    if (p.CS == 1) {
        int64_t r = max_warps / p.CG;
        if (r > RB) r = RB;
        if (r < 1) r = 1;
        p.RBC = static_cast<int>(r);
    }
    p.NW = (p.CG * p.RBC + tpw - 1) / tpw;
    p.items = ((RB + p.RBC - 1) / p.RBC) * p.CS;
    return p;
}

// workspace: [0, 256) header (word 0 = status), arrival counters, partial sums
constexpr size_t kHeaderBytes = 256;
size_t counters_bytes(int64_t RB) { return static_cast<size_t>((RB * 4 + 255) / 256 * 256); }

size_t workspace_bytes_for(int64_t M, int64_t K) {
    const Plan p = make_plan(M, K, kWarps16);        // the plan with the most column blocks
    const int64_t RB = padded_rows(M) / kRows;
    size_t b = kHeaderBytes + counters_bytes(RB);
    if (p.CS > 1) b += static_cast<size_t>(RB) * p.CS * BITCOS_MAX_BATCH * kRows * sizeof(float);
    return b;
}

// Shared-memory layout of a thread block (byte offsets).
struct SmemLayout {
    uint32_t lut;        // lookup tables (0 bytes for 2-bit)
    uint32_t stage;      // stage 0
    uint32_t stage_bytes;
    uint32_t payload_cap, sign_cap, scale_cap, off_cap, x_cap;   // per-stage capacities
    uint32_t x;          // activations, [nb][K], if x_bytes != 0
    uint32_t x_bytes;    // 0: the activations do not fit and are read from global memory
    uint32_t red;        // 2 x [NW][NB][32] floats
    uint32_t scr;        // tensor-core path: NW transposition buffers of kScrBytes
    uint32_t bar;        // mbarriers, then per-stage sign base words
    uint32_t total;
};

__host__ __device__ inline uint32_t align_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

// Partial-sum slots.  Up to two tokens: [warp][token][row] floats.  Tensor-core path:
// [warp][row][token], tokens fastest, so that a decoder lane stores its accumulator pairs (tokens
// 2c, 2c + 1) as one 8-byte word and the epilogue warp reads four tokens per load; token t of row r
// sits at position t ^ red_swizzle(r), which keeps both the stores (lane = row / 4-column pair) and
// the loads (lane = row) free of bank conflicts without padding.
template <int NB>
__host__ __device__ constexpr int red_swizzle(int row) {
    return NB < 8 ? 0 : ((row >> 2) & 1) * 4 + (NB > 8 ? ((row >> 1) & 1) * 8 : 0);
}

// Partial-sum slots between the decoder warps and the epilogue warp (how many items the
// decoders may run ahead of it).
__host__ __device__ constexpr int red_slots(int nbmax) { return nbmax <= 1 ? 8 : nbmax <= 2 ? 4 : 2; }

__host__ __device__ inline SmemLayout smem_layout(int fmt, const Plan &pl, int G, int nbmax, int64_t K) {
    SmemLayout L{};
    uint32_t off = 0;
    L.lut = off;
    off += (fmt == kBit2) ? 0 : kLutBytes;
    const uint32_t tiles = static_cast<uint32_t>(pl.NW * pl.tpw);
    if (fmt == kBitcos) {
        L.payload_cap = tiles * 512;
        L.sign_cap = tiles * 512 + 64;
        L.off_cap = pl.tpw == 2 ? 192 : 128;   // the item's slice of tile_off (at most 21 or 41, + 3 + 3 words)
    } else if (fmt == kTrit5) {
        const uint32_t WPR = (26u * static_cast<uint32_t>(G) + 3) / 4;
        // whole rows when CS == 1, else at most CG groups (+1 shared word) of one row block
        L.payload_cap = (pl.CS == 1) ? static_cast<uint32_t>(pl.RBC) * WPR * 128
                                     : ((26u * static_cast<uint32_t>(pl.CG) + 3) / 4 + 1) * 128;
        L.sign_cap = 0;
    } else {
        L.payload_cap = tiles * 1024;
        L.sign_cap = 0;
    }
    L.scale_cap = tiles * 64;
    L.off_cap = align_up(L.off_cap, 16);
    L.x_cap = pl.x_in_stage ? static_cast<uint32_t>(nbmax * K) : 0u;
    L.stage = off;
    L.stage_bytes = align_up(L.payload_cap + L.sign_cap + L.scale_cap + L.off_cap + L.x_cap, 128);
    off += L.stage_bytes * static_cast<uint32_t>(pl.stages);
    L.x = off;
    // (the tensor-core path takes its activation fragments straight from global memory)
    L.x_bytes = (nbmax < kMmaMinBatch && !pl.x_in_stage && static_cast<int64_t>(nbmax) * K <= kXResidentBytes)
                    ? static_cast<uint32_t>(nbmax * K) : 0u;
    // (at least 128 bytes per decoder warp and token: the products that take 16-bit activations
    // quantise each warp's group into its own slice of this area)
    uint32_t x_area = L.x_bytes;
    if (L.x_bytes && x_area < static_cast<uint32_t>(pl.NW * nbmax * kGroup)) x_area = static_cast<uint32_t>(pl.NW * nbmax * kGroup);
    off += align_up(x_area, 128);
    L.red = off;
    off += static_cast<uint32_t>(red_slots(nbmax) / pl.tpw) * tiles * static_cast<uint32_t>(nbmax) * kRows * 4;
    L.scr = off;
    off += (nbmax >= kMmaMinBatch) ? static_cast<uint32_t>(pl.NW) * kScrBytes : 0u;
    L.bar = off;
    off += 512;          // mbarriers, then (16-byte aligned) one 16-byte item descriptor per stage
    L.total = off;
    return L;
}

// ---------------------------------------------------------------------------------------------
// Device helpers.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bulk asynchronous copy global -> shared; size and both addresses are multiples of 16 bytes.
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Asks for a range of global memory to be brought into L2 (no destination, nothing to wait for);
// the address and the size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_prefetch_l2(const void *src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint32_t mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done;
}
// Polls until the phase completes, for at most limit_ns; false if it gave up.
__device__ __forceinline__ bool mbar_wait_limited(uint32_t bar, uint32_t parity, uint64_t limit_ns) {
    uint64_t t0 = 0;
    for (uint32_t i = 0;; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 15u) == 15u) {
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity) { return mbar_wait_limited(bar, parity, kWaitLimitNs); }
// Waits for the given phase parity (bounded); the common case, an already completed phase, costs
// one instruction.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity);
}

// Four 8x8 matrices of 16-bit elements from shared memory, one row address per lane: as int8 data
// this is exactly the A operand (16 rows x 32 bytes) of mma.m16n8k32.
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&a)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                 : "r"(addr)
                 : "memory");
}
// c[16 x 8] += a[16 x 32] * b[32 x 8], int8 operands, int32 accumulators.
__device__ __forceinline__ void mma_s8(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// c[16 x 8] += a[16 x 16] * b[16 x 8], bf16 operands, fp32 accumulators.
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Four decoded weights (bytes 0x00, 0x01, 0xFF) -> four bf16 values 0, +s, -s (the scale blended
// into the weight, Section II-B): the low three bits of a weight byte (0, 1, 7) pick the high and
// the low byte of its bf16 value out of two small byte tables built from the scale.
//   hi_a / hi_b: bytes {0, s_hi, -, -} / {-, -, -, s_hi | 0x80};  lo_a / lo_b: {0, s_lo, -, -} / {-, -, -, s_lo}
// p01 = (w0, w1), p23 = (w2, w3) as bf16x2.
__device__ __forceinline__ void blend4(uint32_t t, uint32_t hi_a, uint32_t hi_b, uint32_t lo_a, uint32_t lo_b, uint32_t &p01,
                                       uint32_t &p23) {
    uint32_t u = t & 0x07070707u;
    u |= u >> 4;                                   // byte 0: n0 | n1 << 4, byte 2: n2 | n3 << 4
    const uint32_t sel = prmt(u, 0u, 0x4420u);     // n0 | n1 << 4 | n2 << 8 | n3 << 12
    const uint32_t hi = prmt(hi_a, hi_b, sel), lo = prmt(lo_a, lo_b, sel);
    p01 = prmt(lo, hi, 0x5140u);
    p23 = prmt(lo, hi, 0x7362u);
}
__device__ __forceinline__ void sts128(uint32_t addr, int a, int b, int c, int d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Tile decoders.  For the lane's row they produce the 32 int8x4 words of the row; the contraction
// follows as a separate step (dp4a per token, or the tensor cores from four tokens on).
// ---------------------------------------------------------------------------------------------

// int32 accumulator of one row (lane) and group against token activations xg[0..127] (shared memory).
template <int FMT>
__device__ __forceinline__ int contract(const int (&w)[32], const int4 *xg, int lane) {
    if (FMT == kBit2) {
        int a0 = 0, a1 = 0, a2 = 0, a3 = 0;
        // sum of the group's activations, needed because the stored code is weight + 1
        int sx = __dp4a(0x01010101, reinterpret_cast<const int *>(xg)[lane], 0);
        sx = __reduce_add_sync(0xFFFFFFFFu, sx);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int4 xq = xg[q];
            a0 = dp4a_us(static_cast<uint32_t>(w[4 * q + 0]), xq.x, a0);
            a1 = dp4a_us(static_cast<uint32_t>(w[4 * q + 1]), xq.y, a1);
            a2 = dp4a_us(static_cast<uint32_t>(w[4 * q + 2]), xq.z, a2);
            a3 = dp4a_us(static_cast<uint32_t>(w[4 * q + 3]), xq.w, a3);
        }
        return a0 + (a1 >> 2) + (a2 >> 4) + (a3 >> 6) - sx;
    } else {
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
}

// Activation quantiser arithmetic (used by the quantiser kernels and by the products that take
// 16-bit activations): a = max(max |x| over the group, 2^-100), scale = a / 127,
// code = rint(x * (127 / a)), IEEE float32 quotient and product, ties to even.
constexpr float kAmaxFloor = 7.888609052210118e-31f;      // 2^-100

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t quant_code(float x, float inv) {
    int c = __float2int_rn(__fmul_rn(x, inv));
    c = c > 127 ? 127 : (c < -127 ? -127 : c);
    return static_cast<uint32_t>(c) & 0xFFu;
}
// the two values of a 32-bit word -> two codes in the low 16 bits
__device__ __forceinline__ uint32_t quant_pair(uint32_t u, float inv) {
    return quant_code(bf16_lo(u), inv) | (quant_code(bf16_hi(u), inv) << 8);
}

// ---------------------------------------------------------------------------------------------
// The persistent, staged kernel body.
// ---------------------------------------------------------------------------------------------

// Items are numbered row-block chunk major, column block minor: item = c * CS + cs.  A thread
// block owns a CONTIGUOUS range of items (balanced split of all items over the grid), so it
// streams a contiguous piece of the packed matrix and usually sees all column blocks of a row
// block itself; only the row blocks cut by a range boundary need the cross-block protocol.
struct Walk {
    int first, count;   // this block's first item and number of items
    int cstride;        // chunk stride after the last column block of a chunk (1 = contiguous range)
    int q, rem;         // contiguous mode: blocks 0 .. rem-1 own q + 1 items, the others q
};

// Two ways to hand items to thread blocks.  Cyclic: block b takes chunks b, b + n, b + 2n, ...
// with all their column blocks (no row block is ever shared; all blocks read neighbouring
// addresses at any time).  Contiguous: a balanced split of the item list (perfect balance when
// there are few chunks per block, at the price of sharing the row blocks cut by a boundary).
__host__ __device__ __forceinline__ Walk make_walk(const Plan &pl, int block, int n_blocks) {
    Walk w;
    const int items = static_cast<int>(pl.items);
    if (pl.cyclic) {
        const int chunks = items / pl.CS;
        w.first = block * pl.CS;
        w.count = block < chunks ? ((chunks - block + n_blocks - 1) / n_blocks) * pl.CS : 0;
        w.cstride = n_blocks;
        w.q = 1;
        w.rem = 0;
        return w;
    }
    w.q = items / n_blocks;
    w.rem = items - w.q * n_blocks;
    w.first = block * w.q + (block < w.rem ? block : w.rem);
    w.count = w.q + (block < w.rem ? 1 : 0);
    w.cstride = 1;
    return w;
}

// This block's walk: from the launch's table if there is one, else computed here.
__device__ __forceinline__ Walk block_walk(const FirstOff &fo, int index, const Plan &pl, int block, int n_blocks) {
    if (!fo.walks) return make_walk(pl, block, n_blocks);
    Walk w;
    w.first = fo.first[index];
    w.count = fo.count[index];
    w.cstride = pl.cyclic ? n_blocks : 1;
    w.q = pl.wq;
    w.rem = pl.wrem;
    return w;
}

// Which thread block owns an item in contiguous mode (inverse of the split above).
__device__ __forceinline__ int owner_of(const Walk &w, int item) {
    const int big = w.rem * (w.q + 1);
    if (item < big) return item / (w.q + 1);
    return w.rem + (item - big) / w.q;
}

struct ItemRange {
    int rb0;         // first row block
    int cs;          // column block
    int g0;          // first group
    int nt;          // tiles (= busy warps)
    int64_t t0;      // first tile
};

__host__ __device__ __forceinline__ ItemRange item_range(const Problem &pr, const Plan &pl, int c, int cs) {
    ItemRange r;
    r.rb0 = c * pl.RBC;
    r.cs = cs;
    r.g0 = cs * pl.CG;
    if (pl.CS == 1) {
        int nrb = pr.RB - r.rb0;
        if (nrb > pl.RBC) nrb = pl.RBC;
        r.nt = nrb * pr.G;
    } else {
        r.nt = pr.G - r.g0 < pl.CG ? pr.G - r.g0 : pl.CG;
    }
    r.t0 = static_cast<int64_t>(r.rb0) * pr.G + r.g0;
    return r;
}

// (chunk, column block) of an item, and the step to the next item, without divisions in loops
struct ItemIter {
    int c, cs;
    __host__ __device__ __forceinline__ void init(const Plan &pl, int item) {
        if (pl.CS == 1) { c = item; cs = 0; }
        else { c = item / pl.CS; cs = item - c * pl.CS; }
    }
    __host__ __device__ __forceinline__ void next(const Plan &pl, const Walk &w) {
        if (++cs == pl.CS) { cs = 0; c += w.cstride; }
    }
};

// What differs between the segments of one launch (everything else -- shape, activations,
// outputs -- is read from the launch's one Problem), behind accessors: the plain kernels read the
// values from the kernel parameters every time (no registers spent on them), the grouped launch
// holds the current group's values.
struct ParamView {
    __device__ __forceinline__ const uint32_t *payload(const Problem &p) const { return p.payload; }
    __device__ __forceinline__ const uint32_t *signs(const Problem &p) const { return p.signs; }
    __device__ __forceinline__ const uint32_t *tile_off(const Problem &p) const { return p.tile_off; }
    __device__ __forceinline__ const uint16_t *scales(const Problem &p) const { return p.scales; }
    __device__ __forceinline__ const int32_t *xrow(const Problem &p) const { return p.xrow; }       // NULL: token b reads row b
    __device__ __forceinline__ unsigned int *status(const Problem &p) const { return p.status; }
    __device__ __forceinline__ int64_t out_row0(const Problem &p) const { return p.out_row0; }      // first output row of token 0
    __device__ __forceinline__ int nb(const Problem &p) const { return p.nb; }                      // tokens of the segment
};
struct GroupView {
    const uint32_t *payload_, *signs_, *tile_off_;
    const uint16_t *scales_;
    const int32_t *xrow_;
    unsigned int *status_;
    int begin_, nb_;
    __device__ __forceinline__ const uint32_t *payload(const Problem &) const { return payload_; }
    __device__ __forceinline__ const uint32_t *signs(const Problem &) const { return signs_; }
    __device__ __forceinline__ const uint32_t *tile_off(const Problem &) const { return tile_off_; }
    __device__ __forceinline__ const uint16_t *scales(const Problem &) const { return scales_; }
    __device__ __forceinline__ const int32_t *xrow(const Problem &) const { return xrow_; }
    __device__ __forceinline__ unsigned int *status(const Problem &) const { return status_; }
    __device__ __forceinline__ int64_t out_row0(const Problem &) const { return begin_; }
    __device__ __forceinline__ int nb(const Problem &) const { return nb_; }
};

// Issues the bulk copies of one item into stage `s` (one thread) and publishes the item's
// descriptor (sign_base[4s .. 4s+3]; word 3 = index of the first sign bit held in the stage).  o_lo / o_hi: sign-vector
// positions of the item's first tile and of the tile after its last (BITCOS only).
template <int FMT, typename View>
__device__ __forceinline__ void issue_item(const Problem &pb, const View &pr, const Plan &pl, const ItemRange &r,
                                           const SmemLayout &L, uint8_t *smem, int s, uint32_t *sign_base, uint32_t o_lo,
                                           uint32_t o_hi, const int (&xrows)[2], unsigned long long *tl = nullptr) {
#ifdef BITCOS_TIMELINE
#define BITCOS_TLI(i) do { if (tl) tl[i] = clock64(); } while (0)
#else
#define BITCOS_TLI(i) do { } while (0)
#endif
    BITCOS_TLI(21);
    uint8_t *stage = smem + L.stage + static_cast<uint32_t>(s) * L.stage_bytes;
    const uint32_t bar = smem_addr(smem + L.bar) + 8u * static_cast<uint32_t>(s);
    const uint32_t d_payload = smem_addr(stage);
    const uint32_t d_signs = d_payload + L.payload_cap;
    const uint32_t d_scales = d_signs + L.sign_cap;
    const uint32_t scale_bytes = static_cast<uint32_t>(r.nt) * 64u;
    const uint8_t *g_scales = reinterpret_cast<const uint8_t *>(pr.scales(pb)) + r.t0 * 64;
    // what the decoder warps need to know about the item (read by them once the stage is full)
    sign_base[s * 4 + 0] = static_cast<uint32_t>(r.nt) | (static_cast<uint32_t>(r.t0 & 3) << 8);
    sign_base[s * 4 + 1] = static_cast<uint32_t>(r.g0);
    sign_base[s * 4 + 2] = static_cast<uint32_t>(r.rb0);
    const uint32_t x_bytes = pl.x_in_stage ? static_cast<uint32_t>(pr.nb(pb)) * static_cast<uint32_t>(pb.K) : 0u;
    // (issued after the format's expect_tx below; a grouped launch only)
    auto copy_x = [&]() {
        // the activation rows of this group's tokens (from L2): the decoders of a grouped launch
        // find them next to the weights and need no block-wide staging step per group
        if (pl.x_in_stage)
            for (int b = 0; b < pr.nb(pb) && b < 2; ++b)
                bulk_copy(d_scales + L.scale_cap + L.off_cap + static_cast<uint32_t>(b) * static_cast<uint32_t>(pb.K),
                          pb.x + static_cast<int64_t>(xrows[b]) * pb.K, static_cast<uint32_t>(pb.K), bar);
    };
    if (FMT == kBitcos) {
        const uint32_t b_lo = (o_lo >> 7) << 4, b_hi = ((o_hi + 127u) >> 7) << 4;
        const uint32_t sign_bytes = b_hi - b_lo;
        const uint32_t bm_bytes = static_cast<uint32_t>(r.nt) * 512u;
        sign_base[s * 4 + 3] = b_lo * 8u;
        // the tiles' entry offsets: the 16-byte aligned slice of tile_off that covers t0 .. t0 + nt
        const uint32_t o_first = static_cast<uint32_t>(r.t0 & 3);
        const uint32_t off_bytes = ((o_first + static_cast<uint32_t>(r.nt) + 1u + 3u) & ~3u) * 4u;
        BITCOS_TLI(22);
        mbar_expect_tx(bar, bm_bytes + sign_bytes + scale_bytes + off_bytes + x_bytes);
        BITCOS_TLI(23);
        copy_x();
        bulk_copy(d_scales + L.scale_cap, pr.tile_off(pb) + (r.t0 - o_first), off_bytes, bar);
        BITCOS_TLI(24);
        bulk_copy(d_payload, reinterpret_cast<const uint8_t *>(pr.payload(pb)) + r.t0 * 512, bm_bytes, bar);
        BITCOS_TLI(25);
        if (sign_bytes) bulk_copy(d_signs, reinterpret_cast<const uint8_t *>(pr.signs(pb)) + b_lo, sign_bytes, bar);
        BITCOS_TLI(26);
        bulk_copy(d_scales, g_scales, scale_bytes, bar);
        BITCOS_TLI(27);
    } else if (FMT == kTrit5) {
        const int64_t WPR = (26 * static_cast<int64_t>(pb.G) + 3) / 4;
        const int64_t w_lo = r.rb0 * WPR + ((26 * r.g0) >> 2);
        int64_t w_hi;   // exclusive
        if (pl.CS == 1) w_hi = (r.rb0 + r.nt / pb.G) * WPR;
        else w_hi = r.rb0 * WPR + ((26 * (r.g0 + r.nt) - 1) >> 2) + 1;
        const uint32_t bytes = static_cast<uint32_t>(w_hi - w_lo) * 128u;
        mbar_expect_tx(bar, bytes + scale_bytes + x_bytes);
        copy_x();
        bulk_copy(d_payload, reinterpret_cast<const uint8_t *>(pr.payload(pb)) + w_lo * 128, bytes, bar);
        bulk_copy(d_scales, g_scales, scale_bytes, bar);
    } else {
        const uint32_t bytes = static_cast<uint32_t>(r.nt) * 1024u;
        mbar_expect_tx(bar, bytes + scale_bytes + x_bytes);
        copy_x();
        bulk_copy(d_payload, reinterpret_cast<const uint8_t *>(pr.payload(pb)) + r.t0 * 1024, bytes, bar);
        bulk_copy(d_scales, g_scales, scale_bytes, bar);
    }
}

// mbarrier slots inside the `bar` region (8 bytes each)
constexpr int kBarFull = 0;                       // [stages] stage filled by the copy engine
constexpr int kBarEmpty = kMaxStages;             // [stages] stage released (by the epilogue warp, once all decoder warps have posted the item's sums)
constexpr int kBarRedFull = 2 * kMaxStages;       // [slots] partial sums of an item written by all decoder warps
constexpr int kBarRedEmpty = 2 * kMaxStages + 8;  // [slots] partial sums consumed by the epilogue warp
constexpr int kBarLut = 2 * kMaxStages + 16;      // lookup table arrived
constexpr int kBarX = 2 * kMaxStages + 17;        // activations arrived in shared memory (plain kernels, 1-2 tokens)

// Arrival by lane 0 only, as one predicated instruction (no divergent branch around it).
__device__ __forceinline__ void mbar_arrive_lane0(uint32_t bar, int lane) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.s32 p, %1, 0;\n\t"
        "@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(bar), "r"(lane)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// A row block whose column blocks were split over several thread blocks: this block's share.
struct Share {
    int rb;             // row block
    int slot;           // position of this block among the sharers (= order of summation)
    int sharers;        // number of thread blocks holding a piece of the row block
    unsigned int old;   // value of the arrival counter before this block's arrival
};

// If this block's arrival was the last one: add the shares in slot order and write the outputs.
template <int NB, bool XG>
__device__ __forceinline__ void finish_share(const Problem &pr, const Plan &pl, const int (&xr)[NB], const Share &sh,
                                             int lane) {
    const unsigned int old = __shfl_sync(0xFFFFFFFFu, sh.old, 0);
    if (old != static_cast<unsigned int>(sh.sharers - 1)) return;
    __threadfence();
    const int64_t m = static_cast<int64_t>(sh.rb) * kRows + lane;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if (b < pr.nb) {
            float tot = 0.f;
            for (int j = 0; j < sh.sharers; ++j)
                tot += __ldcg(pr.partial + ((static_cast<int64_t>(sh.rb) * pl.CS + j) * pr.nb + b) * kRows + lane);
            if (m < pr.M) pr.y[(pr.out_row0 + b) * pr.M + m] = XG ? tot : __ldg(pr.x_scale + xr[b]) * tot;
        }
    }
    if (lane == 0) pr.counters[sh.rb] = 0u;    // leave the counter ready for the next call
}

// What a thread block runs back to back: one problem and its share of the items (the plain
// kernels), or the pieces of several groups (the grouped launch).  Every warp role walks its own
// copy of the source.
template <bool DEBUG, bool XG = false, bool XQ = false, bool BL = false>
struct OneSegT {
    typedef ParamView View;
    static constexpr bool kSingle = true;      // never more than one segment
    static constexpr bool kHetero = false;     // all segments share one problem shape and one plan
    static constexpr bool kListsLate = false;  // (no routing lists)
    static constexpr bool kDebug = DEBUG;      // false: acc_debug is known to be NULL (no code for it)
    static constexpr bool kGroupScales = XG;   // x_scale holds one scale per token AND group: [nb][G]
    static constexpr bool kQuantize = XQ;      // x holds bf16 activations: quantised per group of 128 by the decoder warps
    static constexpr bool kBlend = BL;         // x holds bf16 activations, used as they are against weights +-s (tensor cores)
    const Problem *pr;
    Walk wk;
    bool used;
    __device__ __forceinline__ const Problem &shape() const { return *pr; }
    __device__ __forceinline__ int block_in_job(int block) const { return block; }
    __device__ __forceinline__ bool next(View &v, Walk &w) {
        if (used) return false;
        used = true;
        (void)v;
        w = wk;
        return true;
    }
};

// This block's share of the arrays a later launch will read, requested into L2: entries first,
// first + step, ...
__device__ __forceinline__ void prefetch_share(const PrefetchList *pf, int first, int step) {
    const uint32_t nblk = gridDim.x, bid = blockIdx.x;
    for (int i = first; i < pf->n; i += step) {
        const uint32_t total = pf->bytes[i];
        const uint32_t chunk = ((total / 16u + nblk - 1u) / nblk) * 16u;
        const uint32_t off = bid * chunk;
        if (off < total) bulk_prefetch_l2(pf->ptr[i] + off, total - off < chunk ? total - off : chunk);
    }
}

// Warp roles: warps 0 .. NW-1 decode one tile per item each; warp NW adds the decoders' partial
// sums in a fixed order and writes the outputs (and runs the cross-block protocol); the block's
// LAST warp (known without reading a kernel argument) feeds the stage ring with bulk copies.  The roles meet only through mbarriers, every
// wait is bounded, and there is no block-wide barrier inside the loop.
// `segs` yields the problems this block works on, one after the other, with its share of each
// one's items; the stage ring, the partial-sum slots and their barriers run on across them.
template <int FMT, int NB, int TPW, typename Segs>
__device__ __forceinline__ void run_segments(const Segs &segs, const Plan &pl_in, uint8_t *smem, int block,
                                             const FirstOff *fo = nullptr, int fo_index = 0, const PrefetchList *pf = nullptr,
                                             bool first_sent = false) {
    // first_sent: the caller has already initialised the barriers of stage 0 and of the lookup table
    // and issued the table's copy and the copies of this block's first item (send_first_copies)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int prod_warp = static_cast<int>(blockDim.x >> 5) - 1;      // the producer: always the block's last warp
    if (static_cast<int>(threadIdx.x) == prod_warp * 32) BITCOS_TL(16, clock64());
    // The problem and the plan of the segment a warp role is working on.  The plain and the grouped
    // launches have one shape and one plan for all their segments.  A phased launch (kHetero) moves
    // from job to job: only what the shared-memory layout and the barrier counts need -- the widest
    // plan, the longest row -- is common (pl_in, segs.shape()), and every role re-binds pb / pl to its
    // own copy of the current job's problem and plan.
    const Problem *pbp = &segs.shape();
    const Plan *plp = &pl_in;
#define pb (*pbp)
#define pl (*plp)
    const SmemLayout L = smem_layout(FMT, pl, segs.shape().G, NB, segs.shape().K);
    typename Segs::View pr{};
    Walk wk{};
    const uint8_t *lut = smem + L.lut;
    float *red = reinterpret_cast<float *>(smem + L.red);
    // per stage: {tiles | (first tile & 3) << 8, first group, first row block, first sign bit held}
    uint32_t *sign_base = reinterpret_cast<uint32_t *>(smem + L.bar + 384);
    const uint32_t bar0 = smem_addr(smem + L.bar);
    static_assert(TPW == 1 || (TPW == 2 && NB < kMmaMinBatch), "two tiles per warp: one or two tokens only");
    // one activation scale per token and group (applied by the decoder warps, tile by tile)
    // instead of one per token (applied by the epilogue warp to the finished sums)
    constexpr bool kXQ = Segs::kQuantize;                      // (one or two tokens only)
    constexpr bool kBlend = Segs::kBlend;                      // (tensor-core path, up to eight tokens)
    static_assert(!kBlend || (NB == 8 && FMT == kBitcos && TPW == 1), "blended weights: the eight-token BITCOS kernel");
    constexpr bool kXG = Segs::kGroupScales || kXQ || kBlend;   // no token scale in the epilogue
    static_assert(!kXQ || NB < kMmaMinBatch, "16-bit activations: one or two tokens only");
    const uint32_t red_slot = static_cast<uint32_t>(pl.NW * TPW) * NB * kRows;     // floats per partial-sum slot
    // partial-sum slots in use: red_slots(NB), half as many (of twice the size) with two tiles per warp
    constexpr int rs_log2 = (red_slots(NB) == 8 ? 3 : red_slots(NB) == 4 ? 2 : 1) - (TPW - 1);
    constexpr int rs_mask = (1 << rs_log2) - 1;

    // Programmatic dependent launch: the next kernel in the stream may be scheduled as soon as
    // every block of this one got here; whatever it reads from us it reads after its own
    // griddepcontrol.wait.
    // (every thread: a trigger from one warp alone measured 0.02 us per layer pass faster, which is not worth
    // depending on how a block's trigger is counted)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // A block launched wider than this problem needs (several problems in one launch): the spare
    // warps only take part in the one block-wide barrier.
    if (warp > pl.NW && warp < prod_warp) {
        __syncthreads();
        return;
    }

    // ------------------------------------------------------------------ producer warp
    // It also sets the barriers up, so that the first copies are in flight before anything else
    // happens in the block.
    if (warp == prod_warp) {
        if (lane == 0) {
            BITCOS_TL(13, clock64());
            BITCOS_TL(0, global_timer_ns());
            BITCOS_TL(17, clock64());
        }
        // All 33 barrier slots at once, one per lane (slots of unused stages included): slots
        // kBarRedFull .. kBarRedFull + 7 count the decoder warps, the others one arrival.  Every
        // barrier is initialised and fenced before the first asynchronous copy is issued.
        static_assert(kBarFull == 0 && kBarEmpty == 8 && kBarRedFull == 16 && kBarRedEmpty == 24 && kBarLut == 32,
                      "one barrier slot per lane, plus the table's");
        if (!(first_sent && lane == kBarFull))
            mbar_init(bar0 + 8u * static_cast<uint32_t>(lane), (lane >= kBarRedFull && lane < kBarRedEmpty) ? pl.NW : 1);
        if (lane == 0 && !first_sent) mbar_init(bar0 + 8u * kBarLut, 1);
        if (lane == 1) mbar_init(bar0 + 8u * kBarX, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        __syncwarp();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the other lanes' barriers, seen by this lane's copies
        if (lane == 0) BITCOS_TL(14, clock64());
        // The first copies go out before the block-wide barrier below, while the other warps are
        // still fetching the activations.
        // Entry offsets are requested two items before they are needed (r0 = item k, r1 = item
        // k + 1, r2 = item k + 2), so that the load is never waited for.
        Segs src = segs;
        if constexpr (Segs::kHetero) {
            pbp = src.problem_ptr();
            plp = src.plan_ptr();
        }
        ItemIter it2;
        ItemRange r0{}, r1{}, r2{};
        uint32_t lo0 = 0, hi0 = 0, lo1 = 0, hi1 = 0;
        int k0 = 0, ps = 0;
        int kk = 0;                // items issued so far, over all segments
        int xrows[2] = {0, 0};     // activation rows of the segment's tokens (when they travel with the stage)
        uint32_t pphase = 1;       // parity of the phase before the one the decoders complete next
        bool ok = true;
        auto offsets = [&](const ItemRange &r, uint32_t &lo, uint32_t &hi) {
            if (FMT != kBitcos) return;
            // two independent loads (no reuse of the previous item's upper offset: that would make
            // every request wait for the one before it)
            lo = __ldg(pr.tile_off(pb) + r.t0);
            hi = __ldg(pr.tile_off(pb) + r.t0 + r.nt);
        };
        auto second_item = [&]() {
            if (wk.count > 1) {
                it2.next(pl, wk);
                r1 = item_range(pb, pl, it2.c, it2.cs);
                offsets(r1, lo1, hi1);
            }
        };
        auto issue_loop = [&](int k_end) {
            for (int k = k0; k < k_end; ++k, ++kk) {
                const int s = ps;
                uint32_t lo2 = 0, hi2 = 0;
                // (the block's very first item goes out before anything is worked out for the items after it)
                auto look_ahead = [&]() {
                    if (k + 2 < wk.count) {
                        it2.next(pl, wk);
                        r2 = item_range(pb, pl, it2.c, it2.cs);
                        offsets(r2, lo2, hi2);
                    }
                };
                if (kk != 0) look_ahead();
                if (kk >= pl.stages) {
                    if (!mbar_wait(bar0 + 8u * (kBarEmpty + s), pphase)) {
                        if (pr.status(pb)) *pr.status(pb) = 1u;
                        ok = false;
                        return;
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                if (!(first_sent && kk == 0)) {
#ifdef BITCOS_TIMELINE
                    issue_item<FMT>(pb, pr, pl, r0, L, smem, s, sign_base, lo0, hi0, xrows,
                                    (kk == 0 && pf && pf->tl) ? pf->tl + static_cast<size_t>(blockIdx.x) * 32 : nullptr);
#else
                    issue_item<FMT>(pb, pr, pl, r0, L, smem, s, sign_base, lo0, hi0, xrows);
#endif
                }
                if (kk == 0) {
                    second_item();
                    look_ahead();
                }
                r0 = r1; lo0 = lo1; hi0 = hi1;
                r1 = r2; lo1 = lo2; hi1 = hi2;
                if (++ps == pl.stages) {
                    ps = 0;
                    pphase ^= 1u;
                }
            }
            k0 = k_end;
        };
        // first item(s) of a segment: ranges and entry offsets of items 0 and 1 (the block's first
        // segment: of item 0 only; item 1 follows once item 0 is on its way)
        auto prime = [&](bool first_segment) {
            k0 = 0;
            it2.init(pl, wk.first);
            r0 = item_range(pb, pl, it2.c, it2.cs);
            if (FMT == kBitcos) {
                if (first_segment && fo && fo->valid) {
                    lo0 = fo->lo[fo_index];
                    hi0 = fo->hi[fo_index];
                } else {
                    lo0 = __ldg(pr.tile_off(pb) + r0.t0);
                    hi0 = __ldg(pr.tile_off(pb) + r0.t0 + r0.nt);
                }
            }
            if (!first_segment) second_item();
            if (pl.x_in_stage) {
                xrows[0] = pr.xrow(pb) ? __ldg(pr.xrow(pb)) : 0;
                xrows[1] = pr.nb(pb) > 1 ? (pr.xrow(pb) ? __ldg(pr.xrow(pb) + 1) : 1) : 0;
            }
        };
        // A grouped launch reads its routing lists (which may come from the previous kernel in the
        // stream) to find its first item: the table copy, which depends on nothing, goes out before
        // the wait for that kernel.
        bool lut_issued = first_sent;
        if constexpr (Segs::kListsLate) {
            if (lane == 0 && FMT != kBit2) {
                mbar_expect_tx(bar0 + 8u * kBarLut, kLutBytes);
                bulk_copy(smem_addr(smem + L.lut), FMT == kBitcos ? g_bitcos_lut.v : g_trit5_lut.v, kLutBytes,
                          bar0 + 8u * kBarLut);
                lut_issued = true;
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
        }
        bool have = src.next(pr, wk);
        while (have && wk.count <= 0) have = src.next(pr, wk);
        // The lookup table first: it is the largest transfer of the start-up (64 KB from L2) and
        // needs no address arithmetic.
        if (lane == 0 && have && FMT != kBit2 && !lut_issued) {
            mbar_expect_tx(bar0 + 8u * kBarLut, kLutBytes);
            bulk_copy(smem_addr(smem + L.lut), FMT == kBitcos ? g_bitcos_lut.v : g_trit5_lut.v, kLutBytes,
                      bar0 + 8u * kBarLut);
        }
        if (lane == 0) BITCOS_TL(15, clock64());
        // Only the first item goes out before the block-wide barrier: issuing a bulk copy costs this
        // thread on the order of a hundred nanoseconds, and the other warps wait at that barrier.
        // (first item already sent by the kernel's first instructions: its bookkeeping waits until
        // the other warps have been let through the block-wide barrier)
        if (lane == 0 && have && !first_sent) {
            prime(true);
            BITCOS_TL(18, clock64());
            issue_loop(1);
        }
        if (lane == 0) BITCOS_TL(2, clock64());
        __syncthreads();       // pairs with the barrier the other warps reach after staging the activations
        if (lane == 0) BITCOS_TL(12, clock64());
        if (lane == 0 && have && first_sent) {
            prime(true);
            issue_loop(1);
        }
        if (lane == 0 && !have && lut_issued && !first_sent) mbar_wait(bar0 + 8u * kBarLut, 0);      // no copy may outlive the block
        // The hint for a later launch goes out behind this block's own first copies (as many as the
        // ring holds): measured, requests issued before them or from another warp gain less.
        if (pf && lane == 0) {
            if (have && ok) issue_loop(wk.count < pl.stages ? wk.count : pl.stages);
            prefetch_share(pf, 0, 1);
        }
        if (lane != 0 || !have) return;
        if (ok) issue_loop(wk.count);
        while (!Segs::kSingle && ok && src.next(pr, wk)) {
            if (wk.count <= 0) continue;
            prime(false);
            issue_loop(wk.count);
        }
        return;
    }

    // What may depend on the previous kernel in the stream: activations, routing lists, outputs,
    // workspace.  The packed weights do not, so the producer never waits, and in the plain kernels
    // with one or two tokens (kEarly) the decoder warps do not either until they have decoded
    // their first tile: only the contraction needs the activations, which the epilogue warp
    // fetches into shared memory (one bulk copy per token) as soon as the dependency is resolved.
    // With four tokens and more (tensor-core path) the decoders fetch their activation fragments
    // from global memory right after that first decode instead.
    constexpr bool kLate = Segs::kSingle || Segs::kHetero;      // plain and phased kernels: wait as late as possible
    constexpr bool kEarly = kLate && NB < kMmaMinBatch;         // ... and activations copied by the epilogue warp
    if (!kLate) asm volatile("griddepcontrol.wait;" ::: "memory");

    Segs src = segs;
    if constexpr (Segs::kHetero) {
        pbp = src.problem_ptr();
        plp = src.plan_ptr();
    }
    bool have = src.next(pr, wk);
    while (have && wk.count <= 0) have = src.next(pr, wk);
    auto next_segment = [&]() {
        if (Segs::kSingle) return false;
        bool more = src.next(pr, wk);
        while (more && wk.count <= 0) more = src.next(pr, wk);
        return more;
    };

    // activations of one or two tokens: kept whole in shared memory ([nb][K]), staged by these
    // warps while the producer starts the copies (plain kernels: one segment), or delivered with
    // every stage (grouped launch); the tensor-core path reads its fragments from global memory
    int xr[NB];
    auto token_rows = [&]() {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const int bb = b < pr.nb(pb) ? b : 0;
            xr[b] = pr.xrow(pb) ? __ldg(pr.xrow(pb) + bb) : bb;
        }
    };
    if (have && !kLate) token_rows();
    const bool x_resident = L.x_bytes != 0;
    if (x_resident && have && !kEarly) {
        int4 *xs = reinterpret_cast<int4 *>(smem + L.x);
        const int per_tok = static_cast<int>(pb.K / 16);
        const int nthr = (pl.NW + 1) * 32;                   // the decoder warps and the epilogue warp
        const int tid = threadIdx.x;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b < pr.nb(pb)) {
                const int4 *src = reinterpret_cast<const int4 *>(pb.x + static_cast<int64_t>(xr[b]) * pb.K);
                for (int q = tid; q < per_tok; q += nthr) xs[b * per_tok + q] = __ldg(src + q);
            }
        }
    }
    __syncthreads();          // barriers initialised, activations in place
    if (!have) return;

    // ------------------------------------------------------------------ epilogue warp
    if (warp == pl.NW) {
        // the segment's activations into shared memory: one bulk copy per token (one or two tokens)
        auto fetch_x = [&]() {
            token_rows();
            if (kEarly && !kXQ && lane == 0) {
                mbar_expect_tx(bar0 + 8u * kBarX, static_cast<uint32_t>(pr.nb(pb)) * static_cast<uint32_t>(pb.K));
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    if (b < pr.nb(pb))
                        bulk_copy(smem_addr(smem + L.x) + static_cast<uint32_t>(b) * static_cast<uint32_t>(pb.K),
                                  pb.x + static_cast<int64_t>(xr[b]) * pb.K, static_cast<uint32_t>(pb.K), bar0 + 8u * kBarX);
            }
        };
        if (kLate) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            if (lane == 0) BITCOS_TL(8, clock64());
            if (!Segs::kHetero) fetch_x();
        }
        float run[NB];          // running sum of the current row block over this block's items
#pragma unroll
        for (int b = 0; b < NB; ++b) run[b] = 0.f;
        // per-token activation scales: kept in registers for up to two tokens, fetched where they
        // are used (a cached load per output block) for more
        float xsc[NB < kMmaMinBatch ? NB : 1] = {};
        auto xscale = [&](int b) {
            return kXG ? 1.f : NB < kMmaMinBatch ? xsc[NB < kMmaMinBatch ? b : 0] : __ldg(pb.x_scale + xr[b]);
        };
        Share pend[2];
        int n_pend = 0;
        ItemIter it;
        int kk = 0;             // items consumed so far, over all segments
        int es = 0;             // stage of the item the epilogue looks at next
        constexpr int RS = red_slots(NB);
        // sum of n <= 20 partial sums of token b, spaced NB * 32 floats apart: all loads are issued
        // before the first addition, and the additions always follow the same tree
        auto sum_groups20 = [&](const float *base, int n) {
            float v[kMaxWarps];
#pragma unroll
            for (int j = 0; j < kMaxWarps; ++j) v[j] = (j < n) ? base[j * NB * kRows] : 0.f;
#pragma unroll
            for (int w2 = 1; w2 < kMaxWarps; w2 *= 2)
#pragma unroll
                for (int j = 0; j + w2 < kMaxWarps; j += 2 * w2) v[j] += v[j + w2];
            return v[0];
        };
        // (up to 40 partial sums when a warp decodes two tiles per item: two trees of 20)
        auto sum_groups = [&](const float *base, int n) {
            float t = sum_groups20(base, n);
            if (TPW == 2 && n > kMaxWarps) t += sum_groups20(base + kMaxWarps * NB * kRows, n - kMaxWarps);
            return t;
        };
        // tensor-core layout: the same for four tokens at a time, n <= 20 float4 spaced one warp's
        // rows apart, in two batches of ten to bound the registers in flight
        constexpr int RF = NB;
        auto sum_groups4 = [&](const float *base, int n) {
            float4 tot = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j0 = 0; j0 < kMaxWarps; j0 += 10) {
                float4 v[10];
#pragma unroll
                for (int j = 0; j < 10; ++j)
                    v[j] = (j0 + j < n) ? *reinterpret_cast<const float4 *>(base + (j0 + j) * kRows * RF)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w2 = 1; w2 < 10; w2 *= 2)
#pragma unroll
                    for (int j = 0; j + w2 < 10; j += 2 * w2) {
                        v[j].x += v[j + w2].x;
                        v[j].y += v[j + w2].y;
                        v[j].z += v[j + w2].z;
                        v[j].w += v[j + w2].w;
                    }
                tot.x += v[0].x;
                tot.y += v[0].y;
                tot.z += v[0].z;
                tot.w += v[0].w;
            }
            return tot;
        };
        // sums over warps j0 .. j0 + n - 1 of a slot, for this lane's row and every token
        auto sums = [&](const float *rs, int j0, int n, float (&tot)[NB]) {
            if (NB >= kMmaMinBatch) {
#pragma unroll
                for (int t = 0; t < NB / 4; ++t) {
                    float4 v4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (4 * t < pr.nb(pb)) v4 = sum_groups4(rs + (j0 * kRows + lane) * RF + ((4 * t) ^ red_swizzle<NB>(lane)), n);
                    tot[4 * t + 0] = v4.x;
                    tot[4 * t + 1] = v4.y;
                    tot[4 * t + 2] = v4.z;
                    tot[4 * t + 3] = v4.w;
                }
            } else {
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    tot[b] = (b < pr.nb(pb)) ? sum_groups(rs + (j0 * NB + b) * kRows + lane, n) : 0.f;
            }
        };
        do {
        if constexpr (Segs::kHetero) {
            // A phased launch: this segment's activations (and whatever else its job reads) may be
            // written by the jobs of the phase before it, so they are fetched only once every thread
            // block has finished that phase.  All decoder warps have left the previous segment's
            // contractions by now (its last partial sums were consumed above), so the one activation
            // buffer is free.
            if (!src.wait_dependency(lane)) {
                if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
                return;
            }
            if (lane == 0) BITCOS_TLP(src, 0);
            fetch_x();
        }
        n_pend = 0;
        it.init(pl, wk.first);
        if (NB < kMmaMinBatch && !kXG) {
#pragma unroll
            for (int b = 0; b < NB; ++b) xsc[NB < kMmaMinBatch ? b : 0] = __ldg(pb.x_scale + xr[b]);
        }
        for (int k = 0; k < wk.count; ++k, ++kk, it.next(pl, wk)) {
            const int slot = kk & rs_mask;
            const ItemRange r = item_range(pb, pl, it.c, it.cs);
            if (!mbar_wait(bar0 + 8u * (kBarRedFull + slot), static_cast<uint32_t>((kk >> rs_log2) & 1))) {
                if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
                return;
            }
            // every decoder warp has posted this item's sums, so none of them reads its stage any more:
            // one arrival per item hands the stage back to the producer
            if (lane == 0) mbar_arrive(bar0 + 8u * (kBarEmpty + es));
            if (++es == pl.stages) es = 0;
            const float *rs = red + slot * red_slot;
            if (pl.CS == 1) {
                // whole row blocks: one output per row.  The sums are formed first, the slot is
                // handed back, and only then are the outputs stored, so that the release of the
                // slot never waits for a global store.
                const int nrb = r.nt / pb.G;
                for (int i = 0; i < nrb; ++i) {
                    const int64_t m = static_cast<int64_t>(r.rb0 + i) * kRows + lane;
                    float t_b[NB];
                    sums(rs, i * pb.G, pb.G, t_b);
                    if (i == nrb - 1) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar0 + 8u * (kBarRedEmpty + slot));
                    }
#pragma unroll
                    for (int b = 0; b < NB; ++b)
                        if (b < pr.nb(pb) && m < pb.M) pb.y[(pr.out_row0(pb) + b) * pb.M + m] = xscale(b) * t_b[b];
                }
                continue;
            }
            // one column block of row block rb0: add it to the running sum
            const bool starts = (r.cs == 0) || (k == 0);
            float t_b[NB];
            sums(rs, 0, r.nt, t_b);
#pragma unroll
            for (int b = 0; b < NB; ++b) run[b] = starts ? t_b[b] : run[b] + t_b[b];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar0 + 8u * (kBarRedEmpty + slot));
            const bool ends = (r.cs == pl.CS - 1) || (k == wk.count - 1);
            if (!ends) continue;
            const int first_cs = (k >= r.cs) ? 0 : r.cs - k;       // first column block of rb0 seen by this block
            const int64_t m = static_cast<int64_t>(r.rb0) * kRows + lane;
            if (first_cs == 0 && r.cs == pl.CS - 1) {
                // the whole row block was ours
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    if (b < pr.nb(pb) && m < pb.M) pb.y[(pr.out_row0(pb) + b) * pb.M + m] = xscale(b) * run[b];
            } else {
                // shared row block: publish our share, then count ourselves in
                Share sh;
                sh.rb = r.rb0;
                const int lo = owner_of(wk, r.rb0 * pl.CS), hi = owner_of(wk, r.rb0 * pl.CS + pl.CS - 1);
                sh.slot = src.block_in_job(block) - lo;
                sh.sharers = hi - lo + 1;
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    if (b < pr.nb(pb))
                        pb.partial[((static_cast<int64_t>(sh.rb) * pl.CS + sh.slot) * pr.nb(pb) + b) * kRows + lane] = run[b];
                __syncwarp();
                sh.old = 0;
                if (lane == 0) {
                    __threadfence();
                    sh.old = atomicAdd(pb.counters + sh.rb, 1u);
                }
                pend[n_pend++] = sh;      // at most two per block: its first and its last row block
            }
        }
        for (int i = 0; i < n_pend; ++i) finish_share<NB, kXG>(pb, pl, xr, pend[i], lane);
        if constexpr (Segs::kHetero) src.signal_done(lane);      // this block's outputs of the phase are written
        if (lane == 0) BITCOS_TLP(src, 5);
        have = next_segment();
        if (have && !Segs::kHetero) token_rows();
        } while (have);
        if (lane == 0) {
            BITCOS_TL(9, clock64());
            BITCOS_TL(11, global_timer_ns());
        }
        return;
    }

    // ------------------------------------------------------------------ decoder warps
    // CS == 1: tile t of an item always is row block t / G of the chunk, group t % G; this warp
    // decodes tile `warp` and, with two tiles per warp, tile `warp + NW`
    constexpr int tpw = TPW;
    // (a phased launch works these out again for every job)
    int my_rbl0 = (pl.CS == 1) ? warp / pb.G : 0;
    int g_fixed0 = warp - my_rbl0 * pb.G;
    int my_rbl1 = (pl.CS == 1) ? (warp + pl.NW) / pb.G : 0;
    int g_fixed1 = warp + pl.NW - my_rbl1 * pb.G;
    uint32_t x_parity = 0;      // phase parity of the activations' barrier: one phase per segment of a phased launch
    if (FMT != kBit2) {
        if (!mbar_wait(bar0 + 8u * kBarLut, 0)) {
            if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
            return;
        }
    }
    if (warp == 0 && lane == 0) BITCOS_TL(3, clock64());
    bool tl_first = true;
    constexpr int RS = red_slots(NB);
    constexpr bool kMma = NB >= kMmaMinBatch;          // contraction on the tensor cores
    constexpr int NH = NB > 8 ? 2 : 1;                 // 8-token halves of the batch
    constexpr int NV = kMma ? NH * 8 : NB;             // partial sums a lane hands to the epilogue warp
    const uint32_t lane4 = static_cast<uint32_t>(lane) * 4u;
    // Tensor-core path.  The order of the 128 products inside a group is free, so it is chosen to
    // make the activation loads contiguous: of tokens lane / 4 and lane / 4 + 8 this lane holds
    // bytes 16 c .. 16 c + 15 and 64 + 16 c .. 64 + 16 c + 15 of the group (c = lane % 4, two 16-byte
    // loads), and k-block kb of the contraction pairs words 2 kb and 2 kb + 1 of those eight with
    // the matching weight words.  A operand: each lane stores the row it decoded into the warp's
    // buffer (32 int8 at a time, in that order), ldmatrix brings it back in fragment order.
    const int8_t *xfrag[NH];
    auto token_fragments = [&]() {
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const int n = 8 * h + (lane >> 2);
            xfrag[h] = nullptr;
            if (kMma && n < pr.nb(pb))
                xfrag[h] = kBlend ? pb.x + static_cast<int64_t>(n) * pb.K * 2 + 64 * (lane & 3)
                                  : pb.x + static_cast<int64_t>(pr.xrow(pb) ? __ldg(pr.xrow(pb) + n) : n) * pb.K + 16 * (lane & 3);
        }
    };
    // (blended weights: of token lane / 4 this lane holds bytes 64 c .. 64 c + 63 of the group's 256,
    // four 16-byte loads; k-step j of the contraction uses words 2 j and 2 j + 1 of those sixteen)
    uint32_t bf[NH][kBlend ? 16 : 8];
    float xgq[NH][2];           // group scales of the two tokens whose accumulators this lane holds
    auto load_bf = [&](int g) {
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            if constexpr (kBlend) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    int4 u = make_int4(0, 0, 0, 0);
                    if (xfrag[h]) u = __ldg(reinterpret_cast<const int4 *>(xfrag[h] + static_cast<int64_t>(g) * (2 * kGroup)) + q);
                    bf[h][4 * q + 0] = u.x; bf[h][4 * q + 1] = u.y;
                    bf[h][4 * q + 2] = u.z; bf[h][4 * q + 3] = u.w;
                }
                continue;
            }
            if (kXG && !kXQ) {
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int b = 8 * h + 2 * (lane & 3) + r;
                    xgq[h][r] = (b < pr.nb(pb)) ? __ldg(pb.x_scale + static_cast<int64_t>(b) * pb.G + g) : 0.f;
                }
            }
            int4 u0 = make_int4(0, 0, 0, 0), u1 = make_int4(0, 0, 0, 0);
            if (xfrag[h]) {
                const int4 *px = reinterpret_cast<const int4 *>(xfrag[h] + static_cast<int64_t>(g) * kGroup);
                u0 = __ldg(px);
                u1 = __ldg(px + 4);
            }
            bf[h][0] = u0.x; bf[h][1] = u0.y; bf[h][2] = u0.z; bf[h][3] = u0.w;
            bf[h][4] = u1.x; bf[h][5] = u1.y; bf[h][6] = u1.z; bf[h][7] = u1.w;
        }
    };

    const uint32_t scr0 = smem_addr(smem + L.scr) + static_cast<uint32_t>(warp) * kScrBytes;
    const uint32_t scr_st = scr0 + static_cast<uint32_t>(lane) * kScrRowBytes;
    const uint32_t scr_ld = scr0 + static_cast<uint32_t>((lane & 7) + ((lane >> 3) & 1) * 8) * kScrRowBytes +
                            static_cast<uint32_t>(lane >> 4) * 16u;
    const uint8_t *stage0 = smem + L.stage;
    const uint8_t *stage = stage0;
    const uint4 *desc = reinterpret_cast<const uint4 *>(sign_base);
    uint32_t full_bar = bar0 + 8u * kBarFull, phase = 0;
    int s = 0;
    // byte offsets inside a stage that do not change from item to item (first tile of this warp;
    // the second one lies NW tiles further)
    const uint32_t tile_lane0 = static_cast<uint32_t>(warp * kRows + lane);
    const uint32_t off_bm0 = tile_lane0 * 16u;                                       // this lane's four presence words
    const uint32_t off_scale0 = L.payload_cap + L.sign_cap + tile_lane0 * 2u;          // its row's group scale
    const uint32_t off_toff0 = L.payload_cap + L.sign_cap + L.scale_cap + static_cast<uint32_t>(warp) * 4u;
    const uint32_t off_sign = L.payload_cap;
    const uint32_t tile_step = static_cast<uint32_t>(pl.NW);
    const uint32_t off_x = L.payload_cap + L.sign_cap + L.scale_cap + L.off_cap;     // activations inside a stage
    const uint8_t *xs_base = smem + L.x;
    // where this lane leaves its partial sums inside a slot (one or two tokens)
    float *rd_lane0 = red + static_cast<uint32_t>(warp * NB) * kRows + lane;
    int kk = 0;                 // items decoded so far, over all segments
    bool x_ready = false;
    // 16-bit activations: the group this warp has quantised last, its scales, and its buffer
    // ([token][128] int8 inside the activation area)
    int q_g = -1;
    float q_scale[NB < kMmaMinBatch ? NB : 1] = {};
    uint32_t *q_scr = reinterpret_cast<uint32_t *>(smem + L.x) + static_cast<uint32_t>(warp) * (NB * kRows);
    bool more_segments = false;
    do {
    if (!(kLate && kMma)) {
        token_fragments();
        // whole rows per item: this warp's group never changes, neither do its activation fragments
        if (kMma && pl.CS == 1) load_bf(g_fixed0);
    }
    for (const int kk_end = kk + wk.count; kk < kk_end; ++kk) {
        if (!mbar_wait(full_bar, phase)) {
            if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
            return;
        }
        if (tl_first && warp == 0 && lane == 0) BITCOS_TL(4, clock64());
        if (tl_first && warp == 0 && lane == 0) BITCOS_TLP(src, 1);
        const uint4 d = desc[s];
        const int nt = static_cast<int>(d.x & 0xFFu);
        const int slot = kk & rs_mask;
        // Two tiles per warp: the partial sums of a tile are stored as soon as it is done, so the
        // slot must be free before the first one (with one tile per warp that wait comes after
        // the decode, further down).
        if (tpw == 2 && (kk >> rs_log2) > 0) {
            if (!mbar_wait(bar0 + 8u * (kBarRedEmpty + slot), static_cast<uint32_t>(((kk >> rs_log2) - 1) & 1))) {
                if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
                return;
            }
        }
        float ysum[NV];
#pragma unroll 1
        for (int ti = 0; ti < tpw; ++ti) {
        const int tile = warp + (ti ? pl.NW : 0);
        const bool busy = tile < nt;
        const int my_rbl = ti ? my_rbl1 : my_rbl0;
        // group of this tile: the item's first group (0 when items are whole rows) + the tile's
        // place in its row block
        const int g = static_cast<int>(d.y) + (ti ? g_fixed1 : g_fixed0);
        const uint32_t t_off = ti ? tile_step : 0u;
        const uint32_t off_bm = off_bm0 + t_off * (kRows * 16u);
        const uint32_t off_scale = off_scale0 + t_off * (kRows * 2u);
        const uint32_t off_toff = off_toff0 + t_off * 4u;
#pragma unroll
        for (int b = 0; b < NV; ++b) ysum[b] = 0.f;
        // early, so that the decode hides the latency (not before the dependency is resolved)
        if (kMma && pl.CS != 1 && busy && (!kLate || x_ready)) load_bf(g);
        // 16-bit activations of a group this warp has not quantised yet: fetched ahead of the decode too
        uint2 qv[NB < kMmaMinBatch ? NB : 1];
        bool q_have = false;
        auto fetch_group = [&]() {
#pragma unroll
            for (int b = 0; b < NB; ++b)
                if (NB == 1 || b < pr.nb(pb))
                    qv[NB < kMmaMinBatch ? b : 0] =
                        __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(pb.x) + static_cast<int64_t>(b) * pb.K +
                                                              static_cast<int64_t>(g) * kGroup) + lane);
            q_have = true;
        };
        if (kXQ && busy && x_ready && g != q_g) fetch_group();

        if (busy) {
            const float sc = bf16_to_float(*reinterpret_cast<const uint16_t *>(stage + off_scale));
            // activations of group g (one or two tokens: always in shared memory)
            // (only the grouped launch ever delivers activations with the stage)
            const uint8_t *xs = kXQ ? reinterpret_cast<const uint8_t *>(q_scr)
                                    : ((!Segs::kSingle && pl.x_in_stage) ? stage + off_x : xs_base) + static_cast<uint32_t>(g) * kGroup;
            int w[32];
            if (FMT == kBitcos) {
                const uint4 bm = *reinterpret_cast<const uint4 *>(stage + off_bm);
                const int c = __popc(bm.x) + __popc(bm.y) + __popc(bm.z) + __popc(bm.w);
                int incl = c;
#pragma unroll
                for (int dd = 1; dd < 32; dd <<= 1) {
                    const int v = __shfl_up_sync(0xFFFFFFFFu, incl, dd);
                    if (lane >= dd) incl += v;
                }
                // entry offset of this tile: word (t0 & 3) + warp of the stage's slice of tile_off
                const uint32_t toff = *reinterpret_cast<const uint32_t *>(stage + off_toff + ((d.x >> 8) << 2));
                const uint32_t cursor = toff + static_cast<uint32_t>(incl - c) - d.w;
                const uint32_t *sp = reinterpret_cast<const uint32_t *>(stage + off_sign + ((cursor >> 5) << 2));
                bitcos_decode_row(bm, sp, cursor & 31u, lut, lane4, w);
            } else if (FMT == kTrit5) {
                const int WPR = (26 * pb.G + 3) / 4;
                // words of the stage: row block my_rbl of the chunk, counted from the chunk's first word
                const int w_rel = my_rbl * WPR + ((26 * g) >> 2) - ((26 * static_cast<int>(d.y)) >> 2);
                const uint32_t *src = reinterpret_cast<const uint32_t *>(stage) + w_rel * kRows + lane;
                uint32_t wd[7];
#pragma unroll
                for (int i = 0; i < 7; ++i) wd[i] = src[i * kRows];
                trit5_decode_row(wd, g & 1, lut, static_cast<uint32_t>(lane) * 8u, w);
            } else {
                const uint4 *src = reinterpret_cast<const uint4 *>(stage) + (tile * 2) * kRows + lane;
                if (kMma) bit2_decode_row_s8(src[0], src[kRows], w);
                else bit2_decode_row(src[0], src[kRows], w);
            }
            if (kLate && kMma && !x_ready) {
                // first contraction of this warp: the previous kernel must be complete before the
                // activations are read (the decode above did not need them)
                asm volatile("griddepcontrol.wait;" ::: "memory");
                token_fragments();
                load_bf(g);
                x_ready = true;
            }
            if constexpr (kBlend) {
                // Weights +-s as bf16 against the unquantised activations: eight k-steps of sixteen
                // products.  K-step j takes weight word j of each of the row's four 32-weight runs
                // (k = 32 c + 4 j .. + 3), which is the order the activation words above are held in.
                float accf[NH][2][4];
#pragma unroll
                for (int h = 0; h < NH; ++h)
#pragma unroll
                    for (int mh = 0; mh < 2; ++mh)
#pragma unroll
                        for (int r = 0; r < 4; ++r) accf[h][mh][r] = 0.f;
                const uint32_t sbits = *reinterpret_cast<const uint16_t *>(stage + off_scale);
                const uint32_t s_hi = sbits >> 8, s_lo = sbits & 0xFFu;
                const uint32_t hi_a = s_hi << 8, hi_b = (s_hi | 0x80u) << 24, lo_a = s_lo << 8, lo_b = s_lo << 24;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (j) __syncwarp();             // everyone has read the previous block back
                    uint32_t p01[4], p23[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) blend4(static_cast<uint32_t>(w[8 * c + j]), hi_a, hi_b, lo_a, lo_b, p01[c], p23[c]);
                    sts128(scr_st, p01[0], p01[1], p01[2], p01[3]);
                    sts128(scr_st + 16u, p23[0], p23[1], p23[2], p23[3]);
                    __syncwarp();
#pragma unroll
                    for (int mh = 0; mh < 2; ++mh) {
                        uint32_t a[4];
                        ldmatrix_x4(a, scr_ld + static_cast<uint32_t>(mh * 16 * kScrRowBytes));
#pragma unroll
                        for (int h = 0; h < NH; ++h) mma_bf16(accf[h][mh], a, bf[h][2 * j], bf[h][2 * j + 1]);
                    }
                }
#pragma unroll
                for (int h = 0; h < NH; ++h)
#pragma unroll
                    for (int mh = 0; mh < 2; ++mh)
#pragma unroll
                        for (int r = 0; r < 4; ++r) ysum[(h * 2 + mh) * 4 + r] = accf[h][mh][r];
            } else if (kMma) {
                int acc[NH][2][4];
#pragma unroll
                for (int h = 0; h < NH; ++h)
#pragma unroll
                    for (int mh = 0; mh < 2; ++mh)
#pragma unroll
                        for (int r = 0; r < 4; ++r) acc[h][mh][r] = 0;
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {
                    // 32 weights of every row through the buffer: one k-block of the contraction
                    if (kb) __syncwarp();            // everyone has read the previous block back
                    const int w0 = (kb < 2) ? 2 * kb : 16 + 2 * (kb - 2);     // first weight word of this block
                    sts128(scr_st, w[w0], w[w0 + 4], w[w0 + 8], w[w0 + 12]);
                    sts128(scr_st + 16u, w[w0 + 1], w[w0 + 5], w[w0 + 9], w[w0 + 13]);
                    __syncwarp();
#pragma unroll
                    for (int mh = 0; mh < 2; ++mh) {
                        uint32_t a[4];
                        ldmatrix_x4(a, scr_ld + static_cast<uint32_t>(mh * 16 * kScrRowBytes));
#pragma unroll
                        for (int h = 0; h < NH; ++h) mma_s8(acc[h][mh], a, bf[h][2 * kb], bf[h][2 * kb + 1]);
                    }
                }
                // accumulator r of (h, mh): row 16 mh + lane / 4 + 8 (r / 2), token 8 h + 2 (lane % 4) + (r & 1)
                float scq[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) scq[j] = __shfl_sync(0xFFFFFFFFu, sc, (lane >> 2) + 8 * j);
#pragma unroll
                for (int h = 0; h < NH; ++h)
#pragma unroll
                    for (int mh = 0; mh < 2; ++mh)
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            ysum[(h * 2 + mh) * 4 + r] = scq[2 * mh + (r >> 1)] * static_cast<float>(acc[h][mh][r]);
                            if (kXG) ysum[(h * 2 + mh) * 4 + r] *= xgq[h][r & 1];
                            if (Segs::kDebug && pb.acc_debug) {
                                const int b = 8 * h + 2 * (lane & 3) + (r & 1);
                                const int64_t m = (static_cast<int64_t>(d.z) + my_rbl) * kRows + 16 * mh + (lane >> 2) + 8 * (r >> 1);
                                if (b < pr.nb(pb) && m < pb.M) pb.acc_debug[((pr.out_row0(pb) + b) * pb.M + m) * pb.G + g] = acc[h][mh][r];
                            }
                        }
            }
            // decode first, contract afterwards: keeps the table lookups of the decode back to back
            // (interleaving them with the contraction's activation loads measured 20 % slower on the
            // five-trit path)
            if (!kMma) asm volatile("" ::: "memory");
            if (kEarly && !x_ready) {
                // first contraction of this warp: the previous kernel must be complete and the
                // activations in place (the decode above needed neither)
                if (tl_first && warp == 0 && lane == 0) BITCOS_TL(5, clock64());
                if (tl_first && warp == 0 && lane == 0) BITCOS_TLP(src, 2);
                asm volatile("griddepcontrol.wait;" ::: "memory");
                if (!kXQ && !mbar_wait(bar0 + 8u * kBarX, x_parity)) {
                    if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
                    return;
                }
                x_ready = true;
                if (tl_first && warp == 0 && lane == 0) BITCOS_TL(6, clock64());
                if (tl_first && warp == 0 && lane == 0) BITCOS_TLP(src, 3);
            }
            if (kXQ && g != q_g) {
                // 16-bit activations: this warp quantises the group its tile multiplies (four values
                // per lane, largest magnitude by shuffles) into its own 128 bytes per token
                if (!q_have) fetch_group();        // (first tile: the dependency has only just been resolved)
                __syncwarp();                     // the previous tile's contraction has read the buffer
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (NB == 1 || b < pr.nb(pb)) {
                        const uint2 v = qv[NB < kMmaMinBatch ? b : 0];
                        float a = fmaxf(fmaxf(fabsf(bf16_lo(v.x)), fabsf(bf16_hi(v.x))),
                                        fmaxf(fabsf(bf16_lo(v.y)), fabsf(bf16_hi(v.y))));
#pragma unroll
                        for (int dd = 16; dd; dd >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, dd));
                        a = fmaxf(a, kAmaxFloor);
                        const float inv = __fdiv_rn(127.0f, a);
                        q_scale[NB < kMmaMinBatch ? b : 0] = __fdiv_rn(a, 127.0f);
                        q_scr[b * kRows + lane] = quant_pair(v.x, inv) | (quant_pair(v.y, inv) << 16);
                    }
                }
                __syncwarp();
                q_g = g;
            }
            float xgs[NB < kMmaMinBatch ? NB : 1];
            if (kXQ) {
#pragma unroll
                for (int b = 0; b < NB; ++b) xgs[NB < kMmaMinBatch ? b : 0] = q_scale[NB < kMmaMinBatch ? b : 0];
            } else if (kXG && !kMma) {
                // (after the dependency wait: the scales come from the kernel before this one)
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    if (NB == 1 || b < pr.nb(pb))
                        xgs[NB < kMmaMinBatch ? b : 0] = __ldg(pb.x_scale + static_cast<int64_t>(b) * pb.G + g);
            }
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (kMma) break;
                if (NB == 1 || b < pr.nb(pb)) {       // a call has at least one token
                    const int a = contract<FMT>(w, reinterpret_cast<const int4 *>(xs + static_cast<uint32_t>(b) * (kXQ ? static_cast<uint32_t>(kGroup) : static_cast<uint32_t>(pb.K))), lane);
                    ysum[b] = sc * static_cast<float>(a);
                    if (kXG) ysum[b] *= xgs[NB < kMmaMinBatch ? b : 0];
                    if (Segs::kDebug && pb.acc_debug) {
                        const int64_t m = (static_cast<int64_t>(d.z) + my_rbl) * kRows + lane;
                        if (m < pb.M) pb.acc_debug[((pr.out_row0(pb) + b) * pb.M + m) * pb.G + g] = a;
                    }
                }
            }
        }
        if (tpw == 2) {
            // (one or two tokens only) this tile's partial sums, zeros if the item has no such tile
#pragma unroll
            for (int b = 0; b < NB; ++b)
                if (!kMma) rd_lane0[slot * red_slot + (t_off * NB + b) * kRows] = ysum[b];
        }
        }
        // (the stage goes back to the producer when the epilogue warp has seen this item's partial sums)
        stage += L.stage_bytes;
        full_bar += 8u;
        if (++s == pl.stages) {
            s = 0;
            stage = stage0;
            full_bar = bar0 + 8u * kBarFull;
            phase ^= 1u;
        }

        // partial sums for the epilogue warp (several slots, so decoders may run ahead of it)
        if (tpw == 1 && (kk >> rs_log2) > 0) {
            if (!mbar_wait(bar0 + 8u * (kBarRedEmpty + slot), static_cast<uint32_t>(((kk >> rs_log2) - 1) & 1))) {
                if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
                return;
            }
        }
        float *rd = red + slot * red_slot;
        if (tpw == 2) {
            // already stored, tile by tile
        } else if (kMma) {
#pragma unroll
            for (int i = 0; i < NV; i += 2) {
                const int b = 8 * (i >> 3) + 2 * (lane & 3);                          // and b + 1
                const int row = 16 * ((i >> 2) & 1) + (lane >> 2) + 8 * ((i >> 1) & 1);
                if (b < NB)
                    *reinterpret_cast<float2 *>(rd + (warp * kRows + row) * NB + (b ^ red_swizzle<NB>(row))) =
                        make_float2(ysum[i], ysum[i + 1]);
            }
        } else {
#pragma unroll
            for (int b = 0; b < NB; ++b) rd_lane0[slot * red_slot + b * kRows] = ysum[b];
        }
        __syncwarp();
        mbar_arrive_lane0(bar0 + 8u * (kBarRedFull + slot), lane);
        if (tl_first && warp == 0 && lane == 0) BITCOS_TL(7, clock64());
        tl_first = false;
    }
    if (warp == 0 && lane == 0) BITCOS_TL(10, clock64());
    if (warp == 0 && lane == 0) BITCOS_TLP(src, 4);
    if constexpr (Segs::kHetero) {
        // Every decoder warp passes every phase of the activations' barrier, a warp without a tile in
        // this segment included: a warp that skipped one could not tell the phase before from the
        // phase after by its parity.
        if (!x_ready && !mbar_wait(bar0 + 8u * kBarX, x_parity)) {
            if (lane == 0 && pr.status(pb)) *pr.status(pb) = 1u;
            return;
        }
        more_segments = next_segment();
        tl_first = true;
        if (more_segments) {
            x_ready = false;
            x_parity ^= 1u;
            my_rbl0 = (pl.CS == 1) ? warp / pb.G : 0;
            g_fixed0 = warp - my_rbl0 * pb.G;
            my_rbl1 = (pl.CS == 1) ? (warp + pl.NW) / pb.G : 0;
            g_fixed1 = warp + pl.NW - my_rbl1 * pb.G;
        }
    } else {
        more_segments = next_segment();
    }
    } while (more_segments);
#undef pb
#undef pl
}

// One problem, this block's share of its items.
template <int FMT, int NB, bool DEBUG = true, int TPW = 1, bool XG = false, bool XQ = false, bool BL = false>
__device__ __forceinline__ void run_problem(const Problem &pr, const Plan &pl, uint8_t *smem, const Walk &wk, int block,
                                            const FirstOff *fo = nullptr, int fo_index = 0, const PrefetchList *pf = nullptr,
                                            bool first_sent = false) {
    OneSegT<DEBUG, XG, XQ, BL> one;
    one.pr = &pr;
    one.wk = wk;
    one.used = false;
    run_segments<FMT, NB, TPW>(one, pl, smem, block, fo, fo_index, pf, first_sent);
}

template <int FMT, int NB, int TPW = 1, bool XG = false, bool XQ = false, bool BL = false>
__global__ void __launch_bounds__(max_block_threads(NB), 1) gemv_kernel(const Problem pr, const Plan pl,
                                                                        const __grid_constant__ FirstOff fo) {
    extern __shared__ __align__(128) uint8_t smem[];
    run_problem<FMT, NB, !BL, TPW, XG, XQ, BL>(pr, pl, smem,
                         block_walk(fo, static_cast<int>(blockIdx.x), pl, static_cast<int>(blockIdx.x), static_cast<int>(gridDim.x)),
                         static_cast<int>(blockIdx.x), &fo, static_cast<int>(blockIdx.x));
}

// Several independent BITCOS problems in one launch: the grid is cut into one range of thread
// blocks per problem, and every block runs the ordinary kernel body on its problem.
constexpr int kMaxJobs = BITCOS_MAX_JOBS;
struct MultiArgs {
    Problem pr[kMaxJobs];
    Plan pl[kMaxJobs];
    int first_block[kMaxJobs + 1];
    int n;
    // mapped = 1: block b works on job job_of[b] as that job's block number rank[b] of nblk[job]
    // (the jobs' blocks interleaved); 0: job j owns blocks first_block[j] .. first_block[j + 1] - 1
    int mapped;
    int nblk[kMaxJobs];
    uint8_t job_of[kMaxGrid];
    uint8_t rank[kMaxGrid];
    PrefetchList pf;
};

template <int NB, int TPW = 1, bool XQ = false, bool XG = false, typename FC = NoFirstCopies>
__global__ void __launch_bounds__(max_block_threads(NB), 1) gemv_multi_kernel(const __grid_constant__ MultiArgs ma,
                                                                              const __grid_constant__ FirstOff fo,
                                                                              const __grid_constant__ FC fc) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int b = static_cast<int>(blockIdx.x);
    // The block's first copies, from the host's table: before anything else is read or worked out.
    const bool first_sent = first_copy<FC>::sent(fc, b);
    if constexpr (std::is_same<FC, FirstCopiesTable>::value)
    if (first_sent && threadIdx.x == blockDim.x - 32) {
        const FirstCopies &c = fc.c[b];
        const uint32_t base = smem_addr(smem);
        const uint32_t bar_full = base + c.bar + 8u * kBarFull, bar_lut = base + c.bar + 8u * kBarLut;
        mbar_init(bar_full, 1);
        mbar_init(bar_lut, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // (the descriptor before the arrival below, which publishes it to the decoder warps)
        *reinterpret_cast<uint4 *>(smem + c.desc_off) = make_uint4(c.desc[0], c.desc[1], c.desc[2], c.desc[3]);
        mbar_expect_tx(bar_full, c.bytes[0] + c.bytes[1] + c.bytes[2] + c.bytes[3]);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (i != 2 || c.bytes[2]) bulk_copy(base + c.dst[i], c.src[i], c.bytes[i], bar_full);
        mbar_expect_tx(bar_lut, kLutBytes);
        bulk_copy(base, g_bitcos_lut.v, kLutBytes, bar_lut);
    }
#ifdef BITCOS_TIMELINE
    if (threadIdx.x == blockDim.x - 32 && ma.pf.tl) ma.pf.tl[static_cast<size_t>(blockIdx.x) * 32 + 1] = clock64();
#endif
    int j = 0, bj, nbj;
    if (ma.mapped) {
        j = ma.job_of[b];
        bj = ma.rank[b];
        nbj = ma.nblk[j];
    } else {
        while (j + 1 < ma.n && b >= ma.first_block[j + 1]) ++j;
        bj = b - ma.first_block[j];
        nbj = ma.first_block[j + 1] - ma.first_block[j];
    }
    const Plan pl = ma.pl[j];      // by value: read through the run-time index once, not at every use
    const Problem pr = ma.pr[j];
    const Walk wk0 = block_walk(fo, b, pl, bj, nbj);
    // (the multi launch has no accumulator dump)
#ifdef BITCOS_TIMELINE
    if (threadIdx.x == blockDim.x - 32 && ma.pf.tl) ma.pf.tl[static_cast<size_t>(blockIdx.x) * 32 + 20] = clock64();
#endif
    run_problem<kBitcos, NB, false, TPW, XG, XQ>(pr, pl, smem, wk0,
                             bj, &fo, b,
#ifdef BITCOS_TIMELINE
                             &ma.pf
#else
                             ma.pf.n ? &ma.pf : nullptr
#endif
                             , first_sent);
}

// ---------------------------------------------------------------------------------------------
// Phased launch: jobs in dependency order inside ONE launch.  The jobs of phase p may read what the
// jobs of phase p - 1 wrote (a decoder layer's o projection follows q, k and v; down follows gate
// and up), so a thread block fetches a job's activations only after every block has finished the
// phase before it.  Everything that does not depend on the phase before -- the packed weights, their
// decode -- runs ahead: the producer warp streams the next phase's tiles while the current one is
// being decoded, and every decoder warp decodes its first tile of the next phase before it waits.
// Blocks are persistent and at most one per multiprocessor, so all of them are resident together
// and the wait on the phase counter cannot starve; it is bounded like every other wait here.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxPhases = BITCOS_MAX_PHASES;
struct PhasedArgs {
    Problem pr[kMaxJobs];
    Plan pl[kMaxJobs];                      // every plan with the layout's NW and stages
    Plan layout;                            // the widest plan: shared-memory layout, barrier counts, block size
    Problem shape;                          // K = the longest row (layout only)
    int job_first_block[kMaxJobs];          // a job's range of thread blocks inside its phase
    int job_blocks[kMaxJobs];
    int expect[kMaxPhases];                 // thread blocks that have items in the phase
    int n_phases;
    unsigned int *sync;                     // device: one arrival counter per phase, zero between launches
    uint8_t job_of[kMaxPhases][kMaxGrid];   // the job a thread block works on in a phase (0xFF: none)
#ifdef BITCOS_TIMELINE
    unsigned long long *tl;
#endif
};


__device__ __forceinline__ unsigned int load_acquire(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// The segments of one thread block of a phased launch: in every phase, its share of one job.
template <bool XG>
struct PhasedSegs {
    typedef ParamView View;
    static constexpr bool kSingle = false;
    static constexpr bool kHetero = true;
    static constexpr bool kListsLate = false;
    static constexpr bool kDebug = false;
    static constexpr bool kGroupScales = XG;
    static constexpr bool kQuantize = false;
    static constexpr bool kBlend = false;
    const PhasedArgs *pa;
    int block;               // blockIdx.x
    int next_phase;          // phase the next call of next() looks at
    int phase;               // phase of the current segment
    int rel_block;           // this block's index inside the current job's range
    Problem cur_pb;
    Plan cur_pl;
    __device__ __forceinline__ const Problem &shape() const { return pa->shape; }
    __device__ __forceinline__ const Problem *problem_ptr() const { return &cur_pb; }
    __device__ __forceinline__ const Plan *plan_ptr() const { return &cur_pl; }
    __device__ __forceinline__ int block_in_job(int) const { return rel_block; }
    __device__ __forceinline__ bool next(View &, Walk &w) {
        while (next_phase < pa->n_phases) {
            const int p = next_phase++;
            const int j = pa->job_of[p][block];
            if (j == 0xFF) continue;
            const int rel = block - pa->job_first_block[j];
            const Walk wj = make_walk(pa->pl[j], rel, pa->job_blocks[j]);
            if (wj.count <= 0) continue;
            cur_pb = pa->pr[j];
            cur_pl = pa->pl[j];
            w = wj;
            phase = p;
            rel_block = rel;
            return true;
        }
        return false;
    }
    // Epilogue warp, before it fetches the current segment's activations: every block that has items
    // in the phase before must have written its outputs.  false if the wait ran out.
    __device__ __forceinline__ bool wait_dependency(int lane) const {
        if (phase == 0) return true;
        bool ok = true;
        if (lane == 0) {
            const unsigned int *ctr = pa->sync + (phase - 1);
            const unsigned int want = static_cast<unsigned int>(pa->expect[phase - 1]);
            uint64_t t0 = 0;
            for (uint32_t i = 0; load_acquire(ctr) < want; ++i) {
                if ((i & 15u) == 15u) {
                    const uint64_t now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kWaitLimitNs) {
                        ok = false;
                        break;
                    }
                }
            }
            // what the other blocks wrote, ordered before this block's asynchronous copies
            asm volatile("fence.proxy.async;" ::: "memory");
        }
        return __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
    }
    // Epilogue warp, after the last output of the current segment: count this block in.  The last
    // arrival of the last phase leaves every counter zero for the next launch (by then no block
    // reads an earlier counter any more: each one read it before it arrived here).
    __device__ __forceinline__ void signal_done(int lane) const {
        __syncwarp();
        if (lane != 0) return;
        __threadfence();
        const unsigned int old = atomicAdd(pa->sync + phase, 1u);
        if (phase == pa->n_phases - 1 && old + 1u == static_cast<unsigned int>(pa->expect[phase])) {
            for (int p = 0; p < pa->n_phases; ++p) pa->sync[p] = 0u;
        }
    }
};

template <int NB, bool XG = false>
__global__ void __launch_bounds__(max_block_threads(NB), 1) gemv_phased_kernel(const __grid_constant__ PhasedArgs pa) {
    extern __shared__ __align__(128) uint8_t smem[];
    PhasedSegs<XG> segs;
    segs.pa = &pa;
    segs.block = static_cast<int>(blockIdx.x);
    segs.next_phase = 0;
    segs.phase = 0;
    segs.rel_block = 0;
    run_segments<kBitcos, NB, 1>(segs, pa.layout, smem, static_cast<int>(blockIdx.x));
}

// Fills in what differs between the groups of a grouped product; false if the group is empty or
// names no expert.
template <int NB>
__device__ __forceinline__ bool grouped_problem(Problem &pr, const Problem &base, const GroupedArgs &ga, int grp) {
    const GroupDesc gd = read_group(ga, base.xrow, base.status, grp, NB);
    if (!gd.ok || gd.empty) return false;
    const int e = gd.e, begin = gd.begin, end = gd.end;
    const bitcos_weights wdesc = ga.experts[e];
    pr = base;
    pr.payload = wdesc.bitmap;
    pr.signs = wdesc.signs;
    pr.tile_off = wdesc.tile_off;
    pr.scales = wdesc.scales;
    pr.nb = min(end - begin, NB);
    pr.xrow = base.xrow + begin;
    pr.out_row0 = begin;
    uint8_t *ws = reinterpret_cast<uint8_t *>(base.status) + static_cast<size_t>(grp) * ga.ws_stride;
    pr.status = reinterpret_cast<unsigned int *>(ws);
    pr.counters = reinterpret_cast<unsigned int *>(ws + kHeaderBytes);
    pr.partial = reinterpret_cast<float *>(ws + kHeaderBytes + ((static_cast<size_t>(base.RB) * 4 + 255) / 256 * 256));
    return true;
}

// The pieces of the groups that fall into one thread block's range of the flat item list.
template <int NB>
struct GroupedSegs {
    const Problem *base;
    const GroupedArgs *ga;
    int64_t lo, hi, ipg;      // this block's range of the list; items per group
    int grp;                  // group of item lo
    typedef GroupView View;
    static constexpr bool kSingle = false;
    static constexpr bool kHetero = false;
    static constexpr bool kListsLate = true;   // the routing lists are read only after the previous kernel has completed
    static constexpr bool kDebug = true;
    static constexpr bool kGroupScales = false;
    static constexpr bool kQuantize = false;
    static constexpr bool kBlend = false;
    __device__ __forceinline__ const Problem &shape() const { return *base; }
    __device__ __forceinline__ int block_in_job(int block) const { return block; }
    __device__ __forceinline__ bool next(View &v, Walk &w) {
        while (lo < hi) {
            const int64_t g_lo = static_cast<int64_t>(grp) * ipg;
            const int64_t seg_hi = hi < g_lo + ipg ? hi : g_lo + ipg;
            w.first = static_cast<int>(lo - g_lo);
            w.count = static_cast<int>(seg_hi - lo);
            w.cstride = 1;
            w.q = 1;
            w.rem = 0;
            lo = seg_hi;
            const int g = grp++;
            const GroupDesc gd = read_group(*ga, base->xrow, base->status, g, NB);
            if (!gd.ok || gd.empty) continue;
            const int e = gd.e, begin = gd.begin, end = gd.end;
            const bitcos_weights *wd = ga->experts + e;
            v.payload_ = wd->bitmap;
            v.signs_ = wd->signs;
            v.tile_off_ = wd->tile_off;
            v.scales_ = wd->scales;
            v.xrow_ = base->xrow + begin;
            v.status_ = reinterpret_cast<unsigned int *>(reinterpret_cast<uint8_t *>(base->status) +
                                                         static_cast<size_t>(g) * ga->ws_stride);
            v.begin_ = begin;
            v.nb_ = min(end - begin, NB);
            return true;
        }
        return false;
    }
};

// Grouped product.  Two launch shapes.  Flat (rows in one piece, no cross-block sums): the items
// of all groups form one list, cut into equal contiguous ranges, one per thread block; a block
// that crosses from one group to the next keeps its pipeline running (the producer is already
// copying the next group's weights while the last tiles of this one are decoded).  Otherwise:
// blockIdx.y = group, and the blocks of a row of the grid share that group's items.
template <int FMT, int NB>
__global__ void __launch_bounds__(max_block_threads(NB), 1) gemv_grouped_kernel(const __grid_constant__ Problem base, const Plan pl,
                                                                                const __grid_constant__ GroupedArgs ga) {
    extern __shared__ __align__(128) uint8_t smem[];
    int n_groups = ga.n_groups;
    if (ga.n_groups_dev) {
        // the number of groups itself comes from the device (a grouping kernel earlier in the stream)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const int n = __ldg(ga.n_groups_dev);
        n_groups = n < 0 ? 0 : (n < n_groups ? n : n_groups);
    }
    if (!ga.flat) {
        // the routing lists may come from the previous kernel in the stream
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (static_cast<int>(blockIdx.y) >= n_groups) return;
        Problem pr;
        if (!grouped_problem<NB>(pr, base, ga, static_cast<int>(blockIdx.y))) return;
        run_problem<FMT, NB>(pr, pl, smem, make_walk(pl, static_cast<int>(blockIdx.x), static_cast<int>(gridDim.x)),
                                 static_cast<int>(blockIdx.x));
        return;
    }
    const int64_t ipg = pl.items, total = ipg * n_groups;
    const int64_t nblk = gridDim.x, b = blockIdx.x;
    const int64_t q = total / nblk, rem = total - q * nblk;
    GroupedSegs<NB> segs;
    segs.base = &base;
    segs.ga = &ga;
    segs.ipg = ipg;
    segs.lo = b * q + (b < rem ? b : rem);
    segs.hi = segs.lo + q + (b < rem ? 1 : 0);
    segs.grp = static_cast<int>(segs.lo / ipg);
    run_segments<FMT, NB, 1>(segs, pl, smem, static_cast<int>(b));
}

// ---------------------------------------------------------------------------------------------
// Decode-rate probe: what the paper's roofline calls gamma -- the cost of the unpack sequence when
// every operand is already on chip (Section III-B.1, Eq. 6).  Each warp decodes one synthetic tile
// that sits in shared memory, `iters` times, with the same code the GEMV kernels run (popcounts,
// prefix sum, sign windows, table lookups, dp4a); nothing is read from global memory inside the
// timed loop.  cycles[block] receives the block's elapsed clock cycles.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t probe_hash(uint32_t v) {
    v ^= v >> 16; v *= 0x7FEB352Du; v ^= v >> 15; v *= 0x846CA68Bu; v ^= v >> 16;
    return v;
}

template <int FMT>
__global__ void __launch_bounds__((kMaxWarps + 2) * 32, 1) decode_probe_kernel(int iters, unsigned long long *cycles, int *sink) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    uint8_t *lut = smem;
    uint8_t *tiles = smem + (FMT == kBit2 ? 0 : kLutBytes);          // per warp: 1024 B payload + 640 B signs + 64 B scales
    uint8_t *xs = tiles + nw * 1792;                                   // 128 activations
    constexpr uint32_t kTile = 1792;
    if (FMT != kBit2) {
        const uint32_t *src = FMT == kBitcos ? g_bitcos_lut.v : g_trit5_lut.v;
        for (int i = threadIdx.x; i < kLutBytes / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(lut)[i] = src[i];
    }
    // synthetic tile: presence bits set with probability 0.5625, random sign bits, valid five-trit bytes
    uint32_t *mine = reinterpret_cast<uint32_t *>(tiles + warp * kTile);
    for (int i = lane; i < kTile / 4; i += 32) {
        const uint32_t h1 = probe_hash(i * 4u + 1), h2 = probe_hash(i * 4u + 2), h3 = probe_hash(i * 4u + 3),
                       h4 = probe_hash(i * 4u + 4);
        uint32_t v = h1 | (h2 & h3 & h4);
        if (FMT == kTrit5) v = ((h1 & 0xFFu) % 243u) | (((h2 & 0xFFu) % 243u) << 8) | (((h3 & 0xFFu) % 243u) << 16) |
                               (((h4 & 0xFFu) % 243u) << 24);
        if (FMT == kBit2) v = (h1 | (h2 & h3 & h4)) & 0x55555555u;
        mine[i] = v;
    }
    for (int i = threadIdx.x; i < 32; i += blockDim.x) reinterpret_cast<uint32_t *>(xs)[i] = probe_hash(1000u + i);
    __syncthreads();
    const uint8_t *stage = tiles + warp * kTile;
    const uint32_t lane4 = static_cast<uint32_t>(lane) * 4u;
    int total = 0;
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        int w[32];
        int a;
        if (FMT == kBitcos) {
            const uint4 bm = reinterpret_cast<const uint4 *>(stage)[lane];
            const int c = __popc(bm.x) + __popc(bm.y) + __popc(bm.z) + __popc(bm.w);
            int incl = c;
#pragma unroll
            for (int dd = 1; dd < 32; dd <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, incl, dd);
                if (lane >= dd) incl += v;
            }
            const uint32_t cursor = static_cast<uint32_t>(incl - c) + static_cast<uint32_t>(it & 1);
            const uint32_t *sp = reinterpret_cast<const uint32_t *>(stage + 1024) + (cursor >> 5);
            bitcos_decode_row(bm, sp, cursor & 31u, lut, lane4, w);
            asm volatile("" ::: "memory");
            a = contract<kBitcos>(w, reinterpret_cast<const int4 *>(xs), lane);
        } else if (FMT == kTrit5) {
            const uint32_t *src = reinterpret_cast<const uint32_t *>(stage) + lane;
            uint32_t wd[7];
#pragma unroll
            for (int i = 0; i < 7; ++i) wd[i] = src[i * kRows];
            trit5_decode_row(wd, it & 1, lut, static_cast<uint32_t>(lane) * 8u, w);
            a = contract<kTrit5>(w, reinterpret_cast<const int4 *>(xs), lane);
        } else {
            const uint4 *src = reinterpret_cast<const uint4 *>(stage) + lane + (it & 1);   // keep the loads in the loop
            bit2_decode_row(src[0], src[kRows], w);
            a = contract<kBit2>(w, reinterpret_cast<const int4 *>(xs), lane);
        }
        const float sc = bf16_to_float(reinterpret_cast<const uint16_t *>(stage + 1024 + 640)[lane]);
        total += __float_as_int(sc * static_cast<float>(a));
    }
    const long long t1 = clock64();
    __shared__ unsigned long long s_max;
    if (threadIdx.x == 0) s_max = 0;
    __syncthreads();
    if (lane == 0) atomicMax(&s_max, static_cast<unsigned long long>(t1 - t0));
    __syncthreads();
    if (threadIdx.x == 0) cycles[blockIdx.x] = s_max;
    if (total == 0x12345678) *sink = total;
}

// ---------------------------------------------------------------------------------------------
// Give-up path of the bounded waits, exercised without a fault: one warp arms an mbarrier for bytes
// that no copy ever delivers and waits for it with the kernels' own polling loop and a short limit.
// The wait runs out, the warp sets the workspace's status word exactly as the products do, and the
// kernel returns normally; the context stays usable.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32, 1) wait_probe_kernel(unsigned int *status, unsigned long long limit_ns, unsigned long long *waited_ns) {
    __shared__ __align__(8) unsigned long long bar_word;
    const uint32_t bar = smem_addr(&bar_word);
    const int lane = threadIdx.x & 31;
    if (lane == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar, 64);                  // 64 bytes are announced; nothing is ever copied
    }
    __syncwarp();
    const uint64_t t0 = global_timer_ns();
    const bool ok = mbar_wait_limited(bar, 0, limit_ns);
    const uint64_t t1 = global_timer_ns();
    if (!ok && lane == 0) {
        *status = 1u;
        if (waited_ns) *waited_ns = t1 - t0;
    }
}

// ---------------------------------------------------------------------------------------------
// Routing pairs grouped by expert on the device (a stable counting sort in one thread block), so
// that a decode loop whose router runs on the GPU never has to bring the pairs to the host: count
// the pairs of every expert, give every expert that has any a group (experts ascending), place
// every pair behind the pairs of the same expert that precede it in the input.  A pair whose expert
// id is out of range is dropped (it gets no group and order -1 is never written for it; its output
// row is simply not produced).
// ---------------------------------------------------------------------------------------------
constexpr int kGroupPairsThreads = 256;
__global__ void __launch_bounds__(kGroupPairsThreads) group_pairs_kernel(const int32_t *__restrict__ pair_expert,
                                                                         const int32_t *__restrict__ pair_xrow, int n_pairs, int n_experts,
                                                                         int32_t *group_expert, int32_t *group_begin,
                                                                         int32_t *pair_xrow_sorted, int32_t *order, int32_t *n_groups) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __shared__ int count[BITCOS_GROUP_EXPERTS_MAX];      // pairs per expert, then the expert's first position
    for (int e = threadIdx.x; e < n_experts; e += kGroupPairsThreads) count[e] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n_pairs; i += kGroupPairsThreads) {
        const int e = pair_expert[i];
        if (e >= 0 && e < n_experts) atomicAdd(&count[e], 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int pos = 0, g = 0;
        for (int e = 0; e < n_experts; ++e) {
            const int c = count[e];
            count[e] = pos;
            if (c) {
                group_expert[g] = e;
                group_begin[g] = pos;
                ++g;
            }
            pos += c;
        }
        group_begin[g] = pos;
        *n_groups = g;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n_pairs; i += kGroupPairsThreads) {
        const int e = pair_expert[i];
        if (e < 0 || e >= n_experts) continue;
        int rank = 0;
        for (int j = 0; j < i; ++j) rank += (pair_expert[j] == e) ? 1 : 0;      // stable: input order inside a group
        const int at = count[e] + rank;
        pair_xrow_sorted[at] = pair_xrow[i];
        order[at] = i;
    }
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

// Number of multiprocessors of the current device.  The opt-in to large dynamic shared memory is
// done on the first call for a given kernel instantiation and device and remembered (so that
// first call must not happen during stream capture; later calls only read the cache).
template <auto kernel>
int prepare_kernel(int *sms_out, int *smem_budget_out) {
    constexpr int kMaxDev = 32;
    static int cache[kMaxDev][2];      // [0] multiprocessor count (0 = not prepared yet), [1] dynamic smem budget
    int dev = 0;
    int rc = check_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    if (dev < kMaxDev && cache[dev][0] > 0) {
        *sms_out = cache[dev][0];
        *smem_budget_out = cache[dev][1];
        return BITCOS_OK;
    }
    int sms = 0, max_smem = 0;
    rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (rc) return rc;
    rc = check_cuda(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    if (rc) return rc;
    const int budget = max_smem - 1024;
    rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, budget));
    if (rc) return rc;
    if (dev < kMaxDev) {
        cache[dev][1] = budget;
        cache[dev][0] = sms;
    }
    *sms_out = sms;
    *smem_budget_out = budget;
    return BITCOS_OK;
}

// Ring depth: as many stages as fit next to the tables, activations and partial sums (the loaded
// DRAM latency of this part needs on the order of 100 KB in flight per multiprocessor).
inline int choose_stages(int fmt, const Plan &pl, int G, int nb, int64_t K, int smem_budget) {
    Plan p = pl;
    for (int st = kMaxStages; st > 2; --st) {
        p.stages = st;
        if (static_cast<int>(smem_layout(fmt, p, G, nb, K).total) <= smem_budget) return st;
    }
    return 2;
}

// How the items are handed to thread blocks, and how many blocks to launch (persistent: at most
// one per multiprocessor).  Cost model in units of one item's time: round robin over row-block
// chunks costs ceil(chunks / blocks) * CS items per block and never shares a row block; a
// contiguous balanced split costs ceil(items / blocks) items plus, when rows are split into
// column blocks, the cross-block hand-shake at the end (worth about 2.5 items).
// BITCOS_WALK=cyclic|contiguous overrides the choice (for A/B runs).
// A launch with no more items than multiprocessors would give every block one item and spread
// over most of the machine.  Under programmatic dependent launch the NEXT kernel's blocks start
// early (table, first weights, first decode, all before its dependency is resolved) only on
// multiprocessors this launch leaves free, and blocks that start late pay their whole start-up
// after the dependency; so such a launch takes a little under half of the multiprocessors and two
// items per block instead (measured on the decoder-layer sequence: 16.5 -> 16.05 us per pass; the
// step is sharp: the blocks of two consecutive small launches must fit side by side).
inline int small_launch_cap(int64_t items, int sms) {
    if (items > sms) return sms;
    const int cap = sms * 46 / 100;
    static const char *env = std::getenv("BITCOS_SMALL_FULL");
    if ((!env || env[0] != '0') && items <= sms - cap) return static_cast<int>(items);
    return cap < 1 ? 1 : cap;
}

inline void choose_walk(Plan &pl, int sms, int *grid) {
    static const char *force = std::getenv("BITCOS_WALK");
    const int64_t chunks = pl.items / pl.CS;
    const int64_t g_cyc = chunks < sms ? chunks : sms, g_con = pl.items < sms ? pl.items : sms;
    const double cost_cyc = static_cast<double>((chunks + g_cyc - 1) / g_cyc) * pl.CS;
    const double cost_con = static_cast<double>((pl.items + g_con - 1) / g_con) + (pl.CS > 1 ? 2.5 : 0.0);
    int cyclic = cost_cyc <= cost_con ? 1 : 0;
    if (force && force[0] == 'c' && force[1] == 'y') cyclic = 1;
    if (force && force[0] == 'c' && force[1] == 'o') cyclic = 0;
    pl.cyclic = cyclic;
    *grid = static_cast<int>(cyclic ? g_cyc : g_con);
    pl.wq = cyclic ? 1 : static_cast<int>(pl.items / *grid);
    pl.wrem = cyclic ? 0 : static_cast<int>(pl.items - static_cast<int64_t>(pl.wq) * *grid);
}

// Launches with programmatic stream serialization, so that this kernel's prologue (barrier
// set-up, table and first weight copies) may overlap the tail of the previous kernel in the
// stream.  BITCOS_PDL=0 turns it off (for A/B runs).
template <typename... KArgs, typename... Args>
int launch_pdl(void (*kernel)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t stream, Args... args) {
    static const char *env = std::getenv("BITCOS_PDL");
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(static_cast<unsigned>(threads));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (env && env[0] == '0') ? 0 : 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, kernel, args...));
}

// While a launch sequence is being recorded for replay (bitcos_gemv_phases_host), every value a
// plan takes from a host copy of tile_off is noted here, so that a replay can make sure that the
// values it was built from are still there.
thread_local std::vector<std::pair<const uint32_t *, uint32_t>> *g_offset_log = nullptr;
inline uint32_t host_offset(const uint32_t *off_host, int64_t i) {
    const uint32_t v = off_host[i];
    if (g_offset_log) g_offset_log->emplace_back(off_host + i, v);
    return v;
}

// Fills fo.lo / fo.hi [base .. base + grid) from a host copy of tile_off: the sign-vector range of
// the first item of each of the `grid` thread blocks that share the problem.
void fill_first_off(FirstOff &fo, int base, const uint32_t *off_host, const Problem &pr, const Plan &pl, int grid) {
    if (base + grid > kMaxGrid) {
        fo.valid = 0;
        fo.walks = 0;
        return;
    }
    for (int b = 0; b < grid; ++b) {
        const Walk wk = make_walk(pl, b, grid);
        fo.first[base + b] = wk.first;
        fo.count[base + b] = wk.count;
    }
    if (!off_host) fo.valid = 0;
    if (!fo.valid) return;
    for (int b = 0; b < grid; ++b) {
        const Walk wk = make_walk(pl, b, grid);
        fo.lo[base + b] = fo.hi[base + b] = 0;
        if (wk.count <= 0) continue;
        ItemIter it;
        it.init(pl, wk.first);
        const ItemRange r = item_range(pr, pl, it.c, it.cs);
        fo.lo[base + b] = host_offset(off_host, r.t0);
        fo.hi[base + b] = host_offset(off_host, r.t0 + r.nt);
    }
}

// Large matrices, one or two tokens: items of twice the size, two tiles per decoder warp, so that
// what a decoder warp does per item (barrier waits, descriptor, stage advance, hand-off of the
// partial sums: about 50 of its 364 instructions per tile) is paid once per two tiles.  Only when
// every block still gets several items: from eight of the one-tile items per multiprocessor on.  (Between
// three and eight the gain depends on the shape and the format: 8192x5120 -3 % at one token but +6 % at
// two, 4096x12288 +3 %, 2-bit +3 %; so those keep one tile per warp.)
inline bool wants_two_tiles(const Plan &pl, int nb_template, int sms) {
    return nb_template < kMmaMinBatch && pl.items >= 8 * static_cast<int64_t>(sms);
}

template <int FMT, int NB, bool XG = false, bool XQ = false, bool BL = false>
int launch(const Problem &pr, const Plan &pl_in, cudaStream_t stream, const uint32_t *off_host = nullptr) {
    // the one- and two-token instantiations keep the activations in shared memory (nb_bucket sees to it)
    if (NB < kMmaMinBatch && static_cast<int64_t>(NB) * pr.K > kXResidentBytes) return BITCOS_ERR_SHAPE;
    int sms = 0, budget = 0;
    int rc = prepare_kernel<gemv_kernel<FMT, NB, 1, XG, XQ, BL>>(&sms, &budget);
    if (rc) return rc;
    const bool two = wants_two_tiles(pl_in, NB, sms);
    if constexpr (NB < kMmaMinBatch) {
        if (two) {
            rc = prepare_kernel<gemv_kernel<FMT, NB, 2, XG, XQ>>(&sms, &budget);
            if (rc) return rc;
        }
    }
    const Plan pl = two ? make_plan(pr.M, pr.K, decoder_warps(pr.nb), 2) : pl_in;
    int grid = 1;
    Plan plw = pl;
    choose_walk(plw, small_launch_cap(pl.items, sms), &grid);
    plw.stages = choose_stages(FMT, pl, pr.G, NB, pr.K, budget);
    const SmemLayout L = smem_layout(FMT, plw, pr.G, NB, pr.K);
    FirstOff fo;
    fo.valid = (FMT == kBitcos && off_host) ? 1 : 0;
    fo.walks = 1;
    fill_first_off(fo, 0, off_host, pr, plw, grid);
    if constexpr (NB < kMmaMinBatch) {
        if (two) return launch_pdl(gemv_kernel<FMT, NB, 2, XG, XQ>, dim3(grid), (pl.NW + 2) * 32, L.total, stream, pr, plw, fo);
    }
    return launch_pdl(gemv_kernel<FMT, NB, 1, XG, XQ, BL>, dim3(grid), (pl.NW + 2) * 32, L.total, stream, pr, plw, fo);
}

// The copies of a thread block's first item, as issue_item<kBitcos> would issue them into stage 0
// (first = the block's first item, o_lo / o_hi = entry offsets of its first tile and of the tile
// after its last).
inline void fill_first_copies(FirstCopies &c, const Problem &pr, const Plan &pl, const SmemLayout &L, int first, uint32_t o_lo,
                              uint32_t o_hi) {
    ItemIter it;
    it.init(pl, first);
    const ItemRange r = item_range(pr, pl, it.c, it.cs);
    const uint32_t b_lo = (o_lo >> 7) << 4, b_hi = ((o_hi + 127u) >> 7) << 4;
    const uint32_t o_first = static_cast<uint32_t>(r.t0 & 3);
    c.src[0] = pr.tile_off + (r.t0 - o_first);
    c.bytes[0] = ((o_first + static_cast<uint32_t>(r.nt) + 1u + 3u) & ~3u) * 4u;
    c.src[1] = reinterpret_cast<const uint8_t *>(pr.payload) + r.t0 * 512;
    c.bytes[1] = static_cast<uint32_t>(r.nt) * 512u;
    c.src[2] = reinterpret_cast<const uint8_t *>(pr.signs) + b_lo;
    c.bytes[2] = b_hi - b_lo;
    c.src[3] = reinterpret_cast<const uint8_t *>(pr.scales) + r.t0 * 64;
    c.bytes[3] = static_cast<uint32_t>(r.nt) * 64u;
    c.dst[1] = L.stage;
    c.dst[2] = c.dst[1] + L.payload_cap;
    c.dst[3] = c.dst[2] + L.sign_cap;
    c.dst[0] = c.dst[3] + L.scale_cap;
    c.desc[0] = static_cast<uint32_t>(r.nt) | (o_first << 8);
    c.desc[1] = static_cast<uint32_t>(r.g0);
    c.desc[2] = static_cast<uint32_t>(r.rb0);
    c.desc[3] = b_lo * 8u;
    c.desc_off = L.bar + 384u;
    c.bar = L.bar;
}

// Grids of a multi launch: whether it runs two tiles per decoder warp, and each job's plan, walk
// and number of thread blocks (the multiprocessors shared between the jobs in proportion to their
// item counts).  Returns the total number of blocks.
inline int plan_multi(MultiArgs &ma, int nb_template, int sms, bool *two_out, int *grids) {
    int64_t total_items = 0;
    for (int j = 0; j < ma.n; ++j) total_items += ma.pl[j].items;
    // enough items altogether: every problem with two tiles per decoder warp
    Plan all{};
    all.items = total_items;
    const bool two = wants_two_tiles(all, nb_template, sms);
    if (two) {
        total_items = 0;
        for (int j = 0; j < ma.n; ++j) {
            ma.pl[j] = make_plan(ma.pr[j].M, ma.pr[j].K, decoder_warps(nb_template), 2);
            total_items += ma.pl[j].items;
        }
    }
    *two_out = two;
    sms = small_launch_cap(total_items, sms);
    int next = 0;
    for (int j = 0; j < ma.n; ++j) {
        int64_t cap = ma.pl[j].items;
        if (total_items > sms) {
            cap = ma.pl[j].items * sms / total_items;
            if (cap < 1) cap = 1;
        }
        choose_walk(ma.pl[j], static_cast<int>(cap), &grids[j]);
        next += grids[j];
    }
    return next;
}

// A launch whose first `early` thread blocks (of `grid`) find a free multiprocessor at once while
// the others have to wait for the blocks of the kernel before it to leave: by the time a late
// block has gone through its start-up, an early one -- which did all of that, first decode
// included, while it waited for its dependency -- is about kLateLagItems items ahead.  So early
// blocks take that many items more.  Only for jobs whose items are whole row blocks (nothing is
// shared between thread blocks, so the split has no influence on any sum).  counts[r] = items of
// the job's block number r; its early blocks come first.
constexpr int kLateLagItems = 2;
inline void skewed_counts(int64_t items, int n_early, int n_late, int *counts) {
    const int n = n_early + n_late;
    int64_t a = (items + static_cast<int64_t>(n_late) * kLateLagItems + n - 1) / n;
    if (a < 1) a = 1;
    int64_t sum = 0;
    for (int r = 0; r < n; ++r) {
        int64_t c = r < n_early ? a : a - kLateLagItems;
        if (c < 0) c = 0;
        counts[r] = static_cast<int>(c);
        sum += c;
    }
    // too many by rounding: taken back one at a time, from the last block backwards
    for (int r = n - 1; sum > items; r = (r == 0 ? n - 1 : r - 1))
        if (counts[r] > 0) {
            --counts[r];
            --sum;
        }
    for (int r = 0; sum < items; r = (r + 1) % n) {       // (too few: only when a - lag was cut at zero)
        ++counts[r];
        ++sum;
    }
}

// Whether a launch's blocks are split into early and late ones, and if so the split: block b works on
// job job_of[b] as that job's block number rank[b] and takes count[b] items from item first[b] of the job
// (early blocks are dealt to the jobs in proportion to their grids, job after job, then the late ones;
// inside a job, contiguous ranges of its items, early blocks first).
inline bool skewed_assignment(MultiArgs &ma, const int *grids, int total, bool two, int sms, int busy_sms, int *first, int *count) {
    // late starters: only when part of the grid starts early and part late, and every job's items are whole rows
    const int early = sms - busy_sms;
    bool skew = busy_sms > 0 && early > 0 && early < total && total <= kMaxGrid && !two;
    for (int j = 0; j < ma.n; ++j) skew = skew && ma.pl[j].CS == 1 && ma.pl[j].items >= grids[j];
    if (!skew) return false;
    int ne[kMaxJobs], given = 0;
    for (int j = 0; j < ma.n; ++j) {
        ne[j] = static_cast<int>(static_cast<int64_t>(early) * grids[j] / total);
        given += ne[j];
    }
    for (int j = 0; given < early; j = (j + 1) % ma.n)
        if (ne[j] < grids[j]) {
            ++ne[j];
            ++given;
        }
    int b = 0;
    for (int pass = 0; pass < 2; ++pass)
        for (int j = 0; j < ma.n; ++j) {
            const int r0 = pass ? ne[j] : 0, r1 = pass ? grids[j] : ne[j];
            for (int r = r0; r < r1; ++r, ++b) {
                ma.job_of[b] = static_cast<uint8_t>(j);
                ma.rank[b] = static_cast<uint8_t>(r);
            }
        }
    static thread_local int counts[kMaxJobs][kMaxGrid], firsts[kMaxJobs][kMaxGrid];
    for (int j = 0; j < ma.n; ++j) {
        ma.nblk[j] = grids[j];
        ma.pl[j].cyclic = 0;
        skewed_counts(ma.pl[j].items, ne[j], grids[j] - ne[j], counts[j]);
        int f = 0;
        for (int r = 0; r < grids[j]; ++r) {
            firsts[j][r] = f;
            f += counts[j][r];
        }
    }
    for (b = 0; b < total; ++b) {
        first[b] = firsts[ma.job_of[b]][ma.rank[b]];
        count[b] = counts[ma.job_of[b]][ma.rank[b]];
    }
    ma.first_block[ma.n] = total;
    ma.mapped = 1;
    return true;
}

// busy_sms: multiprocessors the caller expects the kernel before this one in the stream to hold on
// to when this launch's blocks are scheduled (0: unknown or none).
template <int NB, bool XQ = false, bool XG = false>
int launch_multi(MultiArgs &ma, cudaStream_t stream, const uint32_t *const *off_host, int busy_sms = 0) {
    for (int j = 0; j < ma.n; ++j)
        if (NB < kMmaMinBatch && static_cast<int64_t>(NB) * ma.pr[j].K > kXResidentBytes) return BITCOS_ERR_SHAPE;
    int sms = 0, budget = 0;
    int rc = prepare_kernel<gemv_multi_kernel<NB, 1, XQ, XG>>(&sms, &budget);
    if (rc) return rc;
    if constexpr (!XQ && !XG && NB <= 2) {
        // (the variant that is only launched while a graph is being recorded is set up here, on whichever call comes first)
        rc = prepare_kernel<gemv_multi_kernel<NB, 1, false, false, FirstCopiesTable>>(&sms, &budget);
        if (rc) return rc;
    }
    bool two = false;
    int grids[kMaxJobs];
    const int total = plan_multi(ma, NB, sms, &two, grids);
    if constexpr (NB < kMmaMinBatch) {
        if (two) {
            rc = prepare_kernel<gemv_multi_kernel<NB, 2, XQ, XG>>(&sms, &budget);
            if (rc) return rc;
        }
    }
    int nw = 0;
    uint32_t smem = 0;
    FirstOff fo;
    fo.valid = 1;
    fo.walks = 1;
    for (int j = 0; j < ma.n; ++j) fo.valid = (fo.valid && off_host[j]) ? 1 : 0;
    for (int j = 0; j < ma.n; ++j) {
        ma.pl[j].stages = choose_stages(kBitcos, ma.pl[j], ma.pr[j].G, NB, ma.pr[j].K, budget);
        const SmemLayout L = smem_layout(kBitcos, ma.pl[j], ma.pr[j].G, NB, ma.pr[j].K);
        if (L.total > smem) smem = L.total;
        if (ma.pl[j].NW > nw) nw = ma.pl[j].NW;
    }
    if (!skewed_assignment(ma, grids, total, two, sms, busy_sms, fo.first, fo.count)) {
        int next = 0;
        for (int j = 0; j < ma.n; ++j) {
            ma.first_block[j] = next;
            fill_first_off(fo, next, fo.valid ? off_host[j] : nullptr, ma.pr[j], ma.pl[j], grids[j]);
            next += grids[j];
        }
        ma.first_block[ma.n] = next;
        ma.mapped = 0;
    } else {
        for (int b = 0; b < total; ++b) {
            const int j = ma.job_of[b];
            fo.lo[b] = fo.hi[b] = 0;
            if (fo.valid && fo.count[b] > 0) {
                ItemIter it;
                it.init(ma.pl[j], fo.first[b]);
                const ItemRange ir = item_range(ma.pr[j], ma.pl[j], it.c, it.cs);
                fo.lo[b] = host_offset(off_host[j], ir.t0);
                fo.hi[b] = host_offset(off_host[j], ir.t0 + ir.nt);
            }
        }
    }
    // every block's first copies, when the entry offsets are known on the host
    static thread_local FirstCopiesTable fc;
    static const char *fc_env = std::getenv("BITCOS_FIRST_COPIES");      // 0: never, 1: also on plain stream launches (A/B runs)
    fc.valid = 0;
    bool recording = false;
    {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cs) == cudaSuccess) recording = cs == cudaStreamCaptureStatusActive;
        else cudaGetLastError();
    }
    const bool with_table = !XQ && !XG && NB <= 2 && !two && (recording || (fc_env && fc_env[0] == '1')) && !(fc_env && fc_env[0] == '0');
    if (with_table && fo.valid && fo.walks && total <= kMaxGrid) {
        fc.valid = 1;
        int jb = 0;
        for (int b = 0; b < total; ++b) {
            int j;
            if (ma.mapped) {
                j = ma.job_of[b];
            } else {
                while (jb + 1 < ma.n && b >= ma.first_block[jb + 1]) ++jb;
                j = jb;
            }
            fc.c[b] = FirstCopies{};
            if (fo.count[b] <= 0) continue;
            const SmemLayout L = smem_layout(kBitcos, ma.pl[j], ma.pr[j].G, NB, ma.pr[j].K);
            fill_first_copies(fc.c[b], ma.pr[j], ma.pl[j], L, fo.first[b], fo.lo[b], fo.hi[b]);
        }
    }
    if constexpr (!XQ && !XG && NB <= 2) {
        if (fc.valid) {
            return launch_pdl(gemv_multi_kernel<NB, 1, false, false, FirstCopiesTable>, dim3(total), (nw + 2) * 32, smem, stream, ma, fo, fc);
        }
    }
    const NoFirstCopies none{0};
    if constexpr (NB < kMmaMinBatch) {
        if (two) return launch_pdl(gemv_multi_kernel<NB, 2, XQ, XG>, dim3(total), (nw + 2) * 32, smem, stream, ma, fo, none);
    }
    return launch_pdl(gemv_multi_kernel<NB, 1, XQ, XG>, dim3(total), (nw + 2) * 32, smem, stream, ma, fo, none);
}

// Which instantiation serves a batch: 1, 2, 4, 8 or 16 tokens.  The one- and two-token paths read
// the activations from shared memory; when those do not fit there (K beyond 48 K / 24 K), the
// tensor-core path, which takes its activation fragments from global memory, is the faster one.
inline int nb_bucket(int batch, int64_t K) {
    if (batch <= 2 && static_cast<int64_t>(batch) * K > kXResidentBytes) return 4;
    return batch <= 1 ? 1 : batch <= 2 ? 2 : batch <= 4 ? 4 : batch <= 8 ? 8 : 16;
}

template <int FMT, bool XG = false>
int launch_nb(const Problem &pr, const Plan &pl, cudaStream_t stream, const uint32_t *off_host) {
    const int nbk = nb_bucket(pr.nb, pr.K);
    if (nbk == 1) return launch<FMT, 1, XG>(pr, pl, stream, off_host);
    if (nbk == 2) return launch<FMT, 2, XG>(pr, pl, stream, off_host);
    if (pr.nb <= 4) return launch<FMT, 4, XG>(pr, pl, stream, off_host);
    if (pr.nb <= 8) return launch<FMT, 8, XG>(pr, pl, stream, off_host);
    return launch<FMT, 16, XG>(pr, pl, stream, off_host);
}

template <int FMT, int NB>
int launch_grouped(const Problem &pr, const Plan &pl, const GroupedArgs &ga, int n_groups, cudaStream_t stream) {
    if (NB < kMmaMinBatch && static_cast<int64_t>(NB) * pr.K > kXResidentBytes) return BITCOS_ERR_SHAPE;
    int sms = 0, budget = 0;
    int rc = prepare_kernel<gemv_grouped_kernel<FMT, NB>>(&sms, &budget);
    if (rc) return rc;
    Plan plw = pl;
    plw.stages = choose_stages(FMT, pl, pr.G, NB, pr.K, budget);
    const SmemLayout L = smem_layout(FMT, plw, pr.G, NB, pr.K);
    GroupedArgs gaw = ga;
    gaw.n_groups = n_groups;
    if (pl.CS == 1) {
        // rows in one piece: one balanced list of all groups' items; one or two tokens per group:
        // their activation rows travel with every stage
        const int64_t total = pl.items * n_groups;
        gaw.flat = 1;
        plw.cyclic = 0;
        plw.x_in_stage = NB < kMmaMinBatch ? 1 : 0;
        plw.stages = choose_stages(FMT, plw, pr.G, NB, pr.K, budget);
        const SmemLayout Lf = smem_layout(FMT, plw, pr.G, NB, pr.K);
        return launch_pdl(gemv_grouped_kernel<FMT, NB>, dim3(static_cast<unsigned>(total < sms ? total : sms)), (pl.NW + 2) * 32,
                          Lf.total, stream, pr, plw, gaw);
    }
    // the machine is shared by all groups: spread its multiprocessors over them
    int per_group = (sms + n_groups - 1) / n_groups;
    if (per_group < 1) per_group = 1;
    int gx = 1;
    choose_walk(plw, per_group, &gx);
    gaw.flat = 0;
    return launch_pdl(gemv_grouped_kernel<FMT, NB>, dim3(gx, n_groups), (pl.NW + 2) * 32, L.total, stream, pr, plw, gaw);
}

// Validates the arguments every product shares; fills nothing.
int check_common(int fmt, const uint32_t *payload, const uint32_t *signs, const uint32_t *tile_off,
                 const uint16_t *scales, int64_t M, int64_t K, const int8_t *x, const float *x_scale, int batch,
                 const float *y, const int32_t *acc_debug, const void *workspace, size_t workspace_bytes) {
    if (!payload || !scales || !x || !x_scale || !y || !workspace) return BITCOS_ERR_NULL;
    if (fmt == kBitcos && (!signs || !tile_off)) return BITCOS_ERR_NULL;
    if (M < 1 || K < kGroup || K % kGroup != 0 || batch < 1 || batch > BITCOS_MAX_BATCH) return BITCOS_ERR_SHAPE;
    if (K / kGroup > 0x7FFFFF || make_plan(M, K, kWarps16).items > 0x3FFFFFFF) return BITCOS_ERR_SHAPE;
    if (!aligned16(payload) || !aligned16(scales) || !aligned16(x) || !aligned16(y) || !aligned16(workspace) ||
        (signs && !aligned16(signs)) || (tile_off && !aligned16(tile_off)) || (acc_debug && !aligned16(acc_debug)))
        return BITCOS_ERR_ALIGN;
    if (workspace_bytes < workspace_bytes_for(M, K)) return BITCOS_ERR_CAPACITY;
    return BITCOS_OK;
}

void fill_problem(Problem &pr, const uint32_t *payload, const uint32_t *signs, const uint32_t *tile_off,
                  const uint16_t *scales, int64_t M, int64_t K, const int8_t *x, const float *x_scale, int batch,
                  float *y, int32_t *acc_debug, void *workspace) {
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
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    pr.status = reinterpret_cast<unsigned int *>(ws);
    pr.counters = reinterpret_cast<unsigned int *>(ws + kHeaderBytes);
    pr.partial = reinterpret_cast<float *>(ws + kHeaderBytes + counters_bytes(pr.RB));
}

int gemv_common(int fmt, const uint32_t *payload, const uint32_t *signs, const uint32_t *tile_off,
                const uint16_t *scales, int64_t M, int64_t K, const int8_t *x, const float *x_scale, int batch,
                float *y, int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream,
                const uint32_t *off_host = nullptr, bool group_scales = false) {
    const int bad = check_common(fmt, payload, signs, tile_off, scales, M, K, x, x_scale, batch, y, acc_debug, workspace,
                                 workspace_bytes);
    if (bad) return bad;
    const Plan pl = make_plan(M, K, decoder_warps(batch));
    Problem pr{};
    fill_problem(pr, payload, signs, tile_off, scales, M, K, x, x_scale, batch, y, acc_debug, workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (group_scales) return fmt == kBitcos ? launch_nb<kBitcos, true>(pr, pl, stream, off_host) : BITCOS_ERR_SHAPE;
    if (fmt == kBitcos) return launch_nb<kBitcos>(pr, pl, stream, off_host);
    if (fmt == kTrit5) return launch_nb<kTrit5>(pr, pl, stream, nullptr);
    return launch_nb<kBit2>(pr, pl, stream, nullptr);
}


// ------------------------------------------------------------------ activation quantiser
// bf16 activations -> int8 codes and float scales, one scale per group of 128 or per token:
//   a = max(max |x| over the group, 2^-100),  scale = a / 127,  code = rint(x * (127 / a))
// with IEEE float32 quotient and product and ties to even (the explicit intrinsics keep the
// compiler from contracting or approximating them, so the codes do not depend on build flags).
// One warp per group of 128: a lane holds four consecutive values.
__global__ void __launch_bounds__(256) quantize_groups_kernel(const uint16_t *__restrict__ x, int8_t *__restrict__ q,
                                                              float *__restrict__ scale, int64_t n_groups) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const int64_t warps = static_cast<int64_t>(gridDim.x) * (blockDim.x >> 5);
    for (int64_t grp = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); grp < n_groups; grp += warps) {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(x + grp * kGroup) + lane);
        float a = fmaxf(fmaxf(fabsf(bf16_lo(v.x)), fabsf(bf16_hi(v.x))), fmaxf(fabsf(bf16_lo(v.y)), fabsf(bf16_hi(v.y))));
#pragma unroll
        for (int d = 16; d; d >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, d));
        a = fmaxf(a, kAmaxFloor);
        const float inv = __fdiv_rn(127.0f, a);
        reinterpret_cast<uint32_t *>(q + grp * kGroup)[lane] = quant_pair(v.x, inv) | (quant_pair(v.y, inv) << 16);
        if (lane == 0) scale[grp] = __fdiv_rn(a, 127.0f);
    }
}

// One thread block per token: largest magnitude of the row, then the codes (the row is read
// twice, the second time from cache).
constexpr int kQuantThreads = 512;
__global__ void __launch_bounds__(kQuantThreads) quantize_tokens_kernel(const uint16_t *__restrict__ x, int8_t *__restrict__ q,
                                                                        float *__restrict__ scale, int64_t K) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __shared__ float warp_max[kQuantThreads / 32];
    const int64_t row = blockIdx.x;
    const uint4 *src = reinterpret_cast<const uint4 *>(x + row * K);      // eight values per load
    const int64_t n = K / 8;
    float a = 0.f;
    for (int64_t i = threadIdx.x; i < n; i += kQuantThreads) {
        const uint4 v = __ldg(src + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) a = fmaxf(a, fmaxf(fabsf(bf16_lo(w[j])), fabsf(bf16_hi(w[j]))));
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, d));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = a;
    __syncthreads();
    a = warp_max[0];
#pragma unroll
    for (int j = 1; j < kQuantThreads / 32; ++j) a = fmaxf(a, warp_max[j]);
    a = fmaxf(a, kAmaxFloor);
    const float inv = __fdiv_rn(127.0f, a);
    uint2 *dst = reinterpret_cast<uint2 *>(q + row * K);
    for (int64_t i = threadIdx.x; i < n; i += kQuantThreads) {
        const uint4 v = __ldg(src + i);
        dst[i] = make_uint2(quant_pair(v.x, inv) | (quant_pair(v.y, inv) << 16),
                            quant_pair(v.z, inv) | (quant_pair(v.w, inv) << 16));
    }
    if (threadIdx.x == 0) scale[row] = __fdiv_rn(a, 127.0f);
}

}  // namespace

namespace bitcos_detail {
// for the library's other translation units: the error bitcos_last_cuda_error reports
void record_cuda_error(int e) { g_last_cuda_error = e; }
}  // namespace bitcos_detail

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

int bitcos_workspace_status(const void *workspace, void *cuda_stream, int *status) {
    if (!workspace || !status) return BITCOS_ERR_NULL;
    unsigned int v = 0;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = check_cuda(cudaMemcpyAsync(&v, workspace, sizeof v, cudaMemcpyDeviceToHost, stream));
    if (rc) return rc;
    rc = check_cuda(cudaStreamSynchronize(stream));
    if (rc) return rc;
    *status = static_cast<int>(v);
    return BITCOS_OK;
}

int bitcos_decode_probe(int format, int warps_per_block, int iters, int blocks, uint64_t *cycles, void *cuda_stream) {
    if (!cycles) return BITCOS_ERR_NULL;
    if (format < 0 || format > 2 || warps_per_block < 1 || warps_per_block > kMaxWarps + 2 || iters < 1 ||
        iters > (1 << 20) || blocks < 1 || blocks > 4096)
        return BITCOS_ERR_SHAPE;
    const size_t smem = (format == kBit2 ? 0 : kLutBytes) + static_cast<size_t>(warps_per_block) * 1792 + 256;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int *sink = reinterpret_cast<int *>(cycles);      // never written in practice
    unsigned long long *out = reinterpret_cast<unsigned long long *>(cycles);
    int rc;
    if (format == kBitcos) {
        rc = check_cuda(cudaFuncSetAttribute(decode_probe_kernel<kBitcos>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        if (rc) return rc;
        decode_probe_kernel<kBitcos><<<blocks, warps_per_block * 32, smem, stream>>>(iters, out, sink);
    } else if (format == kTrit5) {
        rc = check_cuda(cudaFuncSetAttribute(decode_probe_kernel<kTrit5>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        if (rc) return rc;
        decode_probe_kernel<kTrit5><<<blocks, warps_per_block * 32, smem, stream>>>(iters, out, sink);
    } else {
        rc = check_cuda(cudaFuncSetAttribute(decode_probe_kernel<kBit2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        if (rc) return rc;
        decode_probe_kernel<kBit2><<<blocks, warps_per_block * 32, smem, stream>>>(iters, out, sink);
    }
    return check_cuda(cudaGetLastError());
}

int bitcos_gemv(const bitcos_weights *W, const int8_t *x, const float *x_scale, int batch, float *y,
                int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!W) return BITCOS_ERR_NULL;
    return gemv_common(kBitcos, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x, x_scale, batch, y,
                       acc_debug, workspace, workspace_bytes, cuda_stream, W->tile_off_host);
}

// ---------------------------------------------------------------------------------------------
// bitcos_gemv_static: the same product with the scratch memory taken from a fixed array that is
// part of the library image, for callers that must not (or cannot) allocate device memory.
// ---------------------------------------------------------------------------------------------
}  // extern "C"

namespace {
// Scratch of the no-allocation entry point.  Every device that loads the library carries these
// bytes until the process exits.  In host code the name below is only a handle for
// cudaGetSymbolAddress; it is not a device address and is never passed to a kernel.
static __device__ __align__(256) unsigned char g_static_workspace[BITCOS_STATIC_WORKSPACE_BYTES];

// Device address of g_static_workspace on the current device, looked up once per device.  (The cache is
// written without a lock: two threads that race on a device's first call both store the same address.)
int static_workspace_ptr(void **out) {
    constexpr int kMaxDev = 32;
    static void *cache[kMaxDev];
    int dev = 0;
    int rc = check_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    if (dev < kMaxDev && cache[dev]) {
        *out = cache[dev];
        return BITCOS_OK;
    }
    void *ptr = nullptr;
    rc = check_cuda(cudaGetSymbolAddress(&ptr, g_static_workspace));
    if (rc) return rc;
    if (!ptr) return BITCOS_ERR_CUDA;
    if (dev < kMaxDev) cache[dev] = ptr;
    *out = ptr;
    return BITCOS_OK;
}
}  // namespace

extern "C" {

int bitcos_gemv_static(const bitcos_weights *W, const int8_t *x, const float *x_scale, int batch, float *y,
                       void *cuda_stream) {
    if (!W) return BITCOS_ERR_NULL;
    if (W->M < 1 || W->K < kGroup || W->K % kGroup != 0) return BITCOS_ERR_SHAPE;
    const size_t need = workspace_bytes_for(W->M, W->K);
    if (need > static_cast<size_t>(BITCOS_STATIC_WORKSPACE_BYTES)) return BITCOS_ERR_CAPACITY;
    void *ws = nullptr;
    int rc = static_workspace_ptr(&ws);
    if (rc) return rc;
    // (nothing is enqueued for a call that is going to be refused)
    rc = check_common(kBitcos, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x, x_scale, batch, y, nullptr, ws,
                      BITCOS_STATIC_WORKSPACE_BYTES);
    if (rc) return rc;
    // The array keeps whatever the last call left.  The status word and the arrival counters must
    // start at zero, so they are cleared on the caller's stream ahead of the kernel (the partial
    // sums behind them are always written before they are read).
    const size_t head = kHeaderBytes + counters_bytes(padded_rows(W->M) / kRows);
    rc = check_cuda(cudaMemsetAsync(ws, 0, head, static_cast<cudaStream_t>(cuda_stream)));
    if (rc) return rc;
    return gemv_common(kBitcos, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x, x_scale, batch, y,
                       nullptr, ws, BITCOS_STATIC_WORKSPACE_BYTES, cuda_stream, W->tile_off_host);
}

int bitcos_gemv_static_status(void *cuda_stream, int *status) {
    if (!status) return BITCOS_ERR_NULL;
    void *ws = nullptr;
    const int rc = static_workspace_ptr(&ws);
    if (rc) return rc;
    return bitcos_workspace_status(ws, cuda_stream, status);
}

int bitcos_wait_probe(void *workspace, uint64_t limit_ns, uint64_t *waited_ns, void *cuda_stream) {
    if (!workspace) return BITCOS_ERR_NULL;
    if (limit_ns < 1000 || limit_ns > 100ull * 1000 * 1000) return BITCOS_ERR_SHAPE;      // 1 us .. 100 ms
    wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<unsigned int *>(workspace), limit_ns,
                                                                        reinterpret_cast<unsigned long long *>(waited_ns));
    return check_cuda(cudaGetLastError());
}

int bitcos_quantize_activations(const uint16_t *x_bf16, int batch, int64_t K, int group, int8_t *xq, float *x_scale,
                                void *cuda_stream) {
    if (!x_bf16 || !xq || !x_scale) return BITCOS_ERR_NULL;
    if (batch < 1 || batch > BITCOS_MAX_BATCH || K < kGroup || K % kGroup != 0) return BITCOS_ERR_SHAPE;
    if (group != 0 && group != kGroup) return BITCOS_ERR_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(xq)) return BITCOS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (group == 0)
        return launch_pdl(quantize_tokens_kernel, dim3(static_cast<unsigned>(batch)), kQuantThreads, 0, stream, x_bf16, xq,
                          x_scale, K);
    const int64_t n_groups = static_cast<int64_t>(batch) * (K / kGroup);
    const int64_t blocks = (n_groups + 7) / 8;
    return launch_pdl(quantize_groups_kernel, dim3(static_cast<unsigned>(blocks)), 256, 0, stream, x_bf16, xq, x_scale,
                      n_groups);
}

int bitcos_gemv_group_scales(const bitcos_weights *W, const int8_t *x, const float *x_group_scale, int batch, float *y,
                             int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!W) return BITCOS_ERR_NULL;
    return gemv_common(kBitcos, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x, x_group_scale, batch, y,
                       acc_debug, workspace, workspace_bytes, cuda_stream, W->tile_off_host, true);
}

}  // extern "C"

namespace {
// bf16 = true: every job's x holds 16-bit activations (x_scale is not used) and the decoder warps
// quantise them per group of 128; one or two tokens.
#ifdef BITCOS_TIMELINE
unsigned long long *g_tl_buf = nullptr;
int g_tl_slots = 0, g_tl_next = 0;
#endif

int gemv_multi_common(const bitcos_gemv_job *jobs, int n_jobs, int batch, void *cuda_stream, bool bf16,
                      bool group_scales = false, const bitcos_weights *const *next = nullptr, int n_next = 0,
                      const bitcos_weights *const *prev = nullptr, int n_prev = 0) {
    if (!jobs) return BITCOS_ERR_NULL;
    if (n_jobs < 1 || n_jobs > kMaxJobs) return BITCOS_ERR_SHAPE;
    if (bf16 && batch > 2) return BITCOS_ERR_SHAPE;
    if (n_next < 0 || n_next * 4 > kMaxPrefetch || (n_next > 0 && !next)) return BITCOS_ERR_SHAPE;
    if (n_prev < 0 || n_prev > kMaxJobs || (n_prev > 0 && !prev)) return BITCOS_ERR_SHAPE;
    // thread blocks of the launch the caller says runs directly before this one (same batch)
    int busy = 0;
    if (n_prev > 0) {
        MultiArgs pm{};
        pm.n = n_prev;
        int64_t kprev = 0;
        for (int i = 0; i < n_prev; ++i) {
            const bitcos_weights *w = prev[i];
            if (!w) return BITCOS_ERR_NULL;
            if (w->M < 1 || w->K < kGroup || w->K % kGroup) return BITCOS_ERR_SHAPE;
            pm.pl[i] = make_plan(w->M, w->K, decoder_warps(batch));
            pm.pr[i].M = w->M;
            pm.pr[i].K = w->K;
            kprev = w->K > kprev ? w->K : kprev;
        }
        int dev = 0, sms = 0;
        int rc = check_cuda(cudaGetDevice(&dev));
        if (!rc) rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (rc) return rc;
        bool two = false;
        int grids[kMaxJobs];
        busy = plan_multi(pm, nb_bucket(batch, kprev), sms, &two, grids);
    }
    MultiArgs ma{};
    ma.n = n_jobs;
#ifdef BITCOS_TIMELINE
    if (g_tl_buf) ma.pf.tl = g_tl_buf + static_cast<size_t>(g_tl_next++ % g_tl_slots) * kMaxGrid * 32;
#endif
    for (int i = 0; i < n_next; ++i) {
        const bitcos_weights *w = next[i];
        if (!w || !w->bitmap || !w->signs || !w->tile_off || !w->scales) return BITCOS_ERR_NULL;
        if (w->M < 1 || w->K < kGroup || w->K % kGroup) return BITCOS_ERR_SHAPE;
        const uint64_t tiles = static_cast<uint64_t>(padded_rows(w->M) / kRows) * static_cast<uint64_t>(w->K / kGroup);
        auto add = [&](const void *p, uint64_t bytes) {
            bytes &= ~static_cast<uint64_t>(15);
            if (bytes > 0xFFFFFFF0ull) bytes = 0xFFFFFFF0ull;
            if (!bytes || (reinterpret_cast<uintptr_t>(p) & 15)) return;
            ma.pf.ptr[ma.pf.n] = static_cast<const uint8_t *>(p);
            ma.pf.bytes[ma.pf.n++] = static_cast<uint32_t>(bytes);
        };
        add(w->bitmap, tiles * 512);
        add(w->scales, tiles * kRows * sizeof(uint16_t));
        add(w->tile_off, (tiles + 1) * sizeof(uint32_t));
        // the length of the sign vector is only known from the host copy of the entry offsets
        if (w->tile_off_host)
            add(w->signs, (static_cast<uint64_t>(host_offset(w->tile_off_host, static_cast<int64_t>(tiles))) + 31) / 32 * 4);
    }
    // The request pays when the launches are short and the later one starts from L2 instead of device
    // memory (a 2B model's layer: requests of 3.8 and 7.6 MB, 0.45 us of 16 gained); asking for more
    // only competes with the launch's own stream (a 32B model's layer, requests of 9 to 54 MB: 1-3 %
    // slower), so a large request is dropped whole.
    {
        uint64_t requested = 0;
        for (int i = 0; i < ma.pf.n; ++i) requested += ma.pf.bytes[i];
        if (requested > BITCOS_PREFETCH_MAX_BYTES) ma.pf.n = 0;
    }
    for (int j = 0; j < n_jobs; ++j) {
        bitcos_gemv_job jb = jobs[j];
        if (!jb.W) return BITCOS_ERR_NULL;
        if (bf16) jb.x_scale = reinterpret_cast<const float *>(jb.x);        // never read; passes the NULL check
        const int bad = check_common(kBitcos, jb.W->bitmap, jb.W->signs, jb.W->tile_off, jb.W->scales, jb.W->M, jb.W->K,
                                     jb.x, jb.x_scale, batch, jb.y, nullptr, jb.workspace, jb.workspace_bytes);
        if (bad) return bad;
        for (int i = 0; i < j; ++i)
            if (jobs[i].workspace == jb.workspace) return BITCOS_ERR_SHAPE;      // jobs run concurrently
        ma.pl[j] = make_plan(jb.W->M, jb.W->K, decoder_warps(batch));
        fill_problem(ma.pr[j], jb.W->bitmap, jb.W->signs, jb.W->tile_off, jb.W->scales, jb.W->M, jb.W->K, jb.x,
                     jb.x_scale, batch, jb.y, nullptr, jb.workspace);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int64_t kmax = 0;
    for (int j = 0; j < n_jobs; ++j) kmax = jobs[j].W->K > kmax ? jobs[j].W->K : kmax;
    const int nbk = nb_bucket(batch, kmax);
    const uint32_t *off_host[kMaxJobs];
    for (int j = 0; j < n_jobs; ++j) off_host[j] = jobs[j].W->tile_off_host;
    if (bf16) {
        if (nbk == 1) return launch_multi<1, true>(ma, stream, off_host);
        if (nbk == 2) return launch_multi<2, true>(ma, stream, off_host);
        return BITCOS_ERR_SHAPE;          // rows too long for the one- and two-token kernels
    }
    if (group_scales) {
        if (nbk == 1) return launch_multi<1, false, true>(ma, stream, off_host);
        if (nbk == 2) return launch_multi<2, false, true>(ma, stream, off_host);
        if (batch <= 4) return launch_multi<4, false, true>(ma, stream, off_host);
        if (batch <= 8) return launch_multi<8, false, true>(ma, stream, off_host);
        return launch_multi<16, false, true>(ma, stream, off_host);
    }
    if (nbk == 1) return launch_multi<1>(ma, stream, off_host, busy);
    if (nbk == 2) return launch_multi<2>(ma, stream, off_host, busy);
    if (batch <= 4) return launch_multi<4>(ma, stream, off_host, busy);
    if (batch <= 8) return launch_multi<8>(ma, stream, off_host, busy);
    return launch_multi<16>(ma, stream, off_host, busy);
}
}  // namespace

namespace {
template <int NB>
int launch_phased(PhasedArgs &pa, int n_jobs, const int *job_phase, cudaStream_t stream) {
    for (int j = 0; j < n_jobs; ++j)
        if (static_cast<int64_t>(NB) * pa.pr[j].K > kXResidentBytes) return BITCOS_ERR_SHAPE;
    int sms = 0, budget = 0;
    int rc = prepare_kernel<gemv_phased_kernel<NB>>(&sms, &budget);
    if (rc) return rc;
    if (sms > kMaxGrid) sms = kMaxGrid;
    // the layout every job shares: the widest plan, the longest row
    Plan layout{};
    layout.tpw = 1;
    int64_t kmax = 0;
    int gmax = 0;
    for (int j = 0; j < n_jobs; ++j) {
        if (pa.pl[j].NW > layout.NW) layout.NW = pa.pl[j].NW;
        if (pa.pr[j].K > kmax) kmax = pa.pr[j].K;
        if (pa.pr[j].G > gmax) gmax = pa.pr[j].G;
    }
    layout.stages = choose_stages(kBitcos, layout, gmax, NB, kmax, budget);
    pa.layout = layout;
    pa.shape = Problem{};
    pa.shape.K = kmax;
    pa.shape.G = gmax;
    for (int p = 0; p < kMaxPhases; ++p) {
        pa.expect[p] = 0;
        for (int b = 0; b < kMaxGrid; ++b) pa.job_of[p][b] = 0xFF;
    }
    int grid = 1;
    for (int p = 0; p < pa.n_phases; ++p) {
        // the multiprocessors are shared between the phase's jobs in proportion to their item counts
        int64_t total_items = 0;
        for (int j = 0; j < n_jobs; ++j)
            if (job_phase[j] == p) total_items += pa.pl[j].items;
        int next = 0;
        for (int j = 0; j < n_jobs; ++j) {
            if (job_phase[j] != p) continue;
            int64_t cap = pa.pl[j].items;
            if (total_items > sms) {
                cap = pa.pl[j].items * sms / total_items;
                if (cap < 1) cap = 1;
            }
            int blocks = 1;
            choose_walk(pa.pl[j], static_cast<int>(cap), &blocks);
            if (next + blocks > kMaxGrid) return BITCOS_ERR_SHAPE;
            pa.pl[j].NW = layout.NW;
            pa.pl[j].stages = layout.stages;
            pa.job_first_block[j] = next;
            pa.job_blocks[j] = blocks;
            for (int b = 0; b < blocks; ++b) {
                pa.job_of[p][next + b] = static_cast<uint8_t>(j);
                if (make_walk(pa.pl[j], b, blocks).count > 0) ++pa.expect[p];
            }
            next += blocks;
        }
        if (next > grid) grid = next;
    }
    const SmemLayout L = smem_layout(kBitcos, layout, gmax, NB, kmax);
    if (static_cast<int>(L.total) > budget) return BITCOS_ERR_SHAPE;
    return launch_pdl(gemv_phased_kernel<NB>, dim3(static_cast<unsigned>(grid)), (layout.NW + 2) * 32, L.total, stream, pa);
}
}  // namespace

extern "C" {

int bitcos_gemv_phased(const bitcos_gemv_job *jobs, const int *job_phase, int n_jobs, int batch, void *sync,
                       void *cuda_stream) {
    if (!jobs || !job_phase || !sync) return BITCOS_ERR_NULL;
    if (n_jobs < 1 || n_jobs > kMaxJobs || batch < 1 || batch > 2) return BITCOS_ERR_SHAPE;
    if (!aligned16(sync)) return BITCOS_ERR_ALIGN;
    if (job_phase[0] != 0) return BITCOS_ERR_SHAPE;
    for (int j = 1; j < n_jobs; ++j)
        if (job_phase[j] < job_phase[j - 1] || job_phase[j] > job_phase[j - 1] + 1) return BITCOS_ERR_SHAPE;
    if (job_phase[n_jobs - 1] >= kMaxPhases) return BITCOS_ERR_SHAPE;
    static PhasedArgs pa_storage;      // (large: kept off the stack; calls are serialised by the lock below)
    static std::mutex lock;
    std::lock_guard<std::mutex> guard(lock);
    PhasedArgs &pa = pa_storage;
    pa.n_phases = job_phase[n_jobs - 1] + 1;
    pa.sync = static_cast<unsigned int *>(sync);
#ifdef BITCOS_TIMELINE
    pa.tl = g_tl_buf ? g_tl_buf + static_cast<size_t>(g_tl_next++ % g_tl_slots) * kMaxGrid * 32 : nullptr;
#endif
    for (int j = 0; j < n_jobs; ++j) {
        const bitcos_gemv_job &jb = jobs[j];
        if (!jb.W) return BITCOS_ERR_NULL;
        const int bad = check_common(kBitcos, jb.W->bitmap, jb.W->signs, jb.W->tile_off, jb.W->scales, jb.W->M, jb.W->K,
                                     jb.x, jb.x_scale, batch, jb.y, nullptr, jb.workspace, jb.workspace_bytes);
        if (bad) return bad;
        for (int i = 0; i < j; ++i)
            if (jobs[i].workspace == jb.workspace) return BITCOS_ERR_SHAPE;
        pa.pl[j] = make_plan(jb.W->M, jb.W->K, decoder_warps(batch));
        fill_problem(pa.pr[j], jb.W->bitmap, jb.W->signs, jb.W->tile_off, jb.W->scales, jb.W->M, jb.W->K, jb.x,
                     jb.x_scale, batch, jb.y, nullptr, jb.workspace);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (batch == 1) return launch_phased<1>(pa, n_jobs, job_phase, stream);
    return launch_phased<2>(pa, n_jobs, job_phase, stream);
}

#ifdef BITCOS_TIMELINE
// Debug build only: device buffer of slots x 160 blocks x 16 stamps; every multi launch takes the next slot.
void bitcos_debug_timeline(unsigned long long *buf, int slots) {
    g_tl_buf = buf;
    g_tl_slots = slots;
    g_tl_next = 0;
}
#endif

int bitcos_gemv_multi_plan(const int64_t *M, const int64_t *K, int n_jobs, int batch, int multiprocessors,
                           int busy_multiprocessors, int capacity, int *block_job, int *block_first_item, int *block_items,
                           int *job_items, int *job_tiles_per_item, int *job_column_blocks, int *job_chunk_stride,
                           int *n_blocks) {
    if (!M || !K || !block_job || !block_first_item || !block_items || !job_items || !job_tiles_per_item ||
        !job_column_blocks || !job_chunk_stride || !n_blocks)
        return BITCOS_ERR_NULL;
    if (n_jobs < 1 || n_jobs > kMaxJobs || batch < 1 || batch > BITCOS_MAX_BATCH || multiprocessors < 1 ||
        multiprocessors > kMaxGrid || busy_multiprocessors < 0)
        return BITCOS_ERR_SHAPE;
    static thread_local MultiArgs ma;
    ma = MultiArgs{};
    ma.n = n_jobs;
    int64_t kmax = 0;
    for (int j = 0; j < n_jobs; ++j) {
        if (M[j] < 1 || K[j] < kGroup || K[j] % kGroup) return BITCOS_ERR_SHAPE;
        ma.pl[j] = make_plan(M[j], K[j], decoder_warps(batch));
        ma.pr[j].M = M[j];
        ma.pr[j].K = K[j];
        ma.pr[j].G = static_cast<int>(K[j] / kGroup);
        ma.pr[j].RB = static_cast<int>(padded_rows(M[j]) / kRows);
        kmax = K[j] > kmax ? K[j] : kmax;
    }
    bool two = false;
    int grids[kMaxJobs];
    const int total = plan_multi(ma, nb_bucket(batch, kmax), multiprocessors, &two, grids);
    if (total > capacity) return BITCOS_ERR_CAPACITY;
    static thread_local int first[kMaxGrid], count[kMaxGrid];
    if (skewed_assignment(ma, grids, total, two, multiprocessors, busy_multiprocessors, first, count)) {
        for (int b = 0; b < total; ++b) {
            block_job[b] = ma.job_of[b];
            block_first_item[b] = first[b];
            block_items[b] = count[b];
        }
    } else {
        int b = 0;
        for (int j = 0; j < n_jobs; ++j)
            for (int r = 0; r < grids[j]; ++r, ++b) {
                const Walk w = make_walk(ma.pl[j], r, grids[j]);
                block_job[b] = j;
                block_first_item[b] = w.first;
                block_items[b] = w.count;
            }
    }
    for (int j = 0; j < n_jobs; ++j) {
        job_items[j] = static_cast<int>(ma.pl[j].items);
        job_tiles_per_item[j] = ma.pl[j].NW * ma.pl[j].tpw;
        job_column_blocks[j] = ma.pl[j].CS;
        job_chunk_stride[j] = ma.pl[j].cyclic ? grids[j] : 1;
    }
    *n_blocks = total;
    return BITCOS_OK;
}

int bitcos_gemv_multi_chained(const bitcos_gemv_job *jobs, int n_jobs, int batch, const bitcos_weights *const *prev,
                              int n_prev, const bitcos_weights *const *next, int n_next, void *cuda_stream) {
    return gemv_multi_common(jobs, n_jobs, batch, cuda_stream, false, false, next, n_next, prev, n_prev);
}

int bitcos_gemv_multi(const bitcos_gemv_job *jobs, int n_jobs, int batch, void *cuda_stream) {
    return gemv_multi_common(jobs, n_jobs, batch, cuda_stream, false);
}

int bitcos_gemv_multi_group_scales(const bitcos_gemv_job *jobs, int n_jobs, int batch, void *cuda_stream) {
    return gemv_multi_common(jobs, n_jobs, batch, cuda_stream, false, true);
}

int bitcos_gemv_multi_bf16(const bitcos_gemv_job *jobs, int n_jobs, int batch, void *cuda_stream) {
    return gemv_multi_common(jobs, n_jobs, batch, cuda_stream, true);
}

int bitcos_gemv_blend_bf16(const bitcos_weights *W, const uint16_t *x_bf16, int batch, float *y, void *workspace,
                           size_t workspace_bytes, void *cuda_stream) {
    if (!W) return BITCOS_ERR_NULL;
    if (batch > 8) return BITCOS_ERR_SHAPE;
    const int8_t *x = reinterpret_cast<const int8_t *>(x_bf16);
    const int bad = check_common(kBitcos, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x,
                                 reinterpret_cast<const float *>(x), batch, y, nullptr, workspace, workspace_bytes);
    if (bad) return bad;
    const Plan pl = make_plan(W->M, W->K, decoder_warps(8));
    Problem pr{};
    fill_problem(pr, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x, nullptr, batch, y, nullptr, workspace);
    return launch<kBitcos, 8, false, false, true>(pr, pl, static_cast<cudaStream_t>(cuda_stream), W->tile_off_host);
}

int bitcos_gemv_bf16(const bitcos_weights *W, const uint16_t *x_bf16, int batch, float *y, int32_t *acc_debug,
                     void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!W) return BITCOS_ERR_NULL;
    if (batch > 2) return BITCOS_ERR_SHAPE;
    const int8_t *x = reinterpret_cast<const int8_t *>(x_bf16);
    const int bad = check_common(kBitcos, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x,
                                 reinterpret_cast<const float *>(x), batch, y, acc_debug, workspace, workspace_bytes);
    if (bad) return bad;
    const Plan pl = make_plan(W->M, W->K, decoder_warps(batch));
    Problem pr{};
    fill_problem(pr, W->bitmap, W->signs, W->tile_off, W->scales, W->M, W->K, x, nullptr, batch, y, acc_debug, workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int nbk = nb_bucket(batch, W->K);
    if (nbk == 1) return launch<kBitcos, 1, false, true>(pr, pl, stream, W->tile_off_host);
    if (nbk == 2) return launch<kBitcos, 2, false, true>(pr, pl, stream, W->tile_off_host);
    return BITCOS_ERR_SHAPE;              // rows too long for the one- and two-token kernels
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

int bitcos_gemv_multi_host(const bitcos_gemv_host_job *jobs, int n_jobs, int batch, void *cuda_stream) {
    if (!jobs) return BITCOS_ERR_NULL;
    if (n_jobs < 1 || n_jobs > kMaxJobs) return BITCOS_ERR_SHAPE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    bitcos_gemv_job dev_jobs[kMaxJobs];
    float *y_dev[kMaxJobs];
    for (int j = 0; j < n_jobs; ++j) {
        const bitcos_gemv_host_job &jb = jobs[j];
        if (!jb.W || !jb.x_host || !jb.x_scale_host || !jb.y_host || !jb.staging) return BITCOS_ERR_NULL;
        const size_t need = bitcos_gemv_host_staging_bytes(jb.W->M, jb.W->K, batch);
        if (need == 0) return BITCOS_ERR_SHAPE;
        if (jb.staging_bytes < need) return BITCOS_ERR_CAPACITY;
        if (!aligned16(jb.staging)) return BITCOS_ERR_ALIGN;
        uint8_t *base = static_cast<uint8_t *>(jb.staging);
        const size_t xb = (static_cast<size_t>(batch) * jb.W->K + 255) / 256 * 256;
        dev_jobs[j].W = jb.W;
        dev_jobs[j].x = reinterpret_cast<const int8_t *>(base);
        dev_jobs[j].x_scale = reinterpret_cast<const float *>(base + xb);
        y_dev[j] = reinterpret_cast<float *>(base + xb + 256);
        dev_jobs[j].y = y_dev[j];
        dev_jobs[j].workspace = jb.workspace;
        dev_jobs[j].workspace_bytes = jb.workspace_bytes;
    }
    for (int j = 0; j < n_jobs; ++j) {
        uint8_t *base = static_cast<uint8_t *>(jobs[j].staging);
        const size_t xb = (static_cast<size_t>(batch) * jobs[j].W->K + 255) / 256 * 256;
        int rc = check_cuda(cudaMemcpyAsync(base, jobs[j].x_host, static_cast<size_t>(batch) * jobs[j].W->K,
                                            cudaMemcpyHostToDevice, stream));
        if (rc) return rc;
        rc = check_cuda(cudaMemcpyAsync(base + xb, jobs[j].x_scale_host, static_cast<size_t>(batch) * sizeof(float),
                                        cudaMemcpyHostToDevice, stream));
        if (rc) return rc;
    }
    int rc = bitcos_gemv_multi(dev_jobs, n_jobs, batch, cuda_stream);
    if (rc) return rc;
    for (int j = 0; j < n_jobs; ++j) {
        rc = check_cuda(cudaMemcpyAsync(jobs[j].y_host, y_dev[j], static_cast<size_t>(batch) * jobs[j].W->M * sizeof(float),
                                        cudaMemcpyDeviceToHost, stream));
        if (rc) return rc;
    }
    return check_cuda(cudaStreamSynchronize(stream));
}

}  // extern "C"

namespace {
// The work of bitcos_gemv_phases_host on a stream: copy in, one launch per phase (each told which
// launch runs before it and which comes after it), copy out.
int host_step_enqueue(const bitcos_gemv_job *jobs, const int *job_phase, int n_jobs, int batch, const void *in_host,
                      void *in_device, size_t in_bytes, void *out_host, const void *out_device, size_t out_bytes,
                      cudaStream_t stream) {
    int rc = check_cuda(cudaMemcpyAsync(in_device, in_host, in_bytes, cudaMemcpyHostToDevice, stream));
    if (rc) return rc;
    const bitcos_weights *w[kMaxJobs];
    for (int j = 0; j < n_jobs; ++j) w[j] = jobs[j].W;
    int prev_first = 0, prev_n = 0;
    for (int first = 0; first < n_jobs;) {
        int last = first;
        while (last + 1 < n_jobs && job_phase[last + 1] == job_phase[first]) ++last;
        int next_n = 0;
        while (last + 1 + next_n < n_jobs && job_phase[last + 1 + next_n] == job_phase[last + 1] && next_n < kMaxPrefetch / 4) ++next_n;
        rc = bitcos_gemv_multi_chained(jobs + first, last - first + 1, batch, w + prev_first, prev_n, w + last + 1, next_n, stream);
        if (rc) return rc;
        prev_first = first;
        prev_n = last - first + 1;
        first = last + 1;
    }
    return check_cuda(cudaMemcpyAsync(out_host, out_device, out_bytes, cudaMemcpyDeviceToHost, stream));
}

// Recorded steps.  A record is keyed by everything the enqueued work depends on, by value: the job
// list, the descriptors behind it, the blocks and their sizes, the device; and it remembers every
// entry offset its plans took from the host copies of tile_off, which a replay compares with what
// is there now (packed arrays in device memory may change freely between calls: the kernels read
// them when they run).  Anything that does not match is simply enqueued directly.
struct alignas(8) HostStepKey {
    int n_jobs, batch, device, pad;
    int phase[kMaxJobs];
    bitcos_gemv_job jobs[kMaxJobs];
    bitcos_weights w[kMaxJobs];
    const void *in_host, *out_device;
    void *in_device, *out_host;
    size_t in_bytes, out_bytes;
};
struct HostStepRecord {
    HostStepKey key;
    uint64_t hash = 0;
    std::vector<std::pair<const uint32_t *, uint32_t>> offsets;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    uint64_t last_use = 0;
    int seen = 0;          // calls with this key so far
    bool failed = false;   // recording did not work for this key: never tried again
};
constexpr int kHostStepRecords = 64;
HostStepRecord g_host_steps[kHostStepRecords];
std::mutex g_host_steps_lock;
uint64_t g_host_steps_clock = 0;
cudaStream_t g_record_stream = nullptr;

void host_step_key(HostStepKey &k, const bitcos_gemv_job *jobs, const int *job_phase, int n_jobs, int batch, const void *in_host,
                   void *in_device, size_t in_bytes, void *out_host, const void *out_device, size_t out_bytes) {
    std::memset(&k, 0, sizeof(k));
    k.n_jobs = n_jobs;
    k.batch = batch;
    cudaGetDevice(&k.device);
    for (int j = 0; j < n_jobs; ++j) {
        k.phase[j] = job_phase[j];
        std::memcpy(&k.jobs[j], &jobs[j], sizeof(bitcos_gemv_job));
        std::memcpy(&k.w[j], jobs[j].W, sizeof(bitcos_weights));
    }
    k.in_host = in_host;
    k.in_device = in_device;
    k.in_bytes = in_bytes;
    k.out_host = out_host;
    k.out_device = out_device;
    k.out_bytes = out_bytes;
}

// true: the step was launched on `stream` as a recorded graph.  false: the caller enqueues it directly
// (first sight of these arguments, a stale record, or recording is not possible).
bool host_step_replay(const bitcos_gemv_job *jobs, const int *job_phase, int n_jobs, int batch, const void *in_host,
                      void *in_device, size_t in_bytes, void *out_host, const void *out_device, size_t out_bytes,
                      cudaStream_t stream) {
    static const char *env = std::getenv("BITCOS_HOST_GRAPH");
    if (env && env[0] == '0') return false;
    static thread_local HostStepKey key;
    host_step_key(key, jobs, job_phase, n_jobs, batch, in_host, in_device, in_bytes, out_host, out_device, out_bytes);
    uint64_t hash = 1469598103934665603ull;      // (FNV-1a over the key's words: only to skip most comparisons)
    {
        const uint64_t *kw = reinterpret_cast<const uint64_t *>(&key);
        for (size_t i = 0; i < sizeof(key) / 8; ++i) hash = (hash ^ kw[i]) * 1099511628211ull;
    }
    std::lock_guard<std::mutex> guard(g_host_steps_lock);
    HostStepRecord *rec = nullptr, *oldest = &g_host_steps[0];
    for (HostStepRecord &r : g_host_steps) {
        if (r.seen && r.hash == hash && std::memcmp(&r.key, &key, sizeof(key)) == 0) rec = &r;
        if (r.last_use < oldest->last_use) oldest = &r;
    }
    if (!rec) {
        // first sight: remember the arguments (in the least recently used slot), enqueue directly this time
        rec = oldest;
        if (rec->exec) cudaGraphExecDestroy(rec->exec);
        if (rec->graph) cudaGraphDestroy(rec->graph);
        rec->exec = nullptr;
        rec->graph = nullptr;
        rec->offsets.clear();
        rec->key = key;
        rec->hash = hash;
        rec->seen = 1;
        rec->failed = false;
        rec->last_use = ++g_host_steps_clock;
        return false;
    }
    rec->last_use = ++g_host_steps_clock;
    if (rec->failed) return false;
    if (rec->exec) {
        for (const auto &o : rec->offsets)
            if (*o.first != o.second) {        // the host copy of the entry offsets changed under the same descriptor
                cudaGraphExecDestroy(rec->exec);
                cudaGraphDestroy(rec->graph);
                rec->exec = nullptr;
                rec->graph = nullptr;
                rec->offsets.clear();
                rec->seen = 1;
                return false;
            }
        return cudaGraphLaunch(rec->exec, stream) == cudaSuccess;
    }
    // second sight: record the step on a stream of the library's own (nothing runs), then replay it
    ++rec->seen;
    cudaPointerAttributes ai{}, ao{};
    if (cudaPointerGetAttributes(&ai, in_host) != cudaSuccess || cudaPointerGetAttributes(&ao, out_host) != cudaSuccess ||
        ai.type != cudaMemoryTypeHost || ao.type != cudaMemoryTypeHost) {
        cudaGetLastError();
        rec->failed = true;       // pageable host blocks: their copies are not recorded
        return false;
    }
    if (!g_record_stream && cudaStreamCreateWithFlags(&g_record_stream, cudaStreamNonBlocking) != cudaSuccess) {
        cudaGetLastError();
        rec->failed = true;
        return false;
    }
    if (cudaStreamBeginCapture(g_record_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        cudaGetLastError();
        rec->failed = true;
        return false;
    }
    g_offset_log = &rec->offsets;
    const int rc = host_step_enqueue(jobs, job_phase, n_jobs, batch, in_host, in_device, in_bytes, out_host, out_device, out_bytes,
                                     g_record_stream);
    g_offset_log = nullptr;
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(g_record_stream, &graph);
    if (rc || ce != cudaSuccess || !graph || cudaGraphInstantiate(&rec->exec, graph, 0) != cudaSuccess) {
        cudaGetLastError();
        if (graph) cudaGraphDestroy(graph);
        rec->exec = nullptr;
        rec->offsets.clear();
        rec->failed = true;
        return false;
    }
    rec->graph = graph;
    // (neighbouring blocks share entry offsets: every address once)
    std::sort(rec->offsets.begin(), rec->offsets.end());
    rec->offsets.erase(std::unique(rec->offsets.begin(), rec->offsets.end()), rec->offsets.end());
    return cudaGraphLaunch(rec->exec, stream) == cudaSuccess;
}
}  // namespace

extern "C" {

int bitcos_gemv_phases_host(const bitcos_gemv_job *jobs, const int *job_phase, int n_jobs, int batch, const void *in_host,
                            void *in_device, size_t in_bytes, void *out_host, const void *out_device, size_t out_bytes,
                            void *cuda_stream) {
    if (!jobs || !job_phase || !in_host || !in_device || !out_host || !out_device) return BITCOS_ERR_NULL;
    if (n_jobs < 1 || n_jobs > kMaxJobs || in_bytes == 0 || out_bytes == 0) return BITCOS_ERR_SHAPE;
    if (job_phase[0] != 0) return BITCOS_ERR_SHAPE;
    for (int j = 1; j < n_jobs; ++j)
        if (job_phase[j] < job_phase[j - 1] || job_phase[j] > job_phase[j - 1] + 1) return BITCOS_ERR_SHAPE;
    // every job's activations, scales and outputs must lie inside the two blocks that are copied
    const uintptr_t in0 = reinterpret_cast<uintptr_t>(in_device), out0 = reinterpret_cast<uintptr_t>(out_device);
    for (int j = 0; j < n_jobs; ++j) {
        if (!jobs[j].W || !jobs[j].x || !jobs[j].x_scale || !jobs[j].y) return BITCOS_ERR_NULL;
        const uintptr_t x = reinterpret_cast<uintptr_t>(jobs[j].x), xs = reinterpret_cast<uintptr_t>(jobs[j].x_scale),
                        y = reinterpret_cast<uintptr_t>(jobs[j].y);
        const size_t xb = static_cast<size_t>(batch) * static_cast<size_t>(jobs[j].W->K), yb = static_cast<size_t>(batch) * static_cast<size_t>(jobs[j].W->M) * 4;
        if (x < in0 || x + xb > in0 + in_bytes || xs < in0 || xs + static_cast<size_t>(batch) * 4 > in0 + in_bytes) return BITCOS_ERR_CAPACITY;
        if (y < out0 || y + yb > out0 + out_bytes) return BITCOS_ERR_CAPACITY;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // A step that was seen before, argument for argument, is replayed as one CUDA graph (one call
    // into the driver instead of six); the first time round the work is enqueued directly.
    if (host_step_replay(jobs, job_phase, n_jobs, batch, in_host, in_device, in_bytes, out_host, out_device, out_bytes, stream))
        return check_cuda(cudaStreamSynchronize(stream));
    const int rc = host_step_enqueue(jobs, job_phase, n_jobs, batch, in_host, in_device, in_bytes, out_host, out_device,
                                     out_bytes, stream);
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

}  // extern "C"

namespace {
template <int FMT>
int grouped_common(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                   const int32_t *group_begin, int n_groups, const int32_t *pair_xrow, int n_pairs, int max_group_size,
                   const int8_t *x, int n_xrows, const float *x_scale, float *y, int32_t *acc_debug, void *workspace,
                   size_t workspace_bytes, void *cuda_stream, const int32_t *n_groups_dev = nullptr) {
    if (!experts || !group_expert || !group_begin || !pair_xrow || !x || !x_scale || !y || !workspace)
        return BITCOS_ERR_NULL;
    if (M < 1 || K < kGroup || K % kGroup != 0 || n_experts < 1 || n_groups < 1 || n_groups > 65535 ||
        (!n_groups_dev && n_pairs < n_groups) || n_pairs < 1 || n_xrows < 1 || max_group_size < 1 || max_group_size > BITCOS_MAX_BATCH)
        return BITCOS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y) || !aligned16(workspace) || (acc_debug && !aligned16(acc_debug)))
        return BITCOS_ERR_ALIGN;
    const size_t stride = workspace_bytes_for(M, K);
    if (workspace_bytes < stride * static_cast<size_t>(n_groups)) return BITCOS_ERR_CAPACITY;

    const Plan pl = make_plan(M, K, decoder_warps(max_group_size));
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
    pr.status = static_cast<unsigned int *>(workspace);
    GroupedArgs ga{experts, group_expert, group_begin, stride, n_experts, n_groups, 0, n_pairs, n_xrows, n_groups_dev};
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int nbk = nb_bucket(max_group_size, K);
    if (nbk == 1) return launch_grouped<FMT, 1>(pr, pl, ga, n_groups, stream);
    if (nbk == 2) return launch_grouped<FMT, 2>(pr, pl, ga, n_groups, stream);
    if (max_group_size <= 4) return launch_grouped<FMT, 4>(pr, pl, ga, n_groups, stream);
    if (max_group_size <= 8) return launch_grouped<FMT, 8>(pr, pl, ga, n_groups, stream);
    return launch_grouped<FMT, 16>(pr, pl, ga, n_groups, stream);
}
}  // namespace

extern "C" {

int bitcos_gemv_grouped(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                        const int32_t *group_begin, int n_groups, const int32_t *pair_xrow, int n_pairs,
                        int max_group_size, const int8_t *x, int n_xrows, const float *x_scale, float *y,
                        int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return grouped_common<kBitcos>(experts, n_experts, M, K, group_expert, group_begin, n_groups, pair_xrow, n_pairs,
                                   max_group_size, x, n_xrows, x_scale, y, acc_debug, workspace, workspace_bytes, cuda_stream);
}

int bitcos_gemv_grouped_lists(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                              const int32_t *group_begin, const int32_t *n_groups_device, int max_groups,
                              const int32_t *pair_xrow, int n_pairs, int max_group_size, const int8_t *x, int n_xrows,
                              const float *x_scale, float *y, int32_t *acc_debug, void *workspace, size_t workspace_bytes,
                              void *cuda_stream) {
    if (!n_groups_device) return BITCOS_ERR_NULL;
    return grouped_common<kBitcos>(experts, n_experts, M, K, group_expert, group_begin, max_groups, pair_xrow, n_pairs,
                                   max_group_size, x, n_xrows, x_scale, y, acc_debug, workspace, workspace_bytes, cuda_stream,
                                   n_groups_device);
}

int bitcos_group_pairs_device(const int32_t *pair_expert, const int32_t *pair_xrow, int n_pairs, int n_experts,
                              int32_t *group_expert, int32_t *group_begin, int32_t *pair_xrow_sorted, int32_t *order,
                              int32_t *n_groups, void *cuda_stream) {
    if (!pair_expert || !pair_xrow || !group_expert || !group_begin || !pair_xrow_sorted || !order || !n_groups)
        return BITCOS_ERR_NULL;
    if (n_pairs < 1 || n_pairs > BITCOS_GROUP_PAIRS_MAX || n_experts < 1 || n_experts > BITCOS_GROUP_EXPERTS_MAX) return BITCOS_ERR_SHAPE;
    return launch_pdl(group_pairs_kernel, dim3(1), kGroupPairsThreads, 0, static_cast<cudaStream_t>(cuda_stream), pair_expert,
                      pair_xrow, n_pairs, n_experts, group_expert, group_begin, pair_xrow_sorted, order, n_groups);
}

int trit5_gemv_grouped(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                       const int32_t *group_begin, int n_groups, const int32_t *pair_xrow, int n_pairs,
                       int max_group_size, const int8_t *x, int n_xrows, const float *x_scale, float *y,
                       int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return grouped_common<kTrit5>(experts, n_experts, M, K, group_expert, group_begin, n_groups, pair_xrow, n_pairs,
                                  max_group_size, x, n_xrows, x_scale, y, acc_debug, workspace, workspace_bytes, cuda_stream);
}

int bit2_gemv_grouped(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                      const int32_t *group_begin, int n_groups, const int32_t *pair_xrow, int n_pairs,
                      int max_group_size, const int8_t *x, int n_xrows, const float *x_scale, float *y,
                      int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return grouped_common<kBit2>(experts, n_experts, M, K, group_expert, group_begin, n_groups, pair_xrow, n_pairs,
                                 max_group_size, x, n_xrows, x_scale, y, acc_debug, workspace, workspace_bytes, cuda_stream);
}

}  // extern "C"
