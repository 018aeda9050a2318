// Device-side BITCOS packer: dense int8 trits and row-major bf16 scales in device memory -> the
// four packed buffers of the layout in bitcos.h (Section II-A of the paper: presence bitmap,
// compacted sign vector in the same order; entry offsets per tile), byte for byte what the host
// packer writes.  Three kernels: bitmap + scales + per-tile counts; an exclusive scan of the counts
// (the entry offsets); the sign vector.  A set-up path, not the hot path: one warp per 32 x 128
// tile, lane = row, the same decomposition as the products.
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "bitcos.h"

namespace bitcos_detail {
void record_cuda_error(int e);      // defined next to bitcos_last_cuda_error
}

namespace {

constexpr int kGroup = BITCOS_GROUP;
constexpr int kRows = BITCOS_TILE_ROWS;
constexpr int kPackWarps = 8;       // tiles per thread block

// words of the caller's scratch
constexpr int kFlagTrit = 0;        // a weight outside {-1, 0, +1}
constexpr int kFlagScale = 1;       // a scale that is negative, NaN or Inf
constexpr int kFlagOverflow = 2;    // more than 2^32 - 1 non-zero weights
constexpr int kNnzLo = 4;           // 64-bit count of non-zero weights (two words, 8-byte aligned)

inline int check_cuda(cudaError_t e) {
    if (e == cudaSuccess) return BITCOS_OK;
    bitcos_detail::record_cuda_error(static_cast<int>(e));
    return BITCOS_ERR_CUDA;
}
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t padded_rows(int64_t M) { return (M + kRows - 1) / kRows * kRows; }

// Presence and negative masks of the four bytes of a word (bit i <-> byte i), and whether all
// four are in {-1, 0, +1}.
__device__ __forceinline__ uint32_t byte_tops(uint32_t m) {
    // bits 7, 15, 23, 31 -> bits 0..3 (the four partial products land on distinct bits: no carries)
    return ((m & 0x80808080u) * 0x00204081u) >> 28;
}
__device__ __forceinline__ void masks4(uint32_t w, uint32_t &pres, uint32_t &neg, bool &ok) {
    const uint32_t zero = __vcmpeq4(w, 0u), one = __vcmpeq4(w, 0x01010101u), minus = __vcmpeq4(w, 0xFFFFFFFFu);
    pres |= byte_tops(~zero);
    neg |= byte_tops(minus);
    ok = ok && ((zero | one | minus) == 0xFFFFFFFFu);
}

// The 128 weights of (row m, group g) as four presence words and four negative words (bit i of
// word j <-> k = 128 g + 32 j + i); rows beyond M read as zero.
__device__ __forceinline__ bool load_row_masks(const int8_t *__restrict__ trits, int64_t M, int64_t K, int64_t m, int g,
                                               uint32_t (&pres)[4], uint32_t (&neg)[4]) {
    bool ok = true;
#pragma unroll
    for (int j = 0; j < 4; ++j) pres[j] = neg[j] = 0u;
    if (m >= M) return true;
    const uint4 *src = reinterpret_cast<const uint4 *>(trits + m * K + static_cast<int64_t>(g) * kGroup);
#pragma unroll
    for (int q = 0; q < 8; ++q) {                     // 16 weights per load
        const uint4 v = __ldg(src + q);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t p = 0u, n = 0u;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t pp = 0u, nn = 0u;
            masks4(w[i], pp, nn, ok);
            p |= pp << (4 * i);
            n |= nn << (4 * i);
        }
        pres[q >> 1] |= p << (16 * (q & 1));
        neg[q >> 1] |= n << (16 * (q & 1));
    }
    return ok;
}

// Kernel 1: bitmap, scales in tile order, number of non-zero weights per tile (into tile_off).
__global__ void __launch_bounds__(kPackWarps * 32) pack_bitmap_kernel(const int8_t *__restrict__ trits,
                                                                      const uint16_t *__restrict__ scales, int64_t M, int64_t K,
                                                                      uint32_t *__restrict__ bitmap,
                                                                      uint16_t *__restrict__ scales_tiled,
                                                                      uint32_t *__restrict__ tile_off, int64_t n_tiles,
                                                                      unsigned int *__restrict__ flags) {
    const int lane = threadIdx.x & 31;
    const int G = static_cast<int>(K / kGroup);
    for (int64_t t = static_cast<int64_t>(blockIdx.x) * kPackWarps + (threadIdx.x >> 5); t < n_tiles;
         t += static_cast<int64_t>(gridDim.x) * kPackWarps) {
        const int64_t rb = t / G;
        const int g = static_cast<int>(t - rb * G);
        const int64_t m = rb * kRows + lane;
        uint32_t pres[4], neg[4];
        const bool ok = load_row_masks(trits, M, K, m, g, pres, neg);
        if (!ok) atomicOr(flags + kFlagTrit, 1u);
        reinterpret_cast<uint4 *>(bitmap)[t * kRows + lane] = make_uint4(pres[0], pres[1], pres[2], pres[3]);
        uint16_t s = 0;
        if (m < M) {
            s = scales[m * G + g];
            if ((s & 0x8000u) || (s & 0x7F80u) == 0x7F80u) atomicOr(flags + kFlagScale, 1u);
        }
        scales_tiled[t * kRows + lane] = s;
        unsigned int c = __popc(pres[0]) + __popc(pres[1]) + __popc(pres[2]) + __popc(pres[3]);
#pragma unroll
        for (int d = 16; d; d >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, d);
        if (lane == 0) tile_off[t] = c;
    }
}

// Kernel 2: exclusive scan of the per-tile counts in place, one thread block walking the array in
// chunks; tile_off[n_tiles] and the 64-bit total receive the sum.
constexpr int kScanThreads = 1024;
__global__ void __launch_bounds__(kScanThreads) scan_counts_kernel(uint32_t *__restrict__ tile_off, int64_t n_tiles,
                                                                   unsigned int *__restrict__ flags) {
    __shared__ unsigned long long warp_sum[kScanThreads / 32];
    __shared__ unsigned long long carry_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0ull;
    __syncthreads();
    for (int64_t base = 0; base < n_tiles; base += kScanThreads) {
        const int64_t i = base + threadIdx.x;
        const unsigned long long v = (i < n_tiles) ? tile_off[i] : 0ull;
        unsigned long long inc = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += o;
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        unsigned long long before = carry_s;
        for (int w = 0; w < warp; ++w) before += warp_sum[w];
        const unsigned long long excl = before + inc - v;
        if (i < n_tiles) {
            if (excl > 0xFFFFFFFFull) atomicOr(flags + kFlagOverflow, 1u);
            tile_off[i] = static_cast<uint32_t>(excl);
        }
        __syncthreads();
        if (threadIdx.x == kScanThreads - 1) carry_s = before + inc;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const unsigned long long total = carry_s;
        if (total > 0xFFFFFFFFull) atomicOr(flags + kFlagOverflow, 1u);
        tile_off[n_tiles] = static_cast<uint32_t>(total);
        flags[kNnzLo] = static_cast<unsigned int>(total);
        flags[kNnzLo + 1] = static_cast<unsigned int>(total >> 32);
    }
}

// The bits of `src` at the set positions of `mask`, packed towards bit 0 (the inverse of the
// deposit of Fig. 4).
__device__ __forceinline__ uint32_t extract_bits(uint32_t src, uint32_t mask) {
    // parallel-suffix compress: in round i every selected bit moves right by 2^i if the number of
    // unselected positions below it has bit i set (five rounds for 32 bits)
    uint32_t x = src & mask, m = mask;
    uint32_t mk = ~m << 1;                       // the unselected positions, moved up by one: what lies below each bit
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        uint32_t mp = mk ^ (mk << 1);            // prefix parity of mk
        mp ^= mp << 2;
        mp ^= mp << 4;
        mp ^= mp << 8;
        mp ^= mp << 16;
        const uint32_t mv = mp & m;              // bits to move in this round
        m = (m ^ mv) | (mv >> (1 << i));
        const uint32_t t = x & mv;
        x = (x ^ t) | (t >> (1 << i));
        mk &= ~mp;
    }
    return x;
}

// Kernel 3: the sign vector.  Row r of tile t owns the bits [tile_off[t] + (non-zeros of rows
// 0 .. r-1 of the tile), + its own non-zeros); it ORs them into the (zero-filled) vector.
__global__ void __launch_bounds__(kPackWarps * 32) pack_signs_kernel(const int8_t *__restrict__ trits, int64_t M, int64_t K,
                                                                     const uint32_t *__restrict__ tile_off,
                                                                     uint32_t *__restrict__ signs, int64_t n_tiles) {
    const int lane = threadIdx.x & 31;
    const int G = static_cast<int>(K / kGroup);
    for (int64_t t = static_cast<int64_t>(blockIdx.x) * kPackWarps + (threadIdx.x >> 5); t < n_tiles;
         t += static_cast<int64_t>(gridDim.x) * kPackWarps) {
        const int64_t rb = t / G;
        const int g = static_cast<int>(t - rb * G);
        uint32_t pres[4], neg[4];
        load_row_masks(trits, M, K, rb * kRows + lane, g, pres, neg);
        const unsigned int c = __popc(pres[0]) + __popc(pres[1]) + __popc(pres[2]) + __popc(pres[3]);
        unsigned int inc = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned int o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += o;
        }
        // this row's sign bits, compacted: up to 128 bits in four words
        uint32_t sb[5] = {0u, 0u, 0u, 0u, 0u};
        int filled = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t bits = extract_bits(neg[j], pres[j]);
            const int n = __popc(pres[j]);
            const int w = filled >> 5, sh = filled & 31;
            if (n) {
                sb[w] |= bits << sh;
                if (sh && sh + n > 32) sb[w + 1] |= bits >> (32 - sh);
            }
            filled += n;
        }
        // shifted to the row's position in the vector
        const uint64_t q0 = static_cast<uint64_t>(__ldg(tile_off + t)) + (inc - c);
        const uint64_t w0 = q0 >> 5;
        const int sh = static_cast<int>(q0 & 31u);
        const int words = (sh + static_cast<int>(c) + 31) >> 5;
        uint32_t prev = 0u;
        for (int i = 0; i < words; ++i) {
            const uint32_t cur = (i < 4) ? sb[i] : 0u;
            const uint32_t out = sh ? ((cur << sh) | (prev >> (32 - sh))) : cur;
            if (out) atomicOr(signs + w0 + i, out);
            prev = cur;
        }
    }
}

// Non-zero count and validity only (to size the sign vector before packing).
__global__ void __launch_bounds__(256) count_nnz_kernel(const int8_t *__restrict__ trits, int64_t n16,
                                                        unsigned int *__restrict__ flags) {
    unsigned long long c = 0ull;
    bool ok = true;
    const uint4 *src = reinterpret_cast<const uint4 *>(trits);
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n16;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const uint4 v = __ldg(src + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t p = 0u, n = 0u;
            masks4(w[j], p, n, ok);
            c += __popc(p);
        }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, d);
    if (!__all_sync(0xFFFFFFFFu, ok) && (threadIdx.x & 31) == 0) atomicOr(flags + kFlagTrit, 1u);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(reinterpret_cast<unsigned long long *>(flags + kNnzLo), c);
}

int grid_for(int64_t units, int per_block) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        sms = 128;
    const int64_t want = (units + per_block - 1) / per_block;
    const int64_t cap = static_cast<int64_t>(sms) * 8;
    return static_cast<int>(want < 1 ? 1 : (want < cap ? want : cap));
}

int read_flags(const void *scratch, cudaStream_t stream, unsigned int (&h)[8]) {
    int rc = check_cuda(cudaMemcpyAsync(h, scratch, sizeof h, cudaMemcpyDeviceToHost, stream));
    if (rc) return rc;
    return check_cuda(cudaStreamSynchronize(stream));
}

}  // namespace

extern "C" {

int bitcos_count_nnz_device(const int8_t *trits, int64_t M, int64_t K, uint64_t *nnz, void *scratch, void *cuda_stream) {
    if (!trits || !nnz || !scratch) return BITCOS_ERR_NULL;
    if (M < 1 || K < kGroup || K % kGroup != 0) return BITCOS_ERR_SHAPE;
    if (!aligned16(trits) || !aligned16(scratch)) return BITCOS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = check_cuda(cudaMemsetAsync(scratch, 0, BITCOS_PACK_SCRATCH_BYTES, stream));
    if (rc) return rc;
    const int64_t n16 = M * K / 16;
    count_nnz_kernel<<<grid_for(n16, 256 * 8), 256, 0, stream>>>(trits, n16, static_cast<unsigned int *>(scratch));
    rc = check_cuda(cudaGetLastError());
    if (rc) return rc;
    unsigned int h[8];
    rc = read_flags(scratch, stream, h);
    if (rc) return rc;
    if (h[kFlagTrit]) return BITCOS_ERR_TRIT;
    *nnz = static_cast<uint64_t>(h[kNnzLo]) | (static_cast<uint64_t>(h[kNnzLo + 1]) << 32);
    return BITCOS_OK;
}

int bitcos_pack_device(const int8_t *trits, const uint16_t *scales_bf16, int64_t M, int64_t K, uint32_t *bitmap,
                       uint32_t *signs, size_t sign_capacity_bytes, uint32_t *tile_off, uint16_t *scales_tiled,
                       uint32_t *tile_off_host, uint64_t *nnz_out, void *scratch, void *cuda_stream) {
    if (!trits || !scales_bf16 || !bitmap || !signs || !tile_off || !scales_tiled || !scratch) return BITCOS_ERR_NULL;
    if (M < 1 || K < kGroup || K % kGroup != 0) return BITCOS_ERR_SHAPE;
    if (!aligned16(trits) || !aligned16(scales_bf16) || !aligned16(bitmap) || !aligned16(signs) || !aligned16(tile_off) ||
        !aligned16(scales_tiled) || !aligned16(scratch))
        return BITCOS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int64_t n_tiles = padded_rows(M) / kRows * (K / kGroup);
    size_t off_bytes = 0;
    int rc = bitcos_pack_sizes(M, K, 0, nullptr, nullptr, &off_bytes, nullptr);
    if (rc) return rc;
    unsigned int *flags = static_cast<unsigned int *>(scratch);
    rc = check_cuda(cudaMemsetAsync(scratch, 0, BITCOS_PACK_SCRATCH_BYTES, stream));
    if (rc) return rc;
    rc = check_cuda(cudaMemsetAsync(tile_off, 0, off_bytes, stream));
    if (rc) return rc;
    pack_bitmap_kernel<<<grid_for(n_tiles, kPackWarps), kPackWarps * 32, 0, stream>>>(trits, scales_bf16, M, K, bitmap,
                                                                                    scales_tiled, tile_off, n_tiles, flags);
    rc = check_cuda(cudaGetLastError());
    if (rc) return rc;
    scan_counts_kernel<<<1, kScanThreads, 0, stream>>>(tile_off, n_tiles, flags);
    rc = check_cuda(cudaGetLastError());
    if (rc) return rc;
    unsigned int h[8];
    rc = read_flags(scratch, stream, h);
    if (rc) return rc;
    if (h[kFlagTrit]) return BITCOS_ERR_TRIT;
    if (h[kFlagScale]) return BITCOS_ERR_SCALE;
    if (h[kFlagOverflow]) return BITCOS_ERR_OVERFLOW;
    const uint64_t nnz = static_cast<uint64_t>(h[kNnzLo]) | (static_cast<uint64_t>(h[kNnzLo + 1]) << 32);
    size_t need = 0;
    rc = bitcos_pack_sizes(M, K, nnz, nullptr, &need, nullptr, nullptr);
    if (rc) return rc;
    if (sign_capacity_bytes < need) return BITCOS_ERR_CAPACITY;
    rc = check_cuda(cudaMemsetAsync(signs, 0, sign_capacity_bytes, stream));
    if (rc) return rc;
    pack_signs_kernel<<<grid_for(n_tiles, kPackWarps), kPackWarps * 32, 0, stream>>>(trits, M, K, tile_off, signs, n_tiles);
    rc = check_cuda(cudaGetLastError());
    if (rc) return rc;
    if (tile_off_host) {
        rc = check_cuda(cudaMemcpyAsync(tile_off_host, tile_off, off_bytes, cudaMemcpyDeviceToHost, stream));
        if (rc) return rc;
    }
    rc = check_cuda(cudaStreamSynchronize(stream));
    if (rc) return rc;
    if (nnz_out) *nnz_out = nnz;
    return BITCOS_OK;
}

}  // extern "C"
