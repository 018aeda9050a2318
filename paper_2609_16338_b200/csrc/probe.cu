// Decode-rate probe for the BITCOS decoders (bitcos_decode_probe_variant).
//
// The paper's two-term roofline (Eq. 6: time per block of weights = max(bytes / bandwidth, gamma))
// needs gamma, the cost of the unpack sequence with every operand already on chip.  This kernel
// measures it for each of the decoders in decode.cuh on REAL packed tiles: a thread block copies
// one item of tiles (bitmap, sign bits, entry offsets, activations) into shared memory once, then
// every warp decodes and contracts its tile `iters` times with nothing but shared-memory traffic,
// and the block's elapsed clock cycles are written out.  The int32 group accumulators of the last
// pass are written out too, so that a test can hold every decoder against the CPU oracle.
#include "bitcos.h"
#include "decode.cuh"

#include <cuda_runtime.h>

#include <cstdint>

namespace bitcos_detail {
void record_cuda_error(int e);
}

namespace {

using namespace bitcos_dev;

constexpr int kProbeMaxWarps = 32;

__device__ const Lut256 g_probe_nibble_lut = make_nibble_lut();

struct ProbeLayout {
    uint32_t lut, second, bitmap, signs, x, xp, total;
    uint32_t sign_words;      // capacity of the sign area in words
};

__host__ __device__ inline ProbeLayout probe_layout(int variant, int n_tiles) {
    ProbeLayout L{};
    uint32_t off = 0;
    L.lut = off;
    off += (variant <= 2 || variant >= 5) ? kLutBytes : 0;
    L.second = off;
    off += (variant == 2) ? ((kByteTableBytes + 127) / 128 * 128) : 0;
    L.bitmap = off;
    off += static_cast<uint32_t>(n_tiles) * 512u;
    L.signs = off;
    L.sign_words = static_cast<uint32_t>(n_tiles) * 128u + 16u;
    off += L.sign_words * 4u;
    L.x = off;
    off += static_cast<uint32_t>(n_tiles) * 128u;
    L.xp = off;
    off += static_cast<uint32_t>(n_tiles) * 128u;
    L.total = off + 64;
    return L;
}

// MAXW: the widest block (in warps) this instantiation is launched with; 32 warps leave 64
// registers per thread, 24 warps 85.
template <int VAR, int MAXW>
__global__ void __launch_bounds__(MAXW * 32, 1)
probe_variant_kernel(const uint32_t *__restrict__ bitmap, const uint32_t *__restrict__ signs, const uint32_t *__restrict__ tile_off,
                     uint32_t sign_words_avail, const int8_t *__restrict__ x, int iters, unsigned long long *cycles,
                     int32_t *acc_out) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_tiles = blockDim.x >> 5;
    const ProbeLayout L = probe_layout(VAR, n_tiles);
    uint8_t *lut = smem + L.lut;
    uint32_t *s_bitmap = reinterpret_cast<uint32_t *>(smem + L.bitmap);
    uint32_t *s_signs = reinterpret_cast<uint32_t *>(smem + L.signs);
    uint8_t *s_x = smem + L.x, *s_xp = smem + L.xp;

    // ---- set-up (untimed): tables, the item's packed bytes, activations in both orders
    if (VAR <= 1 || VAR >= 5) {
        // byte address = key * 256 + sub * 128 + lane * 4 (see make_bitcos_lut)
        for (int idx = threadIdx.x; idx < kLutBytes / 4; idx += blockDim.x) {
            const int key = idx >> 6, sub = (idx >> 5) & 1;
            reinterpret_cast<uint32_t *>(lut)[idx] = g_probe_nibble_lut.v[sub ? (((key & 15) << 4) | (key >> 4)) : key];
        }
    }
    if (VAR == 2) build_byte_tables(lut, smem + L.second);
    for (int i = threadIdx.x; i < n_tiles * 128; i += blockDim.x) s_bitmap[i] = bitmap[i];
    const uint32_t first_bit = tile_off[0];
    const uint32_t w0 = first_bit >> 5;
    for (uint32_t i = threadIdx.x; i < L.sign_words; i += blockDim.x)
        s_signs[i] = (w0 + i < sign_words_avail) ? signs[w0 + i] : 0u;
    for (int i = threadIdx.x; i < n_tiles * 128; i += blockDim.x) {
        s_x[i] = static_cast<uint8_t>(x[i]);
        // bit-plane order: byte b of word 8 j + p of a group = x[32 j + 8 b + p]
        const int g = i >> 7, k = i & 127, j = k >> 5, b = (k >> 3) & 3, p = k & 7;
        s_xp[g * 128 + (8 * j + p) * 4 + b] = static_cast<uint8_t>(x[i]);
    }
    __syncthreads();

    const uint32_t lane4 = static_cast<uint32_t>(lane) * 4u;
    const uint32_t toff = tile_off[warp] - (w0 << 5);          // this tile's first sign bit inside s_signs
    const uint8_t *xg = s_x + warp * 128, *xpg = s_xp + warp * 128;
    int xl[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) xl[j] = static_cast<int8_t>(xg[32 * j + lane]);
    int total = 0, last = 0;
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        asm volatile("" ::: "memory");            // every pass reads its operands from shared memory again
        int a;
        if (VAR == 4) {
            a = bitcos_tile_dot_lanes(s_bitmap + warp * 128, s_signs, toff, xl, lane);
        } else {
            const uint4 bm = reinterpret_cast<const uint4 *>(s_bitmap)[warp * 32 + lane];
            const int c = __popc(bm.x) + __popc(bm.y) + __popc(bm.z) + __popc(bm.w);
            int incl = c;
#pragma unroll
            for (int dd = 1; dd < 32; dd <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, incl, dd);
                if (lane >= dd) incl += v;
            }
            const uint32_t cursor = toff + static_cast<uint32_t>(incl - c);
            const uint32_t *sp = s_signs + (cursor >> 5);
            if (VAR == 0) {
                int w[32];
                bitcos_decode_row(bm, sp, cursor & 31u, lut, lane4, w);
                asm volatile("" ::: "memory");
                a = row_contract(w, reinterpret_cast<const int4 *>(xg));
            } else if (VAR == 1) {
                int acc[1];
                bitcos_row_dot<1>(bm, sp, cursor & 31u, lut, lane4, xg, 0u, 1, acc);
                a = acc[0];
            } else if (VAR == 2) {
                a = bitcos_row_dot_bytes(bm, sp, cursor & 31u, lut, smem + L.second, lane4, xg);
            } else if (VAR == 3) {
                a = bitcos_row_dot_planes(bm, sp, cursor & 31u, xpg);
            } else {
                a = bitcos_row_dot_split<VAR - 4>(bm, sp, cursor & 31u, lut, lane4, xg, xpg);     // variants 5, 6, 7: 1, 2, 3 words through the table
            }
        }
        last = a;
        total += a;
    }
    const long long t1 = clock64();
    __shared__ unsigned long long s_max;
    if (threadIdx.x == 0) s_max = 0;
    __syncthreads();
    if (lane == 0) atomicMax(&s_max, static_cast<unsigned long long>(t1 - t0));
    __syncthreads();
    if (threadIdx.x == 0) cycles[blockIdx.x] = s_max;
    if (acc_out && blockIdx.x == 0) acc_out[warp * 32 + lane] = last;
    if (total == 0x12345678 && acc_out) acc_out[0] = total;       // keeps the sum alive; never true in practice
}

template <int VAR, int MAXW>
int launch_probe_w(const uint32_t *bitmap, const uint32_t *signs, const uint32_t *tile_off, uint32_t sign_words, const int8_t *x,
                 int n_tiles, int iters, int blocks, unsigned long long *cycles, int32_t *acc_out, cudaStream_t stream) {
    const ProbeLayout L = probe_layout(VAR, n_tiles);
    cudaError_t e = cudaFuncSetAttribute(probe_variant_kernel<VAR, MAXW>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(L.total));
    if (e == cudaSuccess) {
        probe_variant_kernel<VAR, MAXW><<<blocks, n_tiles * 32, L.total, stream>>>(bitmap, signs, tile_off, sign_words, x, iters, cycles, acc_out);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        bitcos_detail::record_cuda_error(static_cast<int>(e));
        return BITCOS_ERR_CUDA;
    }
    return BITCOS_OK;
}

template <int VAR>
int launch_probe(const uint32_t *bitmap, const uint32_t *signs, const uint32_t *tile_off, uint32_t sign_words, const int8_t *x,
                 int n_tiles, int iters, int blocks, unsigned long long *cycles, int32_t *acc_out, cudaStream_t stream) {
    if (n_tiles <= 24) return launch_probe_w<VAR, 24>(bitmap, signs, tile_off, sign_words, x, n_tiles, iters, blocks, cycles, acc_out, stream);
    return launch_probe_w<VAR, kProbeMaxWarps>(bitmap, signs, tile_off, sign_words, x, n_tiles, iters, blocks, cycles, acc_out, stream);
}

}  // namespace

extern "C" int bitcos_decode_probe_variant(int variant, const uint32_t *bitmap, const uint32_t *signs, size_t sign_bytes,
                                           const uint32_t *tile_off, int n_tiles, const int8_t *x, int iters, int blocks,
                                           uint64_t *cycles, int32_t *acc_out, void *cuda_stream) {
    if (!bitmap || !signs || !tile_off || !x || !cycles) return BITCOS_ERR_NULL;
    if (variant < 0 || variant >= BITCOS_PROBE_VARIANTS || n_tiles < 1 || n_tiles > kProbeMaxWarps || iters < 1 ||
        iters > (1 << 20) || blocks < 1 || blocks > 4096)
        return BITCOS_ERR_SHAPE;
    const ProbeLayout L = probe_layout(variant, n_tiles);
    if (L.total > 227u * 1024u) return BITCOS_ERR_CAPACITY;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned long long *out = reinterpret_cast<unsigned long long *>(cycles);
    const uint32_t sw = static_cast<uint32_t>(sign_bytes / 4);
    switch (variant) {
        case 0: return launch_probe<0>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
        case 1: return launch_probe<1>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
        case 2: return launch_probe<2>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
        case 3: return launch_probe<3>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
        case 4: return launch_probe<4>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
        case 5: return launch_probe<5>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
        case 6: return launch_probe<6>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
        default: return launch_probe<7>(bitmap, signs, tile_off, sw, x, n_tiles, iters, blocks, out, acc_out, stream);
    }
}
