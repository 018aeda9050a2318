/*
 * bitcos.h -- C ABI of the BITCOS ternary GEMV library for NVIDIA B200 (sm_100a).
 *
 * The library stores a ternary weight matrix W in {-1,0,+1}^{M x K} (M output rows, K
 * reduction length, one bf16 scale per row and group of 128 reduction elements) in three
 * formats and multiplies it with int8 activations:
 *
 *   BITCOS     presence bitmap (1 bit per weight) + compacted sign vector (1 bit per
 *              non-zero weight, same order) + entry offsets: 2 - z bits per weight at zero
 *              density z (paper Section II-A, Eq. 1).
 *   five-trit  five ternary digits per byte, 26 bytes per 128 weights (paper Section I).
 *   2-bit      two bits per weight (the paper's baseline format, Section III).
 *
 *     acc[b][m][g] = sum_{k in group g} W[m][k] * x[b][k]                    (int32, exact)
 *     y[b][m]      = x_scale[b] * sum_g float(scale[m][g]) * float(acc[b][m][g])   (fp32)
 *
 * (integer path of Section II-C: w = p - 2n, Eq. 2; int32 accumulation per group; the
 * group scale applied once per group).  Batch b = 0 .. batch-1, 1 <= batch <= 16; the
 * packed weights are read once per call, not once per token.
 *
 * Conventions
 *   - Every function returns a bitcos_status.  Nothing throws, prints or allocates.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA device memory of
 *     the current device, owned by the caller, 16-byte aligned.
 *   - Device entry points enqueue work on the given stream (a cudaStream_t passed as
 *     void*, NULL = default stream) and return without synchronising.  They never call
 *     cudaMalloc / cudaFree.
 *   - K must be a multiple of 128 (the only group size); any M >= 1.
 *
 * Storage order ("tensor order").  The paper leaves the order of weights inside the
 * bitmap open and itself interleaves 32 output rows (Fig. 2, Section II-D).  Here rows are
 * taken in blocks of 32 (Mp = M rounded up to 32; padding rows hold zero weights) and the
 * reduction in groups of 128.  A tile = (row block rb, group g), numbered
 * t = rb * (K/128) + g.  Inside a tile: row r = 0..31, then k ascending.  Hence
 *   bitmap    uint32[Mp*K/32]; word (t*32 + r)*4 + j holds k = 128g + 32j .. +31 of row
 *             32rb + r, bit i <-> k = 128g + 32j + i (LSB first);
 *   signs     uint32[]; bit q of the sign vector is bit (q & 31) of word q >> 5; the q-th
 *             sign bit belongs to the q-th set bit of the bitmap; 1 = negative (Eq. 4);
 *   tile_off  uint32[n_tiles + 1], zero padded to a multiple of 16 bytes; tile_off[t] = index
 *             of tile t's first sign bit, tile_off[n_tiles] = number of non-zero weights;
 *   scales    uint16[Mp*K/128] bf16 bit patterns, scale of (row 32rb + r, group g) at
 *             t*32 + r (padding rows +0).
 */
#ifndef BITCOS_H
#define BITCOS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BITCOS_GROUP 128
#define BITCOS_TILE_ROWS 32
#define BITCOS_MAX_BATCH 16

typedef enum bitcos_status {
    BITCOS_OK = 0,
    BITCOS_ERR_NULL = 1,      /* a required pointer is NULL */
    BITCOS_ERR_SHAPE = 2,     /* M < 1, K < 128, K % 128 != 0, batch outside 1..16, bad list */
    BITCOS_ERR_ALIGN = 3,     /* a device pointer is not 16-byte aligned */
    BITCOS_ERR_TRIT = 4,      /* a weight outside {-1,0,+1} / an invalid packed code */
    BITCOS_ERR_SCALE = 5,     /* a scale that is NaN, Inf or has its sign bit set */
    BITCOS_ERR_CAPACITY = 6,  /* an output or workspace buffer is too small */
    BITCOS_ERR_OVERFLOW = 7,  /* more than 2^32 - 1 non-zero weights */
    BITCOS_ERR_CUDA = 8       /* a CUDA runtime call failed; see bitcos_last_cuda_error() */
} bitcos_status;

/* Static string naming a status value. */
const char *bitcos_status_string(int status);
/* cudaError_t value of the last failed CUDA call made by this library in this thread. */
int bitcos_last_cuda_error(void);

/* ---------------------------------------------------------------------------------------
 * Host side: packers (paper Section II-A for BITCOS; Section I for five-trit; the 2-bit
 * format of Section III).  Synchronous, deterministic; every padding bit and byte written
 * is zero so that packed buffers can be compared with memcmp.
 * ------------------------------------------------------------------------------------- */

/* Sizes in bytes of the four BITCOS buffers for an M x K matrix with nnz non-zero weights.
 * sign_bytes = ceil(nnz/8) rounded up to 16, plus 32 bytes of zero slack (a decoder may
 * fetch a fixed-size aligned window at the last cursor).  Any output pointer may be NULL. */
int bitcos_pack_sizes(int64_t M, int64_t K, uint64_t nnz, size_t *bitmap_bytes, size_t *sign_bytes,
                      size_t *tile_off_bytes, size_t *scale_bytes);

/* Counts the non-zero weights of trits[M][K] (host, row major); ERR_TRIT on a bad value. */
int bitcos_count_nnz(const int8_t *trits, int64_t M, int64_t K, uint64_t *nnz);

/* Packs trits[M][K] (host, row major, values -1/0/+1) and scales_bf16[M][K/128] (host, row
 * major, bf16 bit patterns, finite and non-negative) into the four caller-provided host
 * buffers sized by bitcos_pack_sizes.  sign_capacity_bytes is the size of `signs`.
 * nnz_out (optional) receives the number of sign bits. */
int bitcos_pack(const int8_t *trits, const uint16_t *scales_bf16, int64_t M, int64_t K,
                uint32_t *bitmap, uint32_t *signs, size_t sign_capacity_bytes, uint32_t *tile_off,
                uint16_t *scales_tiled, uint64_t *nnz_out);

/* Inverse of bitcos_pack: trits_out[M][K] (host).  ERR_TRIT if the offsets do not match the
 * bitmap's population counts. */
int bitcos_unpack(const uint32_t *bitmap, const uint32_t *signs, const uint32_t *tile_off,
                  int64_t M, int64_t K, int8_t *trits_out);

/* Reorders row-major scales[M][K/128] into the tile order described above (and back). */
int bitcos_scales_tile(const uint16_t *scales_bf16, int64_t M, int64_t K, uint16_t *scales_tiled);
int bitcos_scales_untile(const uint16_t *scales_tiled, int64_t M, int64_t K, uint16_t *scales_bf16);

/* Five-trit: byte j of a 128-weight block = sum_{i<5} (t[5j+i] + 1) * 3^i; byte 25 carries
 * trits 125..127 and digit 1 in its two unused places; 26 bytes per block.  A row's K/128
 * blocks are concatenated, zero padded to a multiple of 4 bytes, and read as little-endian
 * 32-bit words; word q of row 32rb + r is stored at index (rb*WPR + q)*32 + r, where
 * WPR = ceil(26*(K/128)/4).  *bytes = Mp * WPR * 4. */
int trit5_pack_sizes(int64_t M, int64_t K, size_t *bytes);
int trit5_pack(const int8_t *trits, int64_t M, int64_t K, uint32_t *words);
int trit5_unpack(const uint32_t *words, int64_t M, int64_t K, int8_t *trits_out);

/* 2-bit: code = t + 1; 16 weights per 32-bit word, weight i at bits [8*(i%4) + 2*(i/4), +2);
 * a row is K/16 words; word j of 16-byte chunk c of row 32rb + r is stored at index
 * ((rb*(K/64) + c)*32 + r)*4 + j.  *bytes = Mp * K / 4. */
int bit2_pack_sizes(int64_t M, int64_t K, size_t *bytes);
int bit2_pack(const int8_t *trits, int64_t M, int64_t K, uint32_t *words);
int bit2_unpack(const uint32_t *words, int64_t M, int64_t K, int8_t *trits_out);

/* Which of the two compact formats stores an M x K matrix with nnz non-zero weights in fewer
 * bytes (Section II-A: BITCOS spends 2 - z bits per weight and the five-trit format 26 bytes
 * per 128 weights, so BITCOS wins above a zero density of 0.375; a tensor takes whichever rate
 * it meets first).  All bytes a product reads are counted, entry offsets included.
 * *format = 0 (BITCOS) or 1 (five-trit); the two byte counts are optional outputs. */
int bitcos_choose_format(int64_t M, int64_t K, uint64_t nnz, int *format, size_t *bitcos_bytes, size_t *trit5_bytes);

/* ---------------------------------------------------------------------------------------
 * Device side: packing.  The same four BITCOS buffers as bitcos_pack writes, byte for byte, from
 * trits and scales that are already in device memory (a checkpoint converted on the GPU).  A
 * set-up path: both calls enqueue on the given stream and WAIT for it before they return (they
 * report counts and errors to the host), so a product launched afterwards finds the packed
 * weights complete.  scratch: BITCOS_PACK_SCRATCH_BYTES of device memory, 16-byte aligned.
 * ------------------------------------------------------------------------------------- */
#define BITCOS_PACK_SCRATCH_BYTES 256

/* Number of non-zero weights of trits[M][K] (device, row major, int8); ERR_TRIT on a value
 * outside {-1, 0, +1}.  Size the sign vector with bitcos_pack_sizes from it. */
int bitcos_count_nnz_device(const int8_t *trits, int64_t M, int64_t K, uint64_t *nnz, void *scratch, void *cuda_stream);

/* Packs trits[M][K] (device int8, row major) and scales_bf16[M][K/128] (device, row major) into
 * the device buffers bitmap, signs (sign_capacity_bytes, zero filled here), tile_off and
 * scales_tiled, all sized by bitcos_pack_sizes.  tile_off_host (optional): host buffer of the
 * tile_off size receiving a copy (for bitcos_weights.tile_off_host).  nnz_out (optional, host).
 * ERR_TRIT / ERR_SCALE / ERR_OVERFLOW as for bitcos_pack; ERR_CAPACITY if the sign vector does
 * not fit (outputs are then incomplete). */
int bitcos_pack_device(const int8_t *trits, const uint16_t *scales_bf16, int64_t M, int64_t K, uint32_t *bitmap,
                       uint32_t *signs, size_t sign_capacity_bytes, uint32_t *tile_off, uint16_t *scales_tiled,
                       uint32_t *tile_off_host, uint64_t *nnz_out, void *scratch, void *cuda_stream);

/* ---------------------------------------------------------------------------------------
 * Device side: the products.
 * ------------------------------------------------------------------------------------- */

/* A packed BITCOS matrix in device memory (layout above). */
typedef struct bitcos_weights {
    const uint32_t *bitmap;
    const uint32_t *signs;
    const uint32_t *tile_off;
    const uint16_t *scales;   /* tile order */
    int64_t M;
    int64_t K;
    /* Optional (NULL if absent): a HOST copy of tile_off, as bitcos_pack wrote it.  With it the
     * launch hands every thread block the entry offsets of its first tiles by value, which takes one
     * dependent device-memory round trip out of the start of each call.  The paper has no
     * counterpart; results do not depend on it.  Ignored by bitcos_gemv_grouped (its descriptors
     * live in device memory). */
    const uint32_t *tile_off_host;
} bitcos_weights;

/* Stream ordering of the device entry points.  They enqueue on the caller's stream and return
 * without waiting.  Kernels of this library are launched with programmatic stream serialization:
 * when the previous kernel in the stream is also one of this library's, a call may start reading
 * its PACKED WEIGHTS (and nothing else) while that kernel is still running; activations, activation
 * scales, routing lists, outputs, accumulator dumps and workspaces are touched only after every
 * earlier kernel in the stream has completed, as usual.  The products and the quantiser never write
 * packed weights, and bitcos_pack_device waits for the stream before it returns, so ordinary use needs
 * no extra care; after any other kernel or copy in the stream the
 * usual order holds in full.  BITCOS_PDL=0 in the environment turns the overlap off. */

/* Scratch memory the GEMV entry points need for an M x K matrix (the same value for all
 * formats and batches): a 256-byte header (word 0 = status), one arrival counter per row
 * block, and the partial row sums of reduction segments that were spread over several
 * thread blocks.  The caller allocates it on the device, fills it with zeros ONCE
 * (bitcos_workspace_init), and may reuse it for any later call whose requirement is not
 * larger: every call leaves the counters zero.  Two calls that may run at the same time
 * must not share a workspace. */
size_t bitcos_gemv_workspace_bytes(int64_t M, int64_t K);
int bitcos_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Every wait inside the kernels (on the arrival of an asynchronous copy) is bounded; if one
 * ever runs out, the thread block stops working on the call and sets the workspace's status
 * word to 1 instead of hanging.  This call copies that word back (it waits for the stream):
 * *status == 0 means every call that used the workspace so far completed normally. */
int bitcos_workspace_status(const void *workspace, void *cuda_stream, int *status);

/* Measurement aid for the paper's two-term roofline (Section III-B.1, Eq. 6: T = max(B/beta, gamma)):
 * gamma is the cost of the unpack sequence when every operand is already on chip.  Launches
 * `blocks` thread blocks of `warps_per_block` warps (1..22); each warp decodes one synthetic
 * 32 x 128 tile held in shared memory `iters` times with the code the GEMV kernels run (format
 * 0 = BITCOS, 1 = five-trit, 2 = 2-bit) and nothing is read from global memory in the timed loop.
 * cycles (device, uint64 [blocks]) receives each block's elapsed SM clock cycles; cycles per 32
 * weights per multiprocessor = cycles / (iters * warps_per_block * 128). */
int bitcos_decode_probe(int format, int warps_per_block, int iters, int blocks, uint64_t *cycles, void *cuda_stream);

/* The same measurement for each of the library's BITCOS decoders, on real packed tiles, with the
 * accumulators handed back so that every decoder can be checked (Section II-D notes that the unpack
 * sequence, not the format, decides whether the saved bytes turn into time; Eq. 6's gamma is what
 * this measures).  bitmap / signs / tile_off describe one item of n_tiles consecutive tiles of a
 * packed matrix (device pointers: bitmap = the first tile's, tile_off = its entry, signs = the
 * matrix's whole sign vector of sign_bytes bytes); x = device int8 [n_tiles][128], the activations of
 * tile t's group.  A block of n_tiles warps (1..32) copies the item into shared memory once; warp t then
 * computes, `iters` times, the 32 int32 group accumulators of tile t (row r in lane r) from shared
 * memory only.  cycles (device uint64 [blocks]) as for bitcos_decode_probe; acc_out = NULL or device
 * int32 [n_tiles][32], written by block 0.
 *   variant 0  shifted window: (presence nibble, sign nibble) table of Eq. 4, the window of a word
 *              shifted by each nibble's population count; decode into registers, then contract
 *   variant 1  running position: the same table, windows never shifted, a running bit position per
 *              word updated by the dp4a that counts; contraction fused (what the products run)
 *   variant 2  byte table: eight weights per step from a 3^8-entry table behind a 256-entry index
 *   variant 3  no table: the deposit of Fig. 4 with shifts and masks, contraction on bit planes
 *   variant 4  lane = bit: one presence word per warp step, sign slot = population count of the
 *              lower bits, products added across the warp
 *   variant 5, 6, 7  split row: the first 1, 2, 3 presence words of a row as variant 1, the others as
 *              variant 3 (loads the shared-memory pipe and the integer ALU at the same time)
 * ERR_CAPACITY if the item does not fit into shared memory with the variant's tables. */
#define BITCOS_PROBE_VARIANTS 8
int bitcos_decode_probe_variant(int variant, const uint32_t *bitmap, const uint32_t *signs, size_t sign_bytes,
                                const uint32_t *tile_off, int n_tiles, const int8_t *x, int iters, int blocks,
                                uint64_t *cycles, int32_t *acc_out, void *cuda_stream);

/* y[b][m] for b < batch, m < M from a BITCOS matrix (steps of Section II-B..II-D on the GPU:
 * entry offset + running population count locate each row's sign window, a 256-entry
 * (presence nibble, sign nibble) table as in Eq. 4 rebuilds four weights at a time as int8,
 * dp4a accumulates int32 per group, the bf16 group scale and the per-token scale are applied
 * in fp32).  The paper measures one token; for batch >= 3 the same int32 group accumulators come
 * from int8 tensor-core instructions (mma.m16n8k32) fed with the decoded rows, so that the weights
 * are decoded once per call whatever the batch.  The accumulators are exact for every batch; y is
 * deterministic for a given batch size and device (fixed summation order), and the summation
 * order over groups may differ between batch sizes.
 *   W            host struct holding device pointers
 *   x            device int8 [batch][K], row major
 *   x_scale      device float [batch]
 *   y            device float [batch][M], overwritten
 *   acc_debug    NULL, or device int32 [batch][M][K/128] receiving every group accumulator
 *   workspace    device scratch of at least bitcos_gemv_workspace_bytes(M, K) bytes */
int bitcos_gemv(const bitcos_weights *W, const int8_t *x, const float *x_scale, int batch, float *y,
                int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Activation quantiser in front of the product.  Section II-C has the integer contraction
 * quantise the activations to int8 per group of 128 and apply the scales once per group; the
 * paper does not spell the rule out, and this library uses symmetric absmax quantisation, decided
 * in float32:
 *     a = max(max |x| over the group, 2^-100)     scale = a / 127     code = rint(x * (127 / a))
 * (IEEE quotient and product, ties to even; |code| <= 127; an all-zero group gets codes 0).
 *   x_bf16   device bf16 [batch][K] (bit patterns; finite values), 16-byte aligned
 *   group    128: one scale per token and group of 128, x_scale = device float [batch][K/128]
 *            0:   one scale per token (the whole row is one group), x_scale = device float [batch]
 *   xq       device int8 [batch][K], 16-byte aligned, overwritten
 * ERR_SHAPE for any other group, K not a multiple of 128, batch outside 1..BITCOS_MAX_BATCH.
 * Stream ordered like the products: it waits for the kernel before it before reading x_bf16,
 * and the product launched after it overlaps its own start-up with this kernel. */
int bitcos_quantize_activations(const uint16_t *x_bf16, int batch, int64_t K, int group, int8_t *xq, float *x_scale,
                                void *cuda_stream);

/* bitcos_gemv with one activation scale per token and group of 128 (Section II-C):
 *     y[b][m] = sum over groups g of  s[m][g] * x_group_scale[b][g] * (int32 sum over the group)
 *   x_group_scale   device float [batch][K/128], e.g. from bitcos_quantize_activations(group = 128)
 * Everything else as for bitcos_gemv (same accumulators, same workspace rules). */
int bitcos_gemv_group_scales(const bitcos_weights *W, const int8_t *x, const float *x_group_scale, int batch, float *y,
                             int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The quantiser fused into the product, for one or two tokens: x_bf16 = device bf16 [batch][K]
 * (bit patterns, 16-byte aligned); every decoder warp quantises the group of 128 its tile
 * multiplies (the rule of bitcos_quantize_activations, group = 128) and applies the group's
 * scale, so the result is exactly that of bitcos_quantize_activations followed by
 * bitcos_gemv_group_scales, without the separate launch and without the int8 copy in memory.
 * ERR_SHAPE for batch > 2 (use the two calls) and for rows too long for the one- and two-token
 * kernels (batch * K > 49152).  Everything else as for bitcos_gemv. */
int bitcos_gemv_bf16(const bitcos_weights *W, const uint16_t *x_bf16, int batch, float *y, int32_t *acc_debug,
                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The 16-bit variant of Sections II-B / II-D: no activation quantisation; the weights are rebuilt
 * as +s / 0 / -s (the bf16 group scale blended into the weight, exact) and multiplied with the
 * bf16 activations as they are,
 *     y[b][m] = sum over k of (W[m][k] * s[m][k / 128]) * x[b][k],
 * on the tensor cores (mma.m16n8k16, bf16 operands, fp32 accumulation over each group of 128; the
 * groups are then added in fp32 in the fixed order of the other products).  Every product is exact
 * in fp32; the sums are within 2e-5 of the sum of |terms|.  batch 1..8 (ERR_SHAPE above);
 * x_bf16 = device bf16 [batch][K], 16-byte aligned; no accumulator dump.  About twice the cost of
 * the integer product at one token (the decoded weights are expanded to 16 bits on the way to the
 * tensor cores), the same at eight. */
int bitcos_gemv_blend_bf16(const bitcos_weights *W, const uint16_t *x_bf16, int batch, float *y, void *workspace,
                           size_t workspace_bytes, void *cuda_stream);

#define BITCOS_MAX_JOBS 8

/* Up to BITCOS_MAX_JOBS independent BITCOS products in ONE launch (same batch; shapes may differ): e.g. the
 * q, k and v projections of a decoder layer, which read the same activations and do not depend on
 * one another, or gate and up.  The multiprocessors are shared between the jobs in proportion to
 * their sizes, so small matrices run side by side instead of one after the other and the fixed
 * cost of a launch is paid once.  Every job has its own outputs and its own workspace (sized and
 * zero filled as for bitcos_gemv; two jobs must not share one).  Results are identical to
 * n_jobs calls of bitcos_gemv. */
typedef struct bitcos_gemv_job {
    const bitcos_weights *W;   /* host struct of device pointers */
    const int8_t *x;           /* device int8 [batch][K] */
    const float *x_scale;      /* device float [batch] */
    float *y;                  /* device float [batch][M] */
    void *workspace;           /* device scratch, >= bitcos_gemv_workspace_bytes(M, K) */
    size_t workspace_bytes;
} bitcos_gemv_job;
int bitcos_gemv_multi(const bitcos_gemv_job *jobs, int n_jobs, int batch, void *cuda_stream);
/* bitcos_gemv_multi for a launch inside a fixed sequence of launches (the products of a decoder
 * layer, token after token), told what runs directly before it and what comes after it in the
 * stream.  Both are hints: results are those of bitcos_gemv_multi, bit for bit, whatever they hold.
 * The paper reads weights from memory as the product reaches them and has one product at a time
 * (Section II-D); neither hint has a counterpart there.
 *   next, n_next   matrices a LATER launch multiplies by (host array of pointers to host structs of
 *                  device pointers, n_next <= 7, may be 0): every thread block asks for its share of
 *                  their packed arrays to be brought into the level-2 cache once its own first copies
 *                  are under way.  Nothing waits for the requests and nothing is written.  The sign
 *                  vector of a matrix is only requested if its descriptor carries tile_off_host (its
 *                  length is not known otherwise).  Pays when launches are short: the later launch
 *                  starts from L2 instead of device memory.  A request for more than
 *                  BITCOS_PREFETCH_MAX_BYTES in total is ignored (it would only compete with the
 *                  launch's own reads).
 *   prev, n_prev   the matrices of the launch directly BEFORE this one in the stream (only M and K
 *                  are read; n_prev <= BITCOS_MAX_JOBS, may be 0 = unknown), same batch.  Kernels of
 *                  this library start before their predecessor has finished (see "stream ordering"),
 *                  but only on multiprocessors it has left free; the thread blocks that have to wait
 *                  for one go through their start-up late and fall about two work items behind.  Knowing
 *                  how many blocks the previous launch runs, this launch hands the blocks that start at
 *                  once correspondingly more items.  Only applied when every job's rows fit one work item
 *                  (K <= 2560 at up to eight tokens), where the split cannot touch any sum.  A wrong
 *                  hint costs time (an uneven split), never correctness.
 * Errors as bitcos_gemv_multi, plus BITCOS_ERR_NULL / BITCOS_ERR_SHAPE for a malformed list. */
#define BITCOS_PREFETCH_MAX_BYTES (8u << 20)
int bitcos_gemv_multi_chained(const bitcos_gemv_job *jobs, int n_jobs, int batch, const bitcos_weights *const *prev,
                              int n_prev, const bitcos_weights *const *next, int n_next, void *cuda_stream);
/* How a multi launch would hand its work to thread blocks, without launching anything (needs no
 * GPU): for tests and for callers who want to see the split.  M, K: the jobs' shapes (host arrays of
 * n_jobs); multiprocessors: of the device the launch is meant for; busy_multiprocessors: thread
 * blocks of the launch before it (what bitcos_gemv_multi_chained works out from `prev`), 0 = none.
 * Work is counted in items: a job's rows are cut into row blocks of 32 and, when a row is too long
 * for one item, into job_column_blocks[j] column blocks; item i of job j is column block
 * i % job_column_blocks[j] of chunk i / job_column_blocks[j] (a chunk = job_tiles_per_item[j] tiles'
 * worth of whole row blocks, or one row block).  Outputs (host): n_blocks; for every block its job,
 * its first item and its number of items (block_* hold `capacity` entries; ERR_CAPACITY if fewer than
 * n_blocks); per job the number of items, tiles per item, column blocks, and the chunk stride: 1 = the
 * block's items are consecutive; s > 1 = after the last column block of a chunk the block moves on
 * s chunks (blocks take chunks round robin). */
int bitcos_gemv_multi_plan(const int64_t *M, const int64_t *K, int n_jobs, int batch, int multiprocessors,
                           int busy_multiprocessors, int capacity, int *block_job, int *block_first_item, int *block_items,
                           int *job_items, int *job_tiles_per_item, int *job_column_blocks, int *job_chunk_stride,
                           int *n_blocks);
/* The same with one activation scale per token and group of 128 (see bitcos_gemv_group_scales):
 * every job's x_scale points to device float [batch][K/128]. */
int bitcos_gemv_multi_group_scales(const bitcos_gemv_job *jobs, int n_jobs, int batch, void *cuda_stream);
/* The same with 16-bit activations quantised inside the launch (see bitcos_gemv_bf16): every
 * job's x points to device bf16 [batch][K], x_scale is ignored (may be NULL); batch 1 or 2. */
int bitcos_gemv_multi_bf16(const bitcos_gemv_job *jobs, int n_jobs, int batch, void *cuda_stream);

/* Jobs in dependency order inside ONE launch.  job_phase[j] (0 .. BITCOS_MAX_PHASES - 1, non-decreasing
 * in j, starting at 0, no phase skipped) puts every job into a phase; the jobs of a phase are
 * independent of one another (as in bitcos_gemv_multi), and a job's activations x, x_scale are read
 * only after EVERY job of the phase before it has written all of its outputs -- so a job may consume
 * what the phase before produced.  The seven products of a decoder layer make four phases:
 * q | k | v, then o, then gate | up, then down (the paper's end-to-end runs execute exactly this
 * sequence per layer, one launch per product; Section III-B.5).  What does not depend on the phase
 * before runs ahead of the dependency: the next phase's packed weights are streamed and its first
 * tiles decoded while the current phase is still being finished, which is what a sequence of
 * launches cannot do.  Inside one launch nothing else can run between two phases: a layer whose
 * attention, normalisation or activation kernels sit between the products uses bitcos_gemv_multi
 * per phase instead.
 *   jobs, n_jobs   as for bitcos_gemv_multi (1 .. BITCOS_MAX_JOBS; own outputs and own workspace each)
 *   batch          1 or 2 (ERR_SHAPE above, and for rows too long for the one- and two-token kernels)
 *   sync           device scratch of BITCOS_PHASED_SYNC_BYTES, 16-byte aligned, zero filled ONCE; the
 *                  launch leaves it zero.  Two phased launches that may overlap must not share it.
 * Results are identical, bit for bit, to one bitcos_gemv_multi call per phase.  Every thread block
 * waits for the phase before with a bounded wait (status word of the job's workspace on expiry);
 * the launch uses at most one thread block per multiprocessor, so all blocks are resident together. */
#define BITCOS_MAX_PHASES 4
#define BITCOS_PHASED_SYNC_BYTES 64
int bitcos_gemv_phased(const bitcos_gemv_job *jobs, const int *job_phase, int n_jobs, int batch, void *sync,
                       void *cuda_stream);

/* The same product as bitcos_gemv without a caller-provided workspace.  (The paper has no
 * counterpart: this entry point exists for the library's users, not for the method.)
 *
 * Who needs it: code that is not allowed to allocate device memory at the point where it
 * multiplies -- a serving loop whose memory was sized and handed out at start-up, a plug-in
 * that runs inside somebody else's memory pool, a latency-critical path where cudaMalloc's
 * implicit device-wide synchronisation is unacceptable.  The scratch bytes come from a fixed
 * array of BITCOS_STATIC_WORKSPACE_BYTES inside the library image; every device that loads the
 * library holds that array until the process exits.  The call allocates nothing and calls no
 * allocating routine; x, x_scale and y are still the caller's device buffers (as in
 * bitcos_gemv; acc_debug is not offered).
 *
 * Limits and rules
 *   - ERR_CAPACITY if bitcos_gemv_workspace_bytes(M, K) exceeds BITCOS_STATIC_WORKSPACE_BYTES
 *     (all shapes of the benchmark configurations fit).
 *   - The first call on a device looks the array's device address up (cudaGetSymbolAddress,
 *     with that device current) and keeps it; make that first call outside stream capture.
 *   - All calls on a device share the one array and it keeps the last call's contents: each
 *     call first clears the status word and the arrival counters on the given stream.  Two
 *     calls that may overlap on the GPU (different streams, no ordering between them) race on
 *     it: order them, or give one of them bitcos_gemv with its own workspace. */
#define BITCOS_STATIC_WORKSPACE_BYTES (8 * 1024 * 1024)
int bitcos_gemv_static(const bitcos_weights *W, const int8_t *x, const float *x_scale, int batch, float *y,
                       void *cuda_stream);
/* The status word of that array (as bitcos_workspace_status for a caller's workspace; waits for the
 * stream): 0 if the last bitcos_gemv_static call on this device completed normally.  Every
 * bitcos_gemv_static call clears the word before its kernel, so ask before the next call. */
int bitcos_gemv_static_status(void *cuda_stream, int *status);

/* Exercises the give-up path of the bounded waits without a fault (every wait inside the kernels is
 * bounded; Section II of the paper has no counterpart: this is the library's own safety net).  One warp
 * arms a barrier for bytes that no copy ever delivers, polls it with the kernels' own loop for limit_ns
 * nanoseconds (1 us .. 100 ms), then sets the status word of `workspace` (device, at least 4 bytes) to 1 and
 * returns normally, as a product whose copy never arrived would.  waited_ns: NULL or device uint64
 * receiving the time spent polling.  The context stays usable; bitcos_workspace_status reads the word. */
int bitcos_wait_probe(void *workspace, uint64_t limit_ns, uint64_t *waited_ns, void *cuda_stream);

/* Host-buffer form of bitcos_gemv for callers whose activations live in host memory: copies
 * x_host[batch][K] and x_scale_host[batch] into `staging`, runs bitcos_gemv, copies
 * y[batch][M] back to y_host and waits for the stream, so y_host is valid on return.  The
 * weights stay resident on the device.  Pinned host buffers make the copies asynchronous
 * until the final wait.  staging: device scratch of bitcos_gemv_host_staging_bytes bytes. */
size_t bitcos_gemv_host_staging_bytes(int64_t M, int64_t K, int batch);
int bitcos_gemv_host(const bitcos_weights *W, const int8_t *x_host, const float *x_scale_host, int batch,
                     float *y_host, void *staging, size_t staging_bytes, void *workspace,
                     size_t workspace_bytes, void *cuda_stream);

/* Host-buffer form of bitcos_gemv_multi: up to BITCOS_MAX_JOBS independent products whose
 * activations and results live in host memory, with ONE launch and ONE wait for all of them
 * (copies every job's x and x_scale into its staging buffer, runs bitcos_gemv_multi, copies every
 * y back, waits for the stream; all y_host are valid on return).  Per job: staging of
 * bitcos_gemv_host_staging_bytes(M, K, batch) bytes and a workspace of its own, as for
 * bitcos_gemv_host.  The paper has no counterpart (it measures resident activations). */
typedef struct bitcos_gemv_host_job {
    const bitcos_weights *W;    /* host struct of device pointers */
    const int8_t *x_host;       /* host int8 [batch][K] (pinned memory keeps the copies asynchronous) */
    const float *x_scale_host;  /* host float [batch] */
    float *y_host;              /* host float [batch][M] */
    void *staging;              /* device scratch */
    size_t staging_bytes;
    void *workspace;            /* device scratch, zero filled once */
    size_t workspace_bytes;
} bitcos_gemv_host_job;
int bitcos_gemv_multi_host(const bitcos_gemv_host_job *jobs, int n_jobs, int batch, void *cuda_stream);

/* A whole sequence of phases from host buffers with ONE copy in, ONE copy out and ONE wait: the
 * host-buffer form for callers that run several dependent products per step (a decoder layer's
 * q | k | v, o, gate | up, down) and keep activations and results on the host.  The caller lays every
 * job's x and x_scale out inside one device block `in_device` (and the same bytes, at the same
 * offsets, inside the host block `in_host`), and every job's y inside one device block
 * `out_device`; jobs[] holds the DEVICE addresses, as for bitcos_gemv_multi.  The call copies
 * in_host -> in_device (in_bytes), runs one launch per phase (job_phase as for bitcos_gemv_phased;
 * each launch is told its neighbours as by bitcos_gemv_multi_chained), copies out_device ->
 * out_host (out_bytes) and waits for the stream, so out_host is valid on return.  Pinned host
 * blocks keep the two copies asynchronous until the wait.
 * Replay: the second call with the same arguments (every pointer, size and descriptor field
 * compared by value) records the step as a CUDA graph on a stream of the library's own; that call and
 * the following ones launch the graph on `cuda_stream` (one driver call instead of six).  The record
 * holds the entry offsets its launch plans read from the descriptors' tile_off_host; every replay
 * compares them with the host arrays' current contents and falls back to enqueueing directly if
 * they differ, so matrices re-packed into the same buffers are handled; the packed arrays in device
 * memory are read when the kernels run and may change freely.  Up to 64 argument sets are kept
 * (least recently used replaced).  Pageable host blocks are never recorded.  Thread safe.
 * ERR_CAPACITY if a job's x, x_scale or y lies outside its block.  The paper has no counterpart (it
 * measures resident activations). */
int bitcos_gemv_phases_host(const bitcos_gemv_job *jobs, const int *job_phase, int n_jobs, int batch, const void *in_host,
                            void *in_device, size_t in_bytes, void *out_host, const void *out_device, size_t out_bytes,
                            void *cuda_stream);

/* The same product from the five-trit and 2-bit layouts (device pointers; scales in tile order). */
int trit5_gemv(const uint32_t *words, const uint16_t *scales_tiled, int64_t M, int64_t K, const int8_t *x,
               const float *x_scale, int batch, float *y, int32_t *acc_debug, void *workspace,
               size_t workspace_bytes, void *cuda_stream);
int bit2_gemv(const uint32_t *words, const uint16_t *scales_tiled, int64_t M, int64_t K, const int8_t *x,
              const float *x_scale, int batch, float *y, int32_t *acc_debug, void *workspace,
              size_t workspace_bytes, void *cuda_stream);

/* Grouped product over selected experts of a mixture-of-experts layer (all experts M x K).
 * The caller lists the P (token, expert) pairs grouped by expert: group i covers pairs
 * group_begin[i] .. group_begin[i+1]-1 (at most max_group_size <= 16 per group), all using expert
 * group_expert[i]; pair p reads activation row pair_xrow[p] of x[n_xrows][K] and writes y[p][M].
 * Each listed expert's packed bytes are read once.  No activation function, routing weight
 * or sum over experts is applied (the paper runs its mixture-of-experts checkpoints end to end only,
 * Table I; this is the per-expert product such a layer needs).
 *   experts       device array of bitcos_weights (device pointers inside), n_experts entries
 *   group_expert  device int32 [n_groups];  group_begin  device int32 [n_groups + 1]
 *   pair_xrow     device int32 [n_pairs];  x device int8 [n_xrows][K];  x_scale device float [n_xrows]
 *   y             device float [n_pairs][M];  acc_debug NULL or device int32 [n_pairs][M][K/128]
 *   workspace     at least n_groups * bitcos_gemv_workspace_bytes(M, K) bytes, zero filled once;
 *                 group i's status word is word 0 of workspace + i * bitcos_gemv_workspace_bytes(M, K)
 * The routing lists live in device memory (they may come from a router kernel) and are checked on
 * the device: a group whose pairs fall outside [0, n_pairs), that has more than max_group_size
 * pairs (rounded up to 1, 2, 4, 8 or 16), that names an expert outside [0, n_experts) or an
 * activation row outside [0, n_xrows) is skipped whole -- nothing of it is read or written -- and
 * its status word and word 0 of the workspace (what bitcos_workspace_status reads) are set to 2.
 * An empty group (group_begin[i+1] <= group_begin[i]) is skipped without a mark. */
int bitcos_gemv_grouped(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                        const int32_t *group_begin, int n_groups, const int32_t *pair_xrow, int n_pairs,
                        int max_group_size, const int8_t *x, int n_xrows, const float *x_scale, float *y,
                        int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Routing with every list on the device, for decode loops whose router runs on the GPU (the paper's
 * mixture-of-experts checkpoints, Table I, route per token; it gives no kernel for it).
 *
 * bitcos_group_pairs_device: the stable grouping by expert that the grouped products expect, done by
 * one small kernel on the caller's stream.  pair_expert / pair_xrow: device int32 [n_pairs]
 * (n_pairs <= BITCOS_GROUP_PAIRS_MAX, expert ids in [0, n_experts), n_experts <=
 * BITCOS_GROUP_EXPERTS_MAX).  Outputs (device): group_expert [min(n_pairs, n_experts)], group_begin
 * [min(n_pairs, n_experts) + 1], pair_xrow_sorted [n_pairs], order [n_pairs] (sorted pair i is input
 * pair order[i]: output row i of the grouped product belongs to it), n_groups [1].  Experts ascending,
 * input order kept inside a group.  A pair with an expert id out of range is left out.
 *
 * bitcos_gemv_grouped_lists: bitcos_gemv_grouped with the NUMBER of groups read from device memory
 * (n_groups_device, as bitcos_group_pairs_device wrote it; values above max_groups are clipped).
 * max_groups sizes the launch and the workspace (max_groups * bitcos_gemv_workspace_bytes(M, K)).
 * max_group_size is an upper bound the caller knows without the lists, e.g. the number of tokens when
 * every token picks distinct experts.  Everything else as for bitcos_gemv_grouped. */
#define BITCOS_GROUP_PAIRS_MAX 4096
#define BITCOS_GROUP_EXPERTS_MAX 1024
int bitcos_group_pairs_device(const int32_t *pair_expert, const int32_t *pair_xrow, int n_pairs, int n_experts,
                              int32_t *group_expert, int32_t *group_begin, int32_t *pair_xrow_sorted, int32_t *order,
                              int32_t *n_groups, void *cuda_stream);
int bitcos_gemv_grouped_lists(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                              const int32_t *group_begin, const int32_t *n_groups_device, int max_groups,
                              const int32_t *pair_xrow, int n_pairs, int max_group_size, const int8_t *x, int n_xrows,
                              const float *x_scale, float *y, int32_t *acc_debug, void *workspace, size_t workspace_bytes,
                              void *cuda_stream);

/* The same grouped product from five-trit and 2-bit experts, so that the layout's gain can be
 * measured on the same chip for the mixture-of-experts shapes too (Section II-A: below a zero
 * density of 0.375 the five-trit format is the smaller one).  experts[e].bitmap points to the packed
 * words (trit5_pack / bit2_pack layout), experts[e].scales to the scales in tile order; signs,
 * tile_off and tile_off_host are not used. */
int trit5_gemv_grouped(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                       const int32_t *group_begin, int n_groups, const int32_t *pair_xrow, int n_pairs,
                       int max_group_size, const int8_t *x, int n_xrows, const float *x_scale, float *y,
                       int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream);
int bit2_gemv_grouped(const bitcos_weights *experts, int n_experts, int64_t M, int64_t K, const int32_t *group_expert,
                      const int32_t *group_begin, int n_groups, const int32_t *pair_xrow, int n_pairs,
                      int max_group_size, const int8_t *x, int n_xrows, const float *x_scale, float *y,
                      int32_t *acc_debug, void *workspace, size_t workspace_bytes, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BITCOS_H */
