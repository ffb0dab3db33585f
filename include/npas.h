/*
 * npas.h - C ABI of the block-punched CONV / block-based GEMM library for NVIDIA B200 (sm_100a).
 *
 * The operations follow the two fine-grained structured pruning schemes of the NPAS paper
 * (Sec. 3, "Proposed Fine-Grained Structured Pruning"):
 *   block-punched pruning (CONV): the weight tensor is cut into blocks of Mb filters x Nb input
 *     channels and the same kernel positions ("taps") are pruned in every kernel of a block;
 *   block-based pruning (FC / 1x1 CONV): the weight matrix is cut into equal blocks and whole
 *     rows and/or columns are pruned inside each block.
 * The paper fixes the mask structure only; the packed format below is this library's own.
 *
 * General rules
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; *_host are HOST pointers.
 *     The library never allocates or frees device memory and keeps no pointer after return.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     the call returns without synchronising, except where stated.
 *   - Every function returns an npas_status.  Argument, shape, alignment and buffer-size errors
 *     are detected on the host before anything is launched.  Nothing aborts or traps.
 *   - Device pointers must be 16-byte aligned (NPAS_ERR_ALIGNMENT otherwise).
 *   - Layouts: activations NHWC, dense weights KRSC ([K][R][S][C]), GEMM operands row major
 *     (X[M][I], W[O][I], Y[M][O]).  bias is always float32.
 *   - Mask words: tap_mask[fb*nCB + cb] is a uint64 bitset, bit t = r*S + s set <=> tap (r,s) is
 *     KEPT in block (fb, cb); row_keep / col_keep [bo*nBi + bi] are bitsets of kept rows / cols.
 *   - Requirements: K % Mb == 0, C % Nb == 0, O % Bo == 0, I % Bi == 0, R*S <= 64, Bo, Bi <= 64,
 *     C, nCB < 65536 (NPAS_ERR_SHAPE otherwise).
 *
 * Packed formats (little endian; every section starts on a 128-byte boundary, padding is zero)
 *   Block-punched blob:
 *     header  32 x uint32: magic 'NPBP' (0x5042504E), version 4, dtype, K, C, R, S, Mb, Nb,
 *             nFB, nCB, nPairs, off_blk_off, off_pairs, off_values, total_bytes, G, off_image,
 *             off_tapu, GI, off_kt_off, off_kt, GS, nKt, zeros (G = channel-group width: 8 if
 *             Nb % 8 == 0, else Nb; GI = the largest power of two <= 128 that divides K)
 *     blk_off uint32[nFB*nCB+1]  exclusive prefix sum of kept-tap counts, blocks fb-major
 *     pairs   uint32[nPairs]     cb | tap << 16, block order, taps ascending within a block
 *     values  weight (pair j, filter f, channel c) at element ((j*(Nb/G) + c/G)*Mb + f)*G + c%G
 *     image   (bf16 blobs with C % 16 == 0 only, else off_image = 0) the masked dense weights as
 *             tensor-core operand tiles: weight (k, tap, c) at element
 *             (((((k/GI)*(C/16) + c/16)*R*S + tap)*2 + (c%16)/8)*GI + k%GI)*8 + c%8, pruned = +0
 *             (a compile-time expansion; blk_off / pairs / values stay the canonical content);
 *             the section starts on a multiple of 2048 bytes
 *     tapu    uint32[K/GI][C/16]: union of the kept-tap bitsets of the blocks that touch the
 *             (filter group, 16-channel chunk); all ones when R*S > 32
 *     kt_off, kt  (bf16 blobs with Mb % 16 == 0, Nb % 16 == 0, R*S <= 16 and Mb dividing FGW, the
 *             largest power of two <= 256 that divides K; else off_kt = 0)  the kept weights cut
 *             into tiles of Mb filters x 16 channels, ordered by (16-channel chunk, group of
 *             GS = FGW/Mb filter blocks, tap, filter block ascending; kept tiles only), so that
 *             what one filter group needs for one chunk is one contiguous run and the tiles of
 *             neighbouring filter blocks that keep the same tap are neighbours (one MMA can then
 *             cover several blocks).  kt_off uint32[(C/16)*(K/FGW) + 1]: exclusive prefix sum of
 *             the tile counts per (chunk, group), chunk major; nKt = nPairs * Nb/16.  Tile =
 *             [Mb/8 filter octets][2 channel octets][8 filters][8 channels], Mb*32 bytes
 *             (a compile-time expansion, like image)
 *   Block-based blob:
 *     header  32 x uint32: magic 'NPBB' (0x4242504E), version 3, dtype, O, I, Bo, Bi, nBo, nBi,
 *             nVals, off_cnt, off_rows, off_cols, off_val_off, off_values, total_bytes, Kp,
 *             off_tiles, off_dense, zeros (Kp = largest kept-column count of a block rounded up
 *             to 16, >= 16)
 *     cnt     uint8[nBlk][2]   kept rows, kept cols (blocks bo-major)
 *     rows    uint8[nBlk][Bo]  kept row indices ascending, unused = 0xFF
 *     cols    uint8[nBlk][Bi]  kept col indices ascending, unused = 0xFF
 *     val_off uint32[nBlk+1]   element offset of each block's values (multiples of 8)
 *     dense   the masked weight matrix [O][I], row major, pruned weights +0: the operand of the
 *             tensor-core kernel that reads both operands by TMA (compile-time expansion of the
 *             compact form; the compact sections stay the canonical content).  It sits before the
 *             values so that its offset follows from the descriptor alone.
 *     values  per block kept-rows x kept-cols, row major
 *     tiles   per block the same weights as a [Kp/8][Bo][8] tensor-core operand image: element
 *             (c/8, rows[r], c%8) = weight (rows[r], cols[c]); pruned rows and unused columns zero
 *   float32 -> bf16 conversion in the packers is round-to-nearest-even on the bit pattern
 *   (bits + 0x7FFF + ((bits >> 16) & 1)) >> 16; a NaN becomes (bits >> 16) | 0x40.
 */
#ifndef NPAS_H_
#define NPAS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NPAS_OK = 0,
    NPAS_ERR_NULL = 1,
    NPAS_ERR_SHAPE = 2,
    NPAS_ERR_DTYPE = 3,
    NPAS_ERR_ALIGNMENT = 4,
    NPAS_ERR_MASK_STRUCTURE = 5,
    NPAS_ERR_BLOB = 6,
    NPAS_ERR_BUFFER_TOO_SMALL = 7,
    NPAS_ERR_UNSUPPORTED = 8,
    NPAS_ERR_CUDA = 9,
    NPAS_ERR_TIMEOUT = 10
} npas_status;

typedef enum { NPAS_F32 = 0, NPAS_BF16 = 1 } npas_dtype;

/* Bytes of caller workspace every compute call needs (holds the device status words). */
#define NPAS_WORKSPACE_BYTES 256

/* Static, NUL-terminated description of a status code. */
const char *npas_status_string(npas_status s);
uint32_t npas_abi_version(void);

/* Weight tensor of a block-punched layer. w_in: dtype of the dense weights handed to the packer;
 * w_packed: dtype stored in the blob.  max_taps: an upper bound, promised by the caller, on the
 * number of kept taps of any single block (0 = no promise, i.e. R*S); the convolution sizes its
 * shared-memory weight buffers by it, and a blob that breaks the promise makes the call report
 * NPAS_ERR_BLOB through the device status words instead of computing. */
typedef struct {
    int32_t K, C, R, S, Mb, Nb;
    int32_t w_in, w_packed; /* npas_dtype */
    int32_t max_taps;
} npas_bp_desc;

/* Weight matrix of a block-based layer.  max_cols: the largest number of kept columns of any single
 * block, as the caller knows it from the masks (0 = unknown).  It fixes the width Kp of the blob's
 * tiles section; the tensor-core GEMM needs it (0 selects the CUDA-core kernel) and reports
 * NPAS_ERR_BLOB through the device status words when it does not match the blob. */
typedef struct {
    int32_t O, I, Bo, Bi;
    int32_t w_in, w_packed; /* npas_dtype */
    int32_t max_cols;
} npas_bb_desc;

/* One convolution call. x_dtype must equal the blob dtype; y_dtype may be f32 or (bf16 path) bf16.
 * path: 0 = automatic, 1 = force the CUDA-core kernel, 2 = automatic among the tcgen05 kernels,
 * 3 = force the tcgen05 kernel with both operands in shared memory, 5 = force the tcgen05 kernel
 * for three-channel 7x7 stride-2 first layers, 6 = force the tcgen05 kernel that multiplies the
 * blob's dense operand image, 7 = force the variant of that kernel that runs on CTA pairs
 * (cta_group::2; C % 64 == 0, K % 64 == 0), 8 = force the tcgen05 kernel that multiplies kept
 * (block, tap) pairs only (stride 1, Mb and Nb multiples of 16, at most 16 taps)
 * (NPAS_ERR_UNSUPPORTED when the geometry is outside the requested kernel's envelope). */
typedef struct {
    int32_t N, H, W, C, K, R, S, stride, pad;
    int32_t x_dtype, y_dtype;
    int32_t relu, has_bias, has_residual;
    int32_t path;
    int32_t variant; /* 0 = the kernel's own planner chooses its tile shape; path 7: NT + (MT << 16), NT =
                        64 (only when 128 does not divide K), 128 or 256 filters per item, MT = 1 or 2 position tiles per CTA (a combination the
                        geometry does not allow gives NPAS_ERR_UNSUPPORTED); other paths ignore it.
                        npas_tune_conv2d_bp measures the candidates and returns the best (path, variant). */
} npas_conv_desc;

/* One block-based GEMM call.  path: 0 = automatic, 1 = force the CUDA-core kernel, 2 = automatic
 * among the tcgen05 kernels, 3 = force the tcgen05 kernel that gathers the kept columns of X,
 * 5 = force the tcgen05 kernel that reads X and the blob's masked dense image by TMA, 6 = force
 * the variant of that kernel that runs on CTA pairs (cta_group::2; O a multiple of 128)
 * (NPAS_ERR_UNSUPPORTED when the geometry is outside the requested kernel's envelope). */
typedef struct {
    int32_t M, I, O;
    int32_t x_dtype, y_dtype;
    int32_t relu, has_bias, has_residual;
    int32_t path;
    int32_t variant; /* 0 = the planner's choice; paths 5 and 6: the column-tile width BN (a power of two
                        from 16 to 256 dividing O; path 6: 128 or 256); npas_tune_linear_bb measures them */
} npas_linear_desc;

/* ---- mask helpers (paper Sec. 3: the structural constraint of each scheme) --------------------
 * Derive block masks from a dense 0/1 mask (uint8 per weight, same layout as the weights).
 * *violations_dev (int32, device) receives the number of blocks whose support is NOT of the
 * scheme's form (taps shared by all kernels of the block / rows x cols product); the call
 * synchronises the stream and returns NPAS_ERR_MASK_STRUCTURE when it is non-zero. */
npas_status npas_mask_bp_from_dense(const npas_bp_desc *d, const uint8_t *dense_mask_dev,
                                    uint64_t *tap_mask_dev, int32_t *violations_dev, void *stream);
npas_status npas_mask_bb_from_dense(const npas_bb_desc *d, const uint8_t *dense_mask_dev,
                                    uint64_t *row_keep_dev, uint64_t *col_keep_dev,
                                    int32_t *violations_dev, void *stream);

/* ---- one-shot magnitude pruning (paper Sec. 5.2, "One-shot Pruning ... for Fast Accuracy
 * Evaluation": the layer is pruned once, by weight magnitude, under the candidate's scheme and
 * rate).  The paper does not define the grouping; here the score of a prunable group - one tap of
 * a block (block-punched), one row or one column of a block scored over the whole block
 * (block-based) - is the sum of the squares of its weights, accumulated in fp64 in the order
 * filters / rows outer, channels / columns inner; each block keeps its keep_* highest-scoring
 * groups, ties go to the lower index.  w_dense_dev is KRSC / [O][I] in d->w_in; the masks are the
 * bitsets the packers take ([K/Mb][C/Nb], [O/Bo][I/Bi], device). */
npas_status npas_prune_bp_magnitude(const npas_bp_desc *d, const void *w_dense_dev, int32_t keep_taps,
                                    uint64_t *tap_mask_dev, void *stream);
/* The same scoring with a layer-wide budget (the pruning rates of the paper's Table 1, e.g. 2.5x or 7x,
 * which no uniform per-block count expresses): of all G = (K/Mb)(C/Nb)(R*S) (block, tap) groups of the
 * layer the n_keep with the largest scores are kept, ties going to the lower group index (blocks
 * filter-block major, taps ascending), so blocks keep different numbers of taps; a rate r corresponds
 * to n_keep = round(G / r).  ws_dev: scratch of the size npas_prune_bp_global_workspace reports (the
 * fp64 scores of all groups), owned by the caller. */
npas_status npas_prune_bp_global_workspace(const npas_bp_desc *d, size_t *ws_bytes);
npas_status npas_prune_bp_magnitude_global(const npas_bp_desc *d, const void *w_dense_dev, int64_t n_keep,
                                           uint64_t *tap_mask_dev, void *ws_dev, size_t ws_bytes, void *stream);
npas_status npas_prune_bb_magnitude(const npas_bb_desc *d, const void *w_dense_dev, int32_t keep_rows,
                                    int32_t keep_cols, uint64_t *row_keep_dev, uint64_t *col_keep_dev,
                                    void *stream);

/* ---- packers (paper Sec. 3; format described at the top of this file) ------------------------
 * *_size: blob size in bytes for HOST masks.  pack: dense weights (dtype w_in, KRSC or [O][I])
 * + DEVICE masks -> blob of exactly the size the size call reports.  The size a blob needs
 * depends on the masks on the device, so the pack calls SYNCHRONISE the stream at their end and
 * return NPAS_ERR_BUFFER_TOO_SMALL when blob_bytes was less than that (such a blob is left with
 * magic 0 and all section offsets 0 and must not be used; word 15 of its header holds the size
 * that would have been needed).
 * unpack: blob -> dense zero-filled masked weights in the blob's dtype + the block masks
 * (either output may be NULL).  unpack(pack(W, mask)) == W (.) mask bit for bit. */
npas_status npas_pack_bp_size(const npas_bp_desc *d, const uint64_t *tap_mask_host, size_t *blob_bytes);
npas_status npas_pack_bp(const npas_bp_desc *d, const void *w_dense_dev, const uint64_t *tap_mask_dev,
                         void *blob_dev, size_t blob_bytes, void *stream);
npas_status npas_unpack_bp(const npas_bp_desc *d, const void *blob_dev, size_t blob_bytes,
                           void *w_dense_out_dev, uint64_t *tap_mask_out_dev, void *stream);
npas_status npas_pack_bb_size(const npas_bb_desc *d, const uint64_t *row_keep_host,
                              const uint64_t *col_keep_host, size_t *blob_bytes);
npas_status npas_pack_bb(const npas_bb_desc *d, const void *w_dense_dev, const uint64_t *row_keep_dev,
                         const uint64_t *col_keep_dev, void *blob_dev, size_t blob_bytes, void *stream);
npas_status npas_unpack_bb(const npas_bb_desc *d, const void *blob_dev, size_t blob_bytes,
                           void *w_dense_out_dev, uint64_t *row_keep_out_dev,
                           uint64_t *col_keep_out_dev, void *stream);

/* ---- compute ---------------------------------------------------------------------------------
 * npas_conv2d_bp: block-punched convolution (paper Sec. 3) with the fused epilogue
 *   Y[n,p,q,k] = act(bias[k] + sum over kept (r,s,c) of W[k,r,s,c] * Xpad[n, p*stride+r-pad,
 *                q*stride+s-pad, c] (+ residual[n,p,q,k])),  act = ReLU when relu != 0.
 *   x [N,H,W,C] and y/residual [N,P,Q,K] are NHWC in x_dtype / y_dtype; accumulation is fp32.
 *   `bp` must describe the blob at blob_dev (the header on device is trusted to match it; use
 *   npas_blob_check to verify a blob of unknown origin).  y must not alias x.
 *   ws_dev: NPAS_WORKSPACE_BYTES of device scratch, zeroed once by the caller before first use;
 *   a kernel whose bounded waits expire records NPAS_ERR_TIMEOUT there (npas_check_device_status).
 * npas_linear_bb: block-based pruned GEMM
 *   Y[m,o] = act(bias[o] + sum over kept i of X[m,i] W[o,i] (+ residual[m,o])); residual [M,O] in
 *   y_dtype, may not alias y.
 * npas_subsample2d: Y[n,p,q,c] = X[n, p*stride, q*stride, c] (NHWC, 2- or 4-byte elements given by
 *   elem_bytes): the input of a strided 1x1 convolution run as a GEMM. */
npas_status npas_conv2d_bp(const npas_conv_desc *d, const npas_bp_desc *bp, const void *x_dev,
                           const void *blob_dev, const float *bias_dev, const void *residual_dev,
                           void *y_dev, void *ws_dev, size_t ws_bytes, void *stream);
/* npas_conv2d_bp_maxpool: convolution + bias + ReLU + max-pool in one kernel (layer fusion, paper Sec. 3
 * "Compiler Optimizations"; Sec. 4 on the memory traffic of intermediate results): y_pooled_dev
 * [N, P', Q', K] = max over the pool_r x pool_r window (stride pool_stride, padding pool_pad that never
 * wins) of the convolution output, which is never written.  The result is bit for bit that of
 * npas_conv2d_bp followed by npas_maxpool2d.  Fused today: three-channel 7x7 stride-2 first layers
 * (path 5's envelope) with ReLU, bf16 output, no residual, and the 3x3 / stride-2 / pad-1 window;
 * any other combination returns NPAS_ERR_UNSUPPORTED and the caller issues the two calls.  The call
 * clears y_pooled_dev on `stream` before the kernel. */
npas_status npas_conv2d_bp_maxpool(const npas_conv_desc *d, const npas_bp_desc *bp, int32_t pool_r,
                                   int32_t pool_stride, int32_t pool_pad, const void *x_dev, const void *blob_dev,
                                   const float *bias_dev, void *y_pooled_dev, void *ws_dev, size_t ws_bytes,
                                   void *stream);

/* Which kernel the call would run (the value `path` takes to force it): convolution 1 = CUDA cores,
 * 3 = tcgen05 with both operands in shared memory, 5 = three-channel first layer, 6 = the blob's dense
 * operand image, 7 = the same on CTA pairs, 8 = kept (block, tap) pairs only; GEMM 1 = CUDA cores,
 * 3 = gathered kept columns, 5 = the blob's masked dense image by TMA, 6 = the same on CTA pairs.
 * Host only, nothing is launched; NPAS_ERR_UNSUPPORTED when the requested path declines the geometry. */
npas_status npas_conv2d_bp_kernel(const npas_conv_desc *d, const npas_bp_desc *bp, int32_t *kernel_id);
npas_status npas_linear_bb_kernel(const npas_linear_desc *d, const npas_bb_desc *bb, int32_t *kernel_id);

/* Auto-tuning (paper Sec. 3, "Compiler Optimizations": the generated code is tuned per layer).  Runs
 * every kernel and tile shape that takes the layer on the caller's own buffers (one warm-up and `reps`
 * timed launches each, CUDA events on `stream`), and returns the fastest as the (path, variant) pair to
 * put into the call descriptor; *us_out (nullable) receives its time per launch in microseconds.  The
 * plan is these two integers: the caller keeps them with the layer.  Synchronises the stream several
 * times (not for use inside a stream capture); y_dev holds the layer's result afterwards.  d->path and
 * d->variant are ignored.  Arguments as in the compute calls. */
npas_status npas_tune_conv2d_bp(const npas_conv_desc *d, const npas_bp_desc *bp, const void *x_dev,
                                const void *blob_dev, const float *bias_dev, const void *residual_dev,
                                void *y_dev, void *ws_dev, size_t ws_bytes, int32_t reps, int32_t *path_out,
                                int32_t *variant_out, float *us_out, void *stream);
npas_status npas_tune_linear_bb(const npas_linear_desc *d, const npas_bb_desc *bb, const void *x_dev,
                                const void *blob_dev, const float *bias_dev, const void *residual_dev,
                                void *y_dev, void *ws_dev, size_t ws_bytes, int32_t reps, int32_t *path_out,
                                int32_t *variant_out, float *us_out, void *stream);

/* Bytes of device scratch (ws_dev) the matching compute call needs for this layer.  Today every
 * kernel needs only the status words (NPAS_WORKSPACE_BYTES); callers that size their workspace
 * through these calls keep working if a later kernel needs global scratch. */
npas_status npas_conv2d_bp_workspace(const npas_conv_desc *d, const npas_bp_desc *bp, size_t *ws_bytes);
npas_status npas_linear_bb_workspace(const npas_linear_desc *d, const npas_bb_desc *bb, size_t *ws_bytes);
npas_status npas_linear_bb(const npas_linear_desc *d, const npas_bb_desc *bb, const void *x_dev,
                           const void *blob_dev, const float *bias_dev, const void *residual_dev,
                           void *y_dev, void *ws_dev, size_t ws_bytes, void *stream);
npas_status npas_subsample2d(int32_t N, int32_t H, int32_t W, int32_t C, int32_t stride,
                             int32_t elem_bytes, const void *x_dev, void *y_dev, void *stream);

/* npas_conv2d_bp_static_ws (the paper has no counterpart: this entry exists for callers that must
 * not allocate).  Some callers cannot obtain device memory at the point where they run a layer:
 * code inside a real-time or fixed-memory-budget inference loop, plug-ins living in a host
 * application that owns every allocation, or code running where cudaMalloc would synchronise or
 * is simply forbidden.  They still own x, the blob, bias, residual and y, but cannot provide the
 * NPAS_WORKSPACE_BYTES of scratch that npas_conv2d_bp wants.  This variant computes exactly what
 * npas_conv2d_bp computes and keeps that scratch in a 256-byte array that is part of the library
 * image on every GPU that loads it (held until the process exits).  It calls no cudaMalloc,
 * cudaFree or any allocating routine.
 *   - The scratch need of a call is 256 bytes whatever the layer shape, which is also the
 *     array's size; a build whose kernels needed more would return NPAS_ERR_BUFFER_TOO_SMALL.
 *     All other arguments are validated exactly as in npas_conv2d_bp.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call clears it on `stream` before the
 *     launch, so nothing carries over from the previous call; two calls whose work overlaps on
 *     the GPU (different streams) race on it and may lose or misreport a time-out status.
 *   - `stream` must belong to the device that is current when the call is made (the array's address
 *     is looked up for the current device).
 *   - device_status_host (nullable, HOST): when given, the call synchronises `stream`, stores the
 *     device status word there (0 = fine) and returns what the kernel recorded: NPAS_ERR_TIMEOUT if
 *     a bounded wait expired, NPAS_ERR_BLOB if the blob contradicts its descriptor; when NULL the
 *     call stays asynchronous and such a device-side error goes unreported. */
npas_status npas_conv2d_bp_static_ws(const npas_conv_desc *d, const npas_bp_desc *bp, const void *x_dev,
                                     const void *blob_dev, const float *bias_dev,
                                     const void *residual_dev, void *y_dev,
                                     int32_t *device_status_host, void *stream);

/* Copies the blob header from the device (synchronises the stream) and checks magic, version,
 * sizes and section offsets against the descriptor.  Exactly one of bp / bb is non-NULL. */
npas_status npas_blob_check(const npas_bp_desc *bp, const npas_bb_desc *bb, const void *blob_dev,
                            size_t blob_bytes, void *stream);

/* Synchronises the stream, reads the status words in ws_dev, clears them, and returns NPAS_OK or
 * the recorded error (NPAS_ERR_TIMEOUT or NPAS_ERR_BLOB); *detail (nullable, host) receives an
 * implementation-defined location code. */
npas_status npas_check_device_status(void *ws_dev, void *stream, int32_t *detail);

/* Number of kernels this library has launched in the calling process (monotonic counter). */
uint64_t npas_launch_count(void);

/* Dense helpers for a full network stack (not pruned; paper Sec. 6 evaluates whole networks):
 * npas_maxpool2d: NHWC bf16 max pooling R x R, given stride and zero... padding that never wins
 * (positions outside the image are skipped). */
npas_status npas_maxpool2d(int32_t N, int32_t H, int32_t W, int32_t C, int32_t R, int32_t stride,
                           int32_t pad, const void *x_dev, void *y_dev, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* NPAS_H_ */
