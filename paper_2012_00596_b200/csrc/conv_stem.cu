// Few-channel first layer (7x7, stride 2, pad 3, C = 3) on the sm_100a tensor cores.
//
// With three channels the operand of a kept (channel block, tap) pair is only three elements wide,
// far below the tensor core's K = 16, so the generic block-punched kernels leave this layer to the
// CUDA cores.  Here the K dimension is built from a whole kernel row instead: in NHWC with C = 3
// the seven taps of one kernel row are 21 consecutive elements of an input row, starting (in
// coordinates padded by three pixels) at element 6q for output column q, i.e. at a 4-byte
// boundary.  Each of the seven kernel rows contributes a window of 24 elements (21 + 3 that meet
// zero weights), K = 7 * 24 = 168, padded to 176 = 11 MMA steps.  The weights come from the same
// block-punched blob as everywhere else (one channel block of Nb = 3): taps a block does not keep
// stay zero, so punched first layers work as well as the dense one.
//
// A CTA walks tiles of 128 consecutive output pixels of one image: (1) the input rows under the
// tile are copied to shared memory with the zero border in place (by bulk copies requested one tile
// ahead when a row is a multiple of 16 bytes, else by loads), (2) 256 threads expand them into
// the K-major operand (im2col in shared memory only), (3) one thread issues 11 MMAs of
// M = 128, N = K filters into TMEM, (4) the epilogue adds bias, applies ReLU and stores NHWC.
//
// Fused 3x3 / stride-2 / pad-1 max-pool (layer fusion, paper Sec. 3 "Compiler Optimizations"): instead
// of storing the convolution's output, the epilogue folds every pixel into the one, two or four pooled
// pixels whose window contains it, with vector max-reductions on packed bf16 pairs in global memory
// (resolved in L2).  After ReLU no value is negative, so the pooled tensor starts as zeros (cleared on
// the stream by the launcher); a maximum is exact and order independent, so the result is bit for bit
// the pooling of the rounded convolution output, which is then never written.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kGatherThreads = 256;
constexpr int kThreads = kGatherThreads + 32;
constexpr int kRows = 128;
constexpr int kR = 7, kC = 3, kWin = 24;          // window of one kernel row: 21 elements + 3
constexpr int kKK = 176, kOct = kKK / 8;           // padded K and its octets
constexpr int kRowBatch = 6;                       // input rows whose loads are in flight together
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kDescHi = (128u >> 4) | (1u << 14);   // SBO = 128 bytes, descriptor version bit

struct StemParams {
    int N, H, W, K, P, Q, Mb;
    int tiles_per_img, n_tiles, pitch_w, max_in_rows;
    int relu, y_bf16;
    int pool, PP, PQ;                                  // fused max-pool: pooled height and width
    int bulk_rows;                                     // input rows arrive by bulk copies, a tile ahead (W * 6 bytes % 16 == 0)
    uint32_t pitch_b, off_rows2, off_zero;             // bulk path: row pitch in bytes, the two row buffers, a row of zeros
    uint32_t off_b, off_a, off_rows, off_bias, off_bar, smem_bytes, tmem_cols;
};

struct StemBars {
    uint64_t done;
    uint64_t rows_full[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    return cvt_bf16x2(lo, hi);
}
// elementwise max of four packed bf16 pairs into global memory (no return value; NaNs are ignored)
__device__ __forceinline__ void red_max_bf16x8(void *addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("red.global.v4.bf16x2.max.noftz [%0], {%1, %2, %3, %4};" ::"l"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint64_t desc64(uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; }
__device__ __forceinline__ void gather_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

template <bool kPool>
__global__ void __launch_bounds__(kThreads, 2)     // two CTAs per SM hide each other's load latency
conv_stem_kernel(const StemParams p, const uint16_t *__restrict__ x, const uint8_t *__restrict__ blob,
                 const float *__restrict__ bias, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *bsm = smem + p.off_b;                    // [kOct][K filters][8] bf16
    uint8_t *asm_ = smem + p.off_a;                   // [kOct][128 pixels][8] bf16
    uint32_t *rows = reinterpret_cast<uint32_t *>(smem + p.off_rows);   // [max_in_rows][pitch_w] words
    float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);
    StemBars *bars = reinterpret_cast<StemBars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_BLK]);
    const uint32_t *pairs = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
    const uint16_t *values = reinterpret_cast<const uint16_t *>(blob + hdr[BP_OFF_VALUES]);

    if (tid == 0) {
        mbar_init(&bars->done, 1);
        mbar_init(&bars->rows_full[0], 1);
        mbar_init(&bars->rows_full[1], 1);
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == kGatherThreads / 32) tmem_alloc(&bars->tmem_base, p.tmem_cols);
    // weights: zero everything, then place every kept (tap, filter, channel) value at
    // k = r * 24 + s * 3 + c; the last octet of the activation operand is zero for good
    for (uint32_t o = tid * 16; o < (uint32_t)kOct * p.K * 16; o += kThreads * 16) *reinterpret_cast<uint4 *>(bsm + o) = make_uint4(0, 0, 0, 0);
    for (uint32_t o = tid * 16; o < (uint32_t)kRows * 16; o += kThreads * 16)
        *reinterpret_cast<uint4 *>(asm_ + (size_t)(kOct - 1) * kRows * 16 + o) = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < p.K; i += kThreads) bias_s[i] = bias ? bias[i] : 0.f;
    if (p.bulk_rows)                                   // borders of the row buffers and the zero row, once
        for (uint32_t o = p.off_rows2 + tid * 16; o < p.off_zero + p.pitch_b; o += kThreads * 16)
            *reinterpret_cast<uint4 *>(smem + o) = make_uint4(0, 0, 0, 0);
    __syncthreads();
    {
        const int nFB = p.K / p.Mb, per_pair = p.Mb * kC;
        for (int fb = 0; fb < nFB; ++fb) {
            const uint32_t lo = blk_off[fb], hi = blk_off[fb + 1];          // one channel block per filter block
            for (uint32_t e = tid; e < (hi - lo) * per_pair; e += kThreads) {
                const uint32_t j = lo + e / per_pair, rem = e % per_pair, f = rem / kC, c = rem % kC;
                const uint32_t tap = pairs[j] >> 16, r = tap / kR, s = tap % kR;
                if (r >= (uint32_t)kR) continue;                            // not a 7x7 tap: ignored
                const uint32_t kk = r * kWin + s * kC + c, n = fb * p.Mb + f;
                *reinterpret_cast<uint16_t *>(bsm + ((size_t)(kk >> 3) * p.K + n) * 16 + (kk & 7) * 2) = values[(size_t)j * per_pair + rem];
            }
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    const int PQ = p.P * p.Q;
    const int words_in = 3 * p.W / 2;                  // 32-bit words of one input row (W is even)
    // Bulk path: the MMA warp requests the input rows of a tile one tile ahead, one bulk copy per row
    // (lane u takes row u) into the buffer the tile before last has finished with; a row lands 32 bytes
    // into its slot, between zero borders; rows outside the image are not requested (the expansion reads
    // the zero row instead).
    auto request_rows = [&](int tile, uint32_t buf) {
        const int n = tile / p.tiles_per_img, t0 = (tile - n * p.tiles_per_img) * kRows;
        const int p0 = t0 / p.Q, p1 = min(PQ - 1, t0 + kRows - 1) / p.Q;
        const int y_lo = 2 * p0 - 3, nrows = 2 * (p1 - p0) + kR;
        const uint32_t row_bytes = (uint32_t)p.W * 6u;
        if (lane == 0) {
            const int lo = max(y_lo, 0), hi = min(y_lo + nrows, p.H);
            fence_proxy_async_smem();                  // the buffer was read by the expansion two tiles ago
            mbar_arrive_expect_tx(&bars->rows_full[buf], (uint32_t)(hi - lo) * row_bytes);
        }
        __syncwarp();
        for (int u = lane; u < nrows; u += 32) {
            const int yy = y_lo + u;
            if (yy >= 0 && yy < p.H)
                bulk_load_1d(smem + p.off_rows2 + ((size_t)buf * p.max_in_rows + u) * p.pitch_b + 32,
                             reinterpret_cast<const uint8_t *>(x) + ((size_t)n * p.H + yy) * row_bytes, row_bytes,
                             &bars->rows_full[buf]);
        }
    };
    bool ok = true;
    uint32_t it = 0;
    if (p.bulk_rows && warp == kGatherThreads / 32 && (int)blockIdx.x < p.n_tiles) request_rows(blockIdx.x, 0u);
    for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++it) {
        const int n = tile / p.tiles_per_img, t0 = (tile - n * p.tiles_per_img) * kRows;
        const int p0 = t0 / p.Q, p1 = min(PQ - 1, t0 + kRows - 1) / p.Q;
        const int y_lo = 2 * p0 - 3, nrows = 2 * (p1 - p0) + kR;
        if (p.bulk_rows && warp == kGatherThreads / 32 && tile + (int)gridDim.x < p.n_tiles)
            request_rows(tile + gridDim.x, (it + 1u) & 1u);
        if (p.bulk_rows && warp < kGatherThreads / 32) {
            // (1+2) the rows are there (requested a tile ago); expand: pixel m, kernel row r -> 24 elements, which
            // start two bytes into a word of the row: thirteen words, funnel-shifted
            if (!mbar_wait(&bars->rows_full[it & 1u], (it >> 1) & 1u, abort_flag, ws, 0x4200)) ok = false;
            const int m = tid & (kRows - 1), t = t0 + m;
            if (ok && t < PQ) {
                const int pp = t / p.Q, q = t - pp * p.Q;
                const uint8_t *buf = smem + p.off_rows2 + (size_t)(it & 1u) * p.max_in_rows * p.pitch_b;
#pragma unroll 2
                for (int r = tid >> 7; r < kR; r += 2) {
                    const int i = 2 * (pp - p0) + r, yy = y_lo + i;
                    const uint32_t *src = reinterpret_cast<const uint32_t *>(
                        ((yy >= 0 && yy < p.H) ? buf + (size_t)i * p.pitch_b : smem + p.off_zero)) + 3 * q + 3;
                    uint32_t w13[13], v[12];
#pragma unroll
                    for (int k = 0; k < 13; ++k) w13[k] = src[k];
#pragma unroll
                    for (int k = 0; k < 12; ++k) v[k] = (w13[k] >> 16) | (w13[k + 1] << 16);
#pragma unroll
                    for (int j = 0; j < 3; ++j)
                        *reinterpret_cast<uint4 *>(asm_ + ((size_t)(r * 3 + j) * kRows + m) * 16) =
                            make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                }
            }
            fence_proxy_async_smem();
        } else if (warp < kGatherThreads / 32) {
            // (1) input rows y_lo .. y_lo + nrows - 1, shifted right by the 9 elements of the left border:
            // shared word w holds input elements 2w - 9 and 2w - 8
            // (kRowBatch rows per trip, all loads of a trip issued before the first store)
            const uint32_t *xin = reinterpret_cast<const uint32_t *>(x) + (size_t)n * p.H * words_in;
            for (int i0 = 0; i0 < nrows; i0 += kRowBatch) {
                for (int w = tid; w < p.pitch_w; w += kGatherThreads) {
                    const int g0 = w - 5, g1 = w - 4;
                    const bool in0 = g0 >= 0 && g0 < words_in, in1 = g1 >= 0 && g1 < words_in;
                    uint32_t a[kRowBatch], b[kRowBatch];
#pragma unroll
                    for (int u = 0; u < kRowBatch; ++u) {
                        const int yy = y_lo + i0 + u;
                        const bool row_in = i0 + u < nrows && yy >= 0 && yy < p.H;
                        const uint32_t *row = xin + (size_t)(row_in ? yy : 0) * words_in;
                        a[u] = (row_in && in0) ? __ldg(row + g0) : 0u;
                        b[u] = (row_in && in1) ? __ldg(row + g1) : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < kRowBatch; ++u)
                        if (i0 + u < nrows) rows[(size_t)(i0 + u) * p.pitch_w + w] = (a[u] >> 16) | (b[u] << 16);
                }
            }
            gather_sync();
            // (2) expand: pixel m, kernel row r -> 24 elements = three operand rows of 16 bytes
            const int m = tid & (kRows - 1), t = t0 + m;
            if (t < PQ) {
                const int pp = t / p.Q, q = t - pp * p.Q;
#pragma unroll 2
                for (int r = tid >> 7; r < kR; r += 2) {
                    const uint32_t *src = rows + (size_t)(2 * (pp - p0) + r) * p.pitch_w + 3 * q;
                    uint32_t v[12];
#pragma unroll
                    for (int k = 0; k < 12; ++k) v[k] = src[k];
#pragma unroll
                    for (int j = 0; j < 3; ++j)
                        *reinterpret_cast<uint4 *>(asm_ + ((size_t)(r * 3 + j) * kRows + m) * 16) =
                            make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                }
            }
            fence_proxy_async_smem();
        }
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        if (warp == kGatherThreads / 32) {
            // (3) D[128 x K] = A[128 x 176] * B[K x 176]^T
            if (elect_one()) {
                const uint32_t idesc = idesc_bf16_f32(128, p.K);
                const uint32_t a_lo = (smem_u32(asm_) >> 4) | ((uint32_t)kRows << 16);      // K octets 128 * 16 bytes apart
                const uint32_t b_lo = (smem_u32(bsm) >> 4) | ((uint32_t)p.K << 16);
                for (int s = 0; s < kKK / 16; ++s)
                    mma_bf16_ss(tmem_base, desc64(a_lo + s * 2 * kRows), desc64(b_lo + s * 2 * p.K), idesc, s > 0 ? 1u : 0u);
                mma_commit(&bars->done);
            }
            __syncwarp();
        } else {
            // (4) epilogue once the MMAs have landed
            if (!mbar_wait(&bars->done, it & 1u, abort_flag, ws, 0x4100)) ok = false;
            tc_fence_after_sync();
            const int quarter = warp & 3, half = warp >> 2, m = quarter * 32 + lane, t = t0 + m;
            const size_t o0 = ((size_t)n * PQ + t) * p.K;
            // fused pooling: conv pixel (cp, cq) lies in pooled rows cp / 2 and, when cp is odd, cp / 2 + 1
            const int cp = t / p.Q, cq = t - cp * p.Q;
            const int pr0 = cp >> 1, pq0 = cq >> 1;
            const int npr = ((cp & 1) && pr0 + 1 < p.PP) ? 2 : 1;
            // Pooling along the row happens in registers first: lanes hold consecutive pixels, so a pixel in an
            // even column takes in its two neighbours (where they are in the same warp and row) and issues the
            // one reduction for its pooled column; a pixel in an odd column issues its own only towards a
            // neighbour that could not take it in.  This cuts the reductions to a third.
            const bool left_ok = lane > 0 && cq > 0, right_ok = lane < 31 && cq + 1 < p.Q && t + 1 < PQ;
            const bool even = (cq & 1) == 0;
            if (ok) {
                for (int c0 = half * 16; c0 < p.K; c0 += 32) {
                    uint32_t r[16];
                    __syncwarp();
                    tmem_ld_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + c0, r);
                    tmem_ld_wait();
                    if (t >= PQ && !kPool) continue;
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) + bias_s[c0 + i];
                    if (p.relu) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
                    }
                    if constexpr (kPool) {
                        uint32_t q[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) q[i] = pack2(v[2 * i], v[2 * i + 1]);
                        uint32_t mx[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {                      // every lane takes part in the exchanges
                            const uint32_t l = __shfl_up_sync(0xFFFFFFFFu, q[i], 1), rr = __shfl_down_sync(0xFFFFFFFFu, q[i], 1);
                            mx[i] = max_bf16x2(q[i], max_bf16x2(left_ok ? l : q[i], right_ok ? rr : q[i]));
                        }
                        if (t >= PQ) continue;
                        for (int dr = 0; dr < npr; ++dr) {
                            uint16_t *row = static_cast<uint16_t *>(y) + (((size_t)n * p.PP + pr0 + dr) * p.PQ) * p.K + c0;
                            if (even) {
                                red_max_bf16x8(row + (size_t)pq0 * p.K, mx[0], mx[1], mx[2], mx[3]);
                                red_max_bf16x8(row + (size_t)pq0 * p.K + 8, mx[4], mx[5], mx[6], mx[7]);
                            } else {
                                if (!left_ok) {
                                    red_max_bf16x8(row + (size_t)pq0 * p.K, q[0], q[1], q[2], q[3]);
                                    red_max_bf16x8(row + (size_t)pq0 * p.K + 8, q[4], q[5], q[6], q[7]);
                                }
                                if (!right_ok && pq0 + 1 < p.PQ) {
                                    red_max_bf16x8(row + (size_t)(pq0 + 1) * p.K, q[0], q[1], q[2], q[3]);
                                    red_max_bf16x8(row + (size_t)(pq0 + 1) * p.K + 8, q[4], q[5], q[6], q[7]);
                                }
                            }
                        }
                    } else if (p.y_bf16) {
                        uint4 *yp = reinterpret_cast<uint4 *>(static_cast<uint16_t *>(y) + o0 + c0);
                        yp[0] = make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
                        yp[1] = make_uint4(pack2(v[8], v[9]), pack2(v[10], v[11]), pack2(v[12], v[13]), pack2(v[14], v[15]));
                    } else {
                        float4 *yp = reinterpret_cast<float4 *>(static_cast<float *>(y) + o0 + c0);
#pragma unroll
                        for (int h = 0; h < 4; ++h) yp[h] = make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]);
                    }
                }
            }
        }
        ok = ok && !*abort_flag;
        // the next tile overwrites the staged rows, the operand and the accumulators
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        ok = ok && !*abort_flag;
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kGatherThreads / 32) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

bool plan(const npas_conv_desc &d, const npas_bp_desc &bp, StemParams &p, bool pool = false)
{
    if (d.x_dtype != NPAS_BF16 || bp.w_packed != NPAS_BF16) return false;
    if (d.C != kC || bp.Nb != kC || d.R != kR || d.S != kR || d.stride != 2 || d.pad != 3) return false;
    if (d.has_residual || d.K % 16 || d.K > 256 || d.K % bp.Mb || d.W % 2) return false;
    p.N = d.N; p.H = d.H; p.W = d.W; p.K = d.K; p.Mb = bp.Mb;
    p.P = (d.H + 2 * d.pad - d.R) / 2 + 1; p.Q = (d.W + 2 * d.pad - d.S) / 2 + 1;
    if (p.P < 1 || p.Q < 1) return false;
    p.tiles_per_img = (p.P * p.Q + kRows - 1) / kRows;
    p.n_tiles = d.N * p.tiles_per_img;
    // padded row: 9 + 3W + 9 elements, and the last window reads 3 elements further
    p.pitch_w = (3 * (d.W + 6) + 6 + 1) / 2;
    const int span = (p.Q - 1 + kRows - 1) / p.Q + 1;          // output rows a tile can touch
    p.max_in_rows = 2 * (span - 1) + kR;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    // the fused pooling needs non-negative bf16 values (ReLU) and 16-byte aligned groups of eight filters
    p.pool = pool ? 1 : 0;
    p.PP = (p.P - 1) / 2 + 1; p.PQ = (p.Q - 1) / 2 + 1;
    if (pool && (!d.relu || !p.y_bf16)) return false;
    p.off_b = 0;
    p.off_a = round_up((uint32_t)kOct * p.K * 16, 1024);
    p.off_rows = p.off_a + (uint32_t)kOct * kRows * 16;
    p.bulk_rows = (d.W * 6) % 16 == 0;
    p.pitch_b = round_up(32u + (uint32_t)d.W * 6u + 32u, 16);      // 16 elements of border on either side
    p.off_rows2 = p.off_rows;                                       // the bulk path replaces the single row buffer
    p.off_zero = p.off_rows2 + 2u * p.max_in_rows * p.pitch_b;
    const uint32_t rows_end = p.bulk_rows ? p.off_zero + p.pitch_b : p.off_rows + (uint32_t)p.max_in_rows * p.pitch_w * 4;
    p.off_bias = round_up(rows_end, 16);
    p.off_bar = round_up(p.off_bias + p.K * 4, 128);
    p.smem_bytes = p.off_bar + sizeof(StemBars) + 1024;
    if (p.smem_bytes > kSmemLimit) return false;
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < p.K) p.tmem_cols *= 2;
    return true;
}

}  // namespace

bool conv_stem_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    StemParams p;
    return plan(d, bp, p);
}

bool conv_stem_pool_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    StemParams p;
    return plan(d, bp, p, true);
}

npas_status conv_stem_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                             const void *blob, const float *bias, void *y, uint32_t *ws, cudaStream_t st, bool pool)
{
    StemParams p;
    if (!plan(d, bp, p, pool)) return NPAS_ERR_UNSUPPORTED;
    // the pooled tensor is built by max-reductions: it starts as zeros (no value is negative after ReLU)
    if (pool && cudaMemsetAsync(y, 0, (size_t)d.N * p.PP * p.PQ * d.K * 2u, st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (allow_dynamic_smem(pool ? reinterpret_cast<const void *>(conv_stem_kernel<true>) : reinterpret_cast<const void *>(conv_stem_kernel<false>),
                           (int)kSmemLimit) != NPAS_OK)
        return NPAS_ERR_CUDA;
    const int sms = sm_count();
    const int slots = (p.smem_bytes <= 110 * 1024 && p.tmem_cols <= 256) ? 2 * sms : sms;
    const int grid = p.n_tiles < slots ? p.n_tiles : slots;
    if (pool)
        conv_stem_kernel<true><<<grid, kThreads, p.smem_bytes, st>>>(p, static_cast<const uint16_t *>(x),
                                                                     static_cast<const uint8_t *>(blob), bias, y, ws);
    else
        conv_stem_kernel<false><<<grid, kThreads, p.smem_bytes, st>>>(p, static_cast<const uint16_t *>(x),
                                                                      static_cast<const uint8_t *>(blob), bias, y, ws);
    count_launch();
    return launch_status();
}

}  // namespace npas
