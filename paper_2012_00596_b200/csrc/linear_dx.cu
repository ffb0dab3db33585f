// Block-based pruned GEMM on the sm_100a tensor cores, zero-expanded weight tiles.
//
// The tensor core reads its operands in units of eight K elements, so kept columns scattered over
// a 64-wide block cannot be skipped by an operand descriptor: compacting them costs a gather of X
// through shared memory whose traffic equals (for four row blocks of 16 kept columns each) that of
// the whole 64-column X tile.  This kernel therefore keeps X as it is in memory and expands the
// weights instead: per column block bi, the BOG row blocks of the CTA are written into one
// [BOG * Bo rows] x [Bi = 64 columns] tile in shared memory, zeros where a row or a column is
// pruned, kept values at (rows[jr], cols[jc]).  Only the compact values and the index lists are
// read from the blob; the X tile arrives by TMA, 128 rows x 64 columns, 128-byte swizzled, and one
// MMA of M = 128, N = BOG * Bo, K = 16 per 16 columns runs at the tensor pipe's full rate.
//
// Roles: warp 0 issues the X tile loads (ring of kStagesX) and bulk-copies the compact values of
// each column block's BOG blocks into a small ring; warp 1 issues the MMAs; sixteen more warps
// write the weight tiles (two buffers: bi + 1 is written while bi is multiplied) and run the
// epilogue (fp32 bias, ReLU, one rounding, 16-byte stores).  A tile is written by destination:
// one item is 16 bytes (row n, eight columns), looked up through inverse index lists (row ->
// kept-row number, column -> kept-column number) that are built once per CTA.  An item is skipped
// when its row is pruned both in this block and in the block that used the buffer before, so no
// clearing pass and no synchronisation among the writers is needed.  Every wait is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kExpandWarps = 16;
constexpr int kExpandThreads = kExpandWarps * 32;
constexpr int kFirstExpandWarp = 2;
constexpr int kThreads = (kFirstExpandWarp + kExpandWarps) * 32;
constexpr int kRows = 128;
constexpr int kStagesX = 4;
constexpr int kMaxStagesV = 3;
constexpr int kItemsPerThread = 4;                        // 256 rows x 8 pieces over 512 writer threads
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kXStageBytes = kRows * 128;            // 128 rows of 64 bf16
// shared-memory descriptor, high word: SBO = 1024 bytes (eight 128-byte rows), version bit, 128-byte swizzle
constexpr uint32_t kDescHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
constexpr uint32_t kDescLboOne = 1u << 16;                // LBO is not used by swizzled K-major layouts

struct LinDxParams {
    int M, I, O, Bo, nBi, BOG, N;             // N = BOG * Bo accumulator columns
    int SV;                                   // stages of the value ring
    uint32_t v_slot;                          // bytes reserved per block in a value stage
    int relu, y_bf16;
    uint32_t b_bytes;                         // one expanded weight tile: N rows of 128 bytes
    uint32_t off_x, off_b, off_v, off_rowpos, off_colpos, off_raw, off_meta, off_bias, off_bar, smem_bytes, tmem_cols;
    BbLayout L;
};

struct LinDxBars {
    uint64_t x_full[kStagesX], x_empty[kStagesX];
    uint64_t b_ready[2], b_free[2];
    uint64_t v_full[kMaxStagesV], v_empty[kMaxStagesV];
    uint64_t tables;
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

// per (row block of the group, column block): kept rows / columns and where the values start
struct __align__(8) BlkMeta { uint32_t voff; uint8_t nr, nc; uint16_t pad; };

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    return cvt_bf16x2(lo, hi);
}
__device__ __forceinline__ uint64_t desc64(uint32_t lo) { return ((uint64_t)kDescHiSw128 << 32) | lo; }

// Eight weights of one kept row: element i is v[pos byte i], or zero where the column is pruned (0xFF).
__device__ __forceinline__ uint4 pick8(const uint16_t *v, uint2 pos)
{
    uint32_t e[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t b = ((i < 4 ? pos.x : pos.y) >> (8 * (i & 3))) & 0xFFu;
        e[i] = b != 0xFFu ? (uint32_t)v[b] : 0u;
    }
    return make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
}

__global__ void __launch_bounds__(kThreads, 1)
linear_bb_dx_kernel(const __grid_constant__ CUtensorMap tmap_x, const LinDxParams p,
                    const uint8_t *__restrict__ blob, const float *__restrict__ bias, const void *__restrict__ res,
                    void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xs = smem + p.off_x;             // [kStagesX][128 rows][128 bytes], swizzled
    uint8_t *bs = smem + p.off_b;             // [2][N rows][128 bytes], swizzled
    uint8_t *vs = smem + p.off_v;             // [SV][BOG] slots of v_slot bytes: compact values
    uint8_t *rowpos = smem + p.off_rowpos;    // [BOG][nBi][Bo]: row -> kept-row number, 0xFF = pruned
    uint8_t *colpos = smem + p.off_colpos;    // [BOG][nBi][64]: column -> kept-column number, 0xFF = pruned
    uint8_t *raw = smem + p.off_raw;          // the blob's kept-row and kept-column lists of the group
    BlkMeta *meta = reinterpret_cast<BlkMeta *>(smem + p.off_meta);   // [BOG][nBi]
    float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);     // [N]
    LinDxBars *bars = reinterpret_cast<LinDxBars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kRows, bo0 = blockIdx.y * p.BOG;
    const int rows_here = min(kRows, p.M - m0);
    const int nblk = p.BOG * p.nBi;
    const uint32_t rb = (uint32_t)nblk * p.Bo, cb = (uint32_t)nblk * 64u;

    if (tid == 0) {
        for (int s = 0; s < kStagesX; ++s) { mbar_init(&bars->x_full[s], 1); mbar_init(&bars->x_empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&bars->b_ready[s], kExpandWarps); mbar_init(&bars->b_free[s], 1); }
        for (int s = 0; s < p.SV; ++s) { mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], kExpandWarps); }
        mbar_init(&bars->acc_full, 1);
        mbar_init(&bars->tables, 1);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
    }
    if (warp == 1) tmem_alloc(&bars->tmem_base, p.tmem_cols);
    __syncthreads();
    // the group's blocks are contiguous in every section of the blob: index lists by bulk copy,
    // and the first X tiles can be on their way while the tables are built
    if (tid == 0) {
        mbar_arrive_expect_tx(&bars->tables, rb + cb);
        for (uint32_t o = 0; o < rb; o += 16384u)
            bulk_load_1d(raw + o, blob + p.L.off_rows + (size_t)bo0 * p.nBi * p.Bo + o, min(16384u, rb - o), &bars->tables);
        for (uint32_t o = 0; o < cb; o += 16384u)
            bulk_load_1d(raw + rb + o, blob + p.L.off_cols + (size_t)bo0 * p.nBi * 64 + o, min(16384u, cb - o), &bars->tables);
        for (int bi = 0; bi < kStagesX && bi < p.nBi; ++bi) {
            mbar_arrive_expect_tx(&bars->x_full[bi], kXStageBytes);
            tma_load_2d(xs + (size_t)bi * kXStageBytes, &tmap_x, &bars->x_full[bi], bi * 64, m0);
        }
    }
    for (int i = tid; i < nblk; i += kThreads) {
        const uint32_t b = bo0 * p.nBi + i;
        BlkMeta e;
        e.voff = reinterpret_cast<const uint32_t *>(blob + p.L.off_voff)[b];
        e.nr = blob[p.L.off_cnt + 2 * (size_t)b];
        e.nc = blob[p.L.off_cnt + 2 * (size_t)b + 1];
        e.pad = 0;
        meta[i] = e;
        // a block wider than the descriptor promised (or taller than Bo) would overrun its value slot
        if ((uint32_t)e.nr * e.nc * 2u > p.v_slot || (int)e.nr > p.Bo || e.nc > 64) {
            bars->abort_flag = 2;
            if (atomicCAS(ws, 0u, 6u /* NPAS_ERR_BLOB */) == 0u) ws[1] = 0x3001;
        }
    }
    for (int i = tid; i < p.N; i += kThreads) bias_s[i] = bias ? bias[bo0 * p.Bo + i] : 0.f;
    // both weight tiles start as zeros; the inverse lists start as "pruned"
    for (uint32_t o = tid * 16; o < 2 * p.b_bytes; o += kThreads * 16) *reinterpret_cast<uint4 *>(bs + o) = make_uint4(0, 0, 0, 0);
    for (uint32_t o = tid * 16; o < rb + cb; o += kThreads * 16)       // rowpos and colpos are adjacent
        *reinterpret_cast<uint4 *>(rowpos + o) = make_uint4(~0u, ~0u, ~0u, ~0u);
    const bool tables_ok = mbar_wait(&bars->tables, 0, abort_flag, ws, 0x3700);
    __syncthreads();
    if (tables_ok) {
        for (uint32_t i = tid; i < rb; i += kThreads) {
            const uint32_t blk = i / p.Bo, j = i - blk * p.Bo, r = raw[i];
            if (r < (uint32_t)p.Bo) rowpos[blk * p.Bo + r] = (uint8_t)j;
        }
        for (uint32_t i = tid; i < cb; i += kThreads) {
            const uint32_t c = raw[rb + i];
            if (c < 64u) colpos[(i & ~63u) + c] = (uint8_t)(i & 63u);
        }
    }
    fence_proxy_async_smem();                   // the zeros of the weight tiles are read by the tensor core
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    bool ok = *abort_flag == 0;                 // a blob that breaks the descriptor's promise: nothing runs
    if (!ok) {
        // fall through to the tear-down, which waits for the X tiles already requested
    } else if (warp == 0) {
        // ---- producer: compact values of column block bi, then (past the first ring lap) its X tile --
        if (lane == 0) {
            const uint8_t *vals = blob + p.L.off_values;
            for (int bi = 0; bi < p.nBi; ++bi) {
                const int sv = bi % p.SV, lapv = bi / p.SV;
                if (lapv >= 1 && !mbar_wait(&bars->v_empty[sv], (lapv & 1) ^ 1, abort_flag, ws, 0x3600 + bi)) break;
                uint32_t total = 0;
                for (int g = 0; g < p.BOG; ++g) {
                    const BlkMeta e = meta[g * p.nBi + bi];
                    total += round_up((uint32_t)e.nr * e.nc * 2u, 16u);
                }
                mbar_arrive_expect_tx(&bars->v_full[sv], total);
                for (int g = 0; g < p.BOG; ++g) {
                    const BlkMeta e = meta[g * p.nBi + bi];
                    const uint32_t bytes = round_up((uint32_t)e.nr * e.nc * 2u, 16u);
                    if (bytes) bulk_load_1d(vs + ((size_t)sv * p.BOG + g) * p.v_slot, vals + (size_t)e.voff * 2, bytes, &bars->v_full[sv]);
                }
                if (bi < kStagesX) continue;
                const int s = bi % kStagesX, lap = bi / kStagesX;
                if (!mbar_wait(&bars->x_empty[s], (lap & 1) ^ 1, abort_flag, ws, 0x3100 + bi)) break;
                mbar_arrive_expect_tx(&bars->x_full[s], kXStageBytes);
                tma_load_2d(xs + (size_t)s * kXStageBytes, &tmap_x, &bars->x_full[s], bi * 64, m0);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue -------------------------------------------------------------------------------
        const uint32_t idesc = idesc_bf16_f32(128, p.N);
        const uint32_t x16 = smem_u32(xs) >> 4, b16 = smem_u32(bs) >> 4;
        for (int bi = 0; bi < p.nBi && ok; ++bi) {
            const int s = bi % kStagesX, buf = bi & 1;
            if (!mbar_wait(&bars->x_full[s], (bi / kStagesX) & 1, abort_flag, ws, 0x3200 + bi)) { ok = false; break; }
            if (!mbar_wait(&bars->b_ready[buf], (bi >> 1) & 1, abort_flag, ws, 0x3300 + bi)) { ok = false; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t a_lo = (x16 + s * (kXStageBytes >> 4)) | kDescLboOne;
                const uint32_t b_lo = (b16 + buf * (p.b_bytes >> 4)) | kDescLboOne;
#pragma unroll
                for (uint32_t k = 0; k < 4; ++k)          // 16 columns = 32 bytes inside the swizzled row
                    mma_bf16_ss(tmem_base, desc64(a_lo + 2 * k), desc64(b_lo + 2 * k), idesc, (bi > 0 || k > 0) ? 1u : 0u);
                mma_commit(&bars->x_empty[s]);
                mma_commit(&bars->b_free[buf]);
                if (bi == p.nBi - 1) mma_commit(&bars->acc_full);
            }
            __syncwarp();
        }
    } else {
        // ---- weight tile writers ---------------------------------------------------------------------
        // a thread's items (row n, 16-byte piece c) are the same for every column block
        const int t = tid - kFirstExpandWarp * 32;
        int it_g[kItemsPerThread], it_r[kItemsPerThread];
        uint32_t it_off[kItemsPerThread], it_c[kItemsPerThread];
#pragma unroll
        for (int u = 0; u < kItemsPerThread; ++u) {
            const int item = t + u * kExpandThreads, n = item >> 3, c = item & 7;
            it_g[u] = n < p.N ? n / p.Bo : -1;
            it_r[u] = n - (n / p.Bo) * p.Bo;
            it_c[u] = (uint32_t)c;
            it_off[u] = (uint32_t)n * 128u + (uint32_t)((c ^ n) & 7) * 16u;
        }
        for (int bi = 0; bi < p.nBi && ok; ++bi) {
            const int buf = bi & 1, sv = bi % p.SV;
            if (bi >= 2 && !mbar_wait(&bars->b_free[buf], ((bi >> 1) - 1) & 1, abort_flag, ws, 0x3400 + bi)) { ok = false; break; }
            if (!mbar_wait(&bars->v_full[sv], (bi / p.SV) & 1, abort_flag, ws, 0x3800 + bi)) { ok = false; break; }
            uint8_t *tile = bs + (size_t)buf * p.b_bytes;
#pragma unroll
            for (int u = 0; u < kItemsPerThread; ++u) {
                if (it_g[u] < 0) continue;
                const int blk = it_g[u] * p.nBi + bi;
                const uint32_t jr = rowpos[blk * p.Bo + it_r[u]];
                const uint32_t jo = bi >= 2 ? rowpos[(blk - 2) * p.Bo + it_r[u]] : 0xFFu;   // the buffer's previous tile
                if (jr == 0xFFu && jo == 0xFFu) continue;
                uint4 o = make_uint4(0, 0, 0, 0);
                if (jr != 0xFFu) {
                    const uint2 pos = *reinterpret_cast<const uint2 *>(colpos + (size_t)blk * 64 + it_c[u] * 8);
                    const uint16_t *v = reinterpret_cast<const uint16_t *>(vs + ((size_t)sv * p.BOG + it_g[u]) * p.v_slot) +
                                        jr * meta[blk].nc;
                    o = pick8(v, pos);
                }
                *reinterpret_cast<uint4 *>(tile + it_off[u]) = o;
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) { mbar_arrive(&bars->b_ready[buf]); mbar_arrive(&bars->v_empty[sv]); }
        }

        // ---- epilogue ----------------------------------------------------------------------------------
        if (ok && !mbar_wait(&bars->acc_full, 0, abort_flag, ws, 0x3500)) ok = false;
        tc_fence_after_sync();
        const int quarter = warp & 3, part = (warp - kFirstExpandWarp) >> 2, m = quarter * 32 + lane;
        const bool valid = m < rows_here;
        const size_t o0 = (size_t)(m0 + m) * p.O + (size_t)bo0 * p.Bo;
        if (ok) {
            for (int c0 = part * 16; c0 < p.N; c0 += 16 * (kExpandWarps / 4)) {
                uint32_t r[16];
                __syncwarp();
                tmem_ld_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_ld_wait();
                if (valid) {
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) + bias_s[c0 + i];
                    if (res) {
                        if (p.y_bf16) {
                            const uint4 *rp = reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(res) + o0 + c0);
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const uint4 u = rp[h];
                                const uint32_t wv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    v[8 * h + 2 * i] += __uint_as_float(wv[i] << 16);
                                    v[8 * h + 2 * i + 1] += __uint_as_float(wv[i] & 0xFFFF0000u);
                                }
                            }
                        } else {
                            const float4 *rp = reinterpret_cast<const float4 *>(static_cast<const float *>(res) + o0 + c0);
#pragma unroll
                            for (int h = 0; h < 4; ++h) {
                                const float4 u = rp[h];
                                v[4 * h] += u.x; v[4 * h + 1] += u.y; v[4 * h + 2] += u.z; v[4 * h + 3] += u.w;
                            }
                        }
                    }
                    if (p.relu) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
                    }
                    if (p.y_bf16) {
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
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        // a role gave up: leave time for copies still in flight to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

bool plan(const npas_linear_desc &d, const npas_bb_desc &bb, LinDxParams &p)
{
    if (d.x_dtype != NPAS_BF16 || bb.w_packed != NPAS_BF16) return false;
    if (bb.Bi != 64 || bb.Bo % 16 || d.I % 64 || d.O % 8) return false;
    p.M = d.M; p.I = d.I; p.O = d.O; p.Bo = bb.Bo;
    p.L = bb_layout(bb);
    p.nBi = p.L.nBi;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    const int nBo = p.L.nBo;
    p.BOG = 0;
    for (int g = 1; g <= nBo && g * bb.Bo <= 256; ++g)
        if (nBo % g == 0) p.BOG = g;
    if (p.BOG == 0) return false;
    p.N = p.BOG * bb.Bo;
    p.b_bytes = (uint32_t)p.N * 128u;
    p.off_x = 0;
    p.off_b = kStagesX * kXStageBytes;
    if (bb.max_cols <= 0 || bb.max_cols > 64) return false;   // bounds the compact values of one block
    p.v_slot = round_up((uint32_t)bb.Bo * bb.max_cols * 2u, 16u);
    p.SV = kMaxStagesV;
    p.off_v = p.off_b + 2 * round_up(p.b_bytes, 1024);
    p.off_rowpos = p.off_v + p.SV * p.BOG * p.v_slot;           // Bo % 16 == 0 keeps all of these 16-byte aligned
    p.off_colpos = p.off_rowpos + p.BOG * p.nBi * bb.Bo;
    p.off_raw = p.off_colpos + p.BOG * p.nBi * 64;
    p.off_meta = p.off_raw + p.BOG * p.nBi * (bb.Bo + 64);
    p.off_bias = round_up(p.off_meta + p.BOG * p.nBi * (uint32_t)sizeof(BlkMeta), 16);
    p.off_bar = round_up(p.off_bias + p.N * 4, 128);
    p.smem_bytes = p.off_bar + sizeof(LinDxBars) + 1024;
    if (p.smem_bytes > kSmemLimit) return false;
    p.b_bytes = round_up(p.b_bytes, 1024);
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < p.N) p.tmem_cols *= 2;
    return true;
}

}  // namespace

bool linear_dx_supported(const npas_linear_desc &d, const npas_bb_desc &bb)
{
    LinDxParams p;
    return plan(d, bb, p);
}

npas_status linear_dx_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                             const void *blob, const float *bias, const void *res, void *y, uint32_t *ws,
                             cudaStream_t st)
{
    LinDxParams p;
    if (!plan(d, bb, p)) return NPAS_ERR_UNSUPPORTED;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return NPAS_ERR_CUDA;
    // X[M][I] bf16: a box of 64 columns x 128 rows lands as 128-byte rows, 16-byte pieces XOR-ed
    // with the row number (rows past M read as zeros)
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)d.I, (cuuint64_t)d.M};
    const cuuint64_t strides[1] = {(cuuint64_t)d.I * 2};
    const cuuint32_t box[2] = {64, kRows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return NPAS_ERR_CUDA;
    if (cudaFuncSetAttribute(linear_bb_dx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess)
        return NPAS_ERR_CUDA;
    const dim3 grid((d.M + kRows - 1) / kRows, p.L.nBo / p.BOG);
    if (grid.y > 65535) return NPAS_ERR_UNSUPPORTED;
    linear_bb_dx_kernel<<<grid, kThreads, p.smem_bytes, st>>>(tmap, p, static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return launch_status();
}

}  // namespace npas
