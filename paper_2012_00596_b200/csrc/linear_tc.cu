// Block-based pruned GEMM on the sm_100a tensor cores (bf16 in, fp32 accumulation in TMEM).
//
// Per weight block (bo, bi) the pruned product keeps nc of the Bi input columns and nr of the Bo
// output rows.  The kept columns are a gather along K, which no operand descriptor can express at
// 2-byte granularity, so the CTA gathers them with plain shared-memory loads:
//   A(bo,bi)[m][j] = X[m][bi*Bi + cols[j]]      (128 rows x Kp columns, Kp = kept columns, padded to 16)
// written directly in the no-swizzle K-major operand layout ([K octet][row][8]).  The kept rows
// are NOT compacted: the B operand is the block's [Bo x Kp] kept-column matrix with zero rows
// where a row is pruned, so every column block accumulates into the same Bo TMEM columns and no
// scatter of partial results is needed.  MMAs are M = 128, N = Bo, K = 16.
//
// One CTA owns 128 rows of X and a group of BOG row blocks (BOG * Bo accumulator columns).  The
// zero-row-expanded weight tiles of the group are a contiguous piece of the blob (the packer
// writes every block's tile in operand layout), fetched with bulk copies once, up front.  Then
// sixteen gather warps walk the column blocks: the X tile of the next column block is already in
// flight (registers) while the current one is gathered into one of two operand buffers, and one
// more warp issues the MMAs of a column block as soon as every gather warp has arrived.
// The X tile is stored with an odd word pitch so that a warp reading one column of 32 rows hits
// 32 different banks; unused gather slots read a zero kept behind every row.  The epilogue adds
// the fp32 bias (staged in shared memory up front), applies ReLU, rounds once and stores 16-byte words.  Every wait is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kGatherWarps = 16;
constexpr int kGatherThreads = kGatherWarps * 32;
constexpr int kThreads = kGatherThreads + 32;    // + one MMA-issuing warp
constexpr int kRows = 128;
constexpr int kPiecesPerThread = 2;              // 16-byte pieces of an X tile per gather thread
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kDescHi = (128u >> 4) | (1u << 14);   // SBO = 128 bytes, descriptor version bit

struct LinTcParams {
    int M, I, O, Bo, Bi, nBi, BOG, Kp;
    int relu, y_bf16;
    uint32_t xt_pitch;                        // bytes per staged X row: Bi elements + 2 zero elements
    uint32_t a_bytes, b_bytes;                // per (row block) gathered operand / per block weight tile
    uint32_t off_b, off_xt, off_a, off_cols, off_bias, off_bar, smem_bytes, tmem_cols;
    BbLayout L;
};

struct LinBars {
    uint64_t ready[2], done[2], tiles;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    return cvt_bf16x2(lo, hi);
}
__device__ __forceinline__ void gather_sync() { asm volatile("bar.sync 1, 512;" ::: "memory"); }
__device__ __forceinline__ uint64_t desc64(uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; }

// Eight elements of one staged X row, picked by eight byte indices, as one 16-byte operand row.
__device__ __forceinline__ uint4 gather8(const uint16_t *row, uint2 ci)
{
    const uint32_t e0 = row[ci.x & 0xFF], e1 = row[(ci.x >> 8) & 0xFF], e2 = row[(ci.x >> 16) & 0xFF], e3 = row[ci.x >> 24];
    const uint32_t e4 = row[ci.y & 0xFF], e5 = row[(ci.y >> 8) & 0xFF], e6 = row[(ci.y >> 16) & 0xFF], e7 = row[ci.y >> 24];
    return make_uint4(e0 | (e1 << 16), e2 | (e3 << 16), e4 | (e5 << 16), e6 | (e7 << 16));
}

__global__ void __launch_bounds__(kThreads, 1)
linear_bb_tc_kernel(const LinTcParams p, const uint16_t *__restrict__ x, const uint8_t *__restrict__ blob,
                    const float *__restrict__ bias, const void *__restrict__ res, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *btiles = smem + p.off_b;         // [BOG][nBi][Kp/8][Bo][8] bf16: weight tiles with zero rows
    uint8_t *xt = smem + p.off_xt;            // [2][128] rows of xt_pitch bytes
    uint8_t *ag = smem + p.off_a;             // [2][BOG][Kp/8][128][8] bf16: gathered operands
    uint8_t *cols_s = smem + p.off_cols;      // [nBi][BOG][Kp] column indices, unused slots -> the zero element
    float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);   // [BOG * Bo]
    LinBars *bars = reinterpret_cast<LinBars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kRows, bo0 = blockIdx.y * p.BOG;
    const int rows_here = min(kRows, p.M - m0);
    const int KH = p.Kp / 8, GH = p.BOG * KH, nblk = p.BOG * p.nBi;
    const int ncol = p.BOG * p.Bo;

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(&bars->ready[s], kGatherWarps); mbar_init(&bars->done[s], 1); }
        mbar_init(&bars->tiles, 1);
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == kGatherWarps) tmem_alloc(&bars->tmem_base, p.tmem_cols);
    // column lists with unused slots pointing at the zero element kept behind every staged row
    for (int i = tid; i < nblk * p.Kp; i += kThreads) {
        const int bi = i / (p.BOG * p.Kp), r = i - bi * (p.BOG * p.Kp), g = r / p.Kp, j = r - g * p.Kp;
        const uint32_t b = (bo0 + g) * p.nBi + bi;
        const uint8_t c = j < p.Bi ? blob[p.L.off_cols + (size_t)b * p.Bi + j] : (uint8_t)0xFF;
        cols_s[i] = c == 0xFF ? (uint8_t)p.Bi : c;
    }
    for (int i = tid; i < ncol; i += kThreads) bias_s[i] = bias ? bias[bo0 * p.Bo + i] : 0.f;
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    if (tid == 0 && hdr[BB_KP] != (uint32_t)p.Kp) bars->abort_flag = 2;   // tiles were packed for another width
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const bool bad = *abort_flag != 0;
    if (bad && tid == 0) { if (atomicCAS(ws, 0u, 6u /* NPAS_ERR_BLOB */) == 0u) ws[1] = 0x2001; }
    // the group's weight tiles: contiguous in the blob, fetched in pieces of at most 16 KB
    if (!bad && tid == 0) {
        const uint32_t total = (uint32_t)nblk * p.b_bytes;
        const uint8_t *src = blob + hdr[BB_OFF_TILES] + (size_t)bo0 * p.nBi * p.b_bytes;
        mbar_arrive_expect_tx(&bars->tiles, total);
        for (uint32_t o = 0; o < total; o += 16384u)
            bulk_load_1d(btiles + o, src + o, min(16384u, total - o), &bars->tiles);
    }

    bool ok = !bad;
    if (bad) {
        // nothing to do
    } else if (warp < kGatherWarps) {
        // ---- gather warps ---------------------------------------------------------------------------
        // the 16-byte pieces of an X tile this thread moves: the same (row, piece) for every column block
        const int chunks_per_row = p.Bi / 8, pieces = kRows * chunks_per_row;
        const uint16_t *src[kPiecesPerThread];
        uint32_t dst[kPiecesPerThread];
#pragma unroll
        for (int k = 0; k < kPiecesPerThread; ++k) {
            const int e = tid + k * kGatherThreads, r = e / chunks_per_row, ch = e - r * chunks_per_row;
            src[k] = (e < pieces && r < rows_here) ? x + (size_t)(m0 + r) * p.I + ch * 8 : nullptr;
            dst[k] = e < pieces ? r * p.xt_pitch + ch * 16 : 0xFFFFFFFFu;
        }
        uint4 pre[kPiecesPerThread];
        auto load_tile = [&](int bi) {
#pragma unroll
            for (int k = 0; k < kPiecesPerThread; ++k)
                pre[k] = src[k] ? *reinterpret_cast<const uint4 *>(src[k] + bi * p.Bi) : make_uint4(0, 0, 0, 0);
        };
        auto store_tile = [&](int buf) {
            uint8_t *t = xt + (size_t)buf * kRows * p.xt_pitch;
#pragma unroll
            for (int k = 0; k < kPiecesPerThread; ++k) {
                if (dst[k] != 0xFFFFFFFFu) {
                    uint32_t *d = reinterpret_cast<uint32_t *>(t + dst[k]);
                    d[0] = pre[k].x; d[1] = pre[k].y; d[2] = pre[k].z; d[3] = pre[k].w;
                }
            }
            if (tid < kRows) *reinterpret_cast<uint32_t *>(t + tid * p.xt_pitch + p.Bi * 2) = 0u;   // the zero element
        };
        load_tile(0);
        store_tile(0);
        gather_sync();
        // item = (K octet gh of the group's operands, row m): 8 gathered elements = one 16-byte operand
        // row.  A thread keeps its row; a warp's 32 rows sit in 32 different banks.
        const int m = tid & (kRows - 1), q = tid >> 7;
        for (int bi = 0; bi < p.nBi; ++bi) {               // every thread runs every iteration (bar.sync inside)
            const int set = bi & 1;
            if (bi + 1 < p.nBi) load_tile(bi + 1);
            if (bi >= 2 && !mbar_wait(&bars->done[set], ((bi >> 1) - 1) & 1, abort_flag, ws, 0x2100 + bi)) ok = false;
            const uint16_t *row = reinterpret_cast<const uint16_t *>(xt + (size_t)set * kRows * p.xt_pitch + m * p.xt_pitch);
            const uint8_t *cb = cols_s + (size_t)bi * GH * 8;
            uint8_t *out = ag + (size_t)set * p.BOG * p.a_bytes + m * 16;
            for (int gh = q; gh < GH; gh += 8) {            // two independent items per trip
                const int gh2 = gh + 4;
                const bool two = gh2 < GH;
                const uint2 c1 = *reinterpret_cast<const uint2 *>(cb + gh * 8);
                const uint2 c2 = *reinterpret_cast<const uint2 *>(cb + (two ? gh2 : gh) * 8);
                const uint4 o1 = gather8(row, c1), o2 = gather8(row, c2);
                *reinterpret_cast<uint4 *>(out + (size_t)gh * (kRows * 16)) = o1;
                if (two) *reinterpret_cast<uint4 *>(out + (size_t)gh2 * (kRows * 16)) = o2;
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->ready[set]);
            if (bi + 1 < p.nBi) store_tile((bi + 1) & 1);
            gather_sync();                                 // tile bi+1 complete; tile bi no longer read
        }
    } else {
        // ---- MMA warp ---------------------------------------------------------------------------------
        const uint32_t idesc = idesc_bf16_f32(128, p.Bo);
        // descriptor low words in 16-byte units: start address | distance between K octets << 16
        const uint32_t a_lo0 = (smem_u32(ag) >> 4) | ((uint32_t)kRows << 16);
        const uint32_t b_lo0 = (smem_u32(btiles) >> 4) | ((uint32_t)p.Bo << 16);
        const uint32_t a16 = p.a_bytes >> 4, b16 = p.b_bytes >> 4, nS = p.Kp / 16;
        if (!mbar_wait(&bars->tiles, 0, abort_flag, ws, 0x2250)) ok = false;
        for (int bi = 0; bi < p.nBi && ok; ++bi) {
            const int set = bi & 1;
            if (!mbar_wait(&bars->ready[set], (bi >> 1) & 1, abort_flag, ws, 0x2200 + bi)) { ok = false; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                uint32_t a_lo = a_lo0 + set * p.BOG * a16, b_lo = b_lo0 + bi * b16;
                for (int g = 0; g < p.BOG; ++g, a_lo += a16, b_lo += p.nBi * b16) {
                    for (uint32_t s = 0; s < nS; ++s)
                        mma_bf16_ss(tmem_base + g * p.Bo, desc64(a_lo + s * (2 * kRows)), desc64(b_lo + s * (2 * p.Bo)),
                                    idesc, (bi > 0 || s > 0) ? 1u : 0u);
                }
                mma_commit(&bars->done[set]);
            }
            __syncwarp();
        }
    }

    // ---- epilogue (gather warps): wait for the last MMAs of both operand sets ----------------------
    if (warp < kGatherWarps && !bad) {
        const int last = p.nBi - 1;
        if (ok && !mbar_wait(&bars->done[last & 1], (last >> 1) & 1, abort_flag, ws, 0x2300)) ok = false;
        if (ok && last >= 1 && !mbar_wait(&bars->done[(last - 1) & 1], ((last - 1) >> 1) & 1, abort_flag, ws, 0x2301)) ok = false;
        tc_fence_after_sync();
        const int quarter = warp & 3, part = warp >> 2, m = quarter * 32 + lane;
        const bool valid = m < rows_here;
        const size_t o0 = (size_t)(m0 + m) * p.O + (size_t)bo0 * p.Bo;
        if (ok) {
            for (int c0 = part * 16; c0 < ncol; c0 += 16 * (kGatherWarps / 4)) {
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
    if (warp == kGatherWarps) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

bool plan(const npas_linear_desc &d, const npas_bb_desc &bb, LinTcParams &p)
{
    if (d.x_dtype != NPAS_BF16 || bb.w_packed != NPAS_BF16) return false;
    if (bb.Bo % 16 || bb.Bi % 8 || bb.Bi > 64 || d.I % 8 || d.O % 8) return false;
    p.M = d.M; p.I = d.I; p.O = d.O; p.Bo = bb.Bo; p.Bi = bb.Bi;
    p.L = bb_layout(bb);
    p.nBi = p.L.nBi;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    if (bb.max_cols <= 0 || bb.max_cols > bb.Bi) return false;   // the tile width of the blob must be known
    p.Kp = max(16, (bb.max_cols + 15) / 16 * 16);
    p.xt_pitch = bb.Bi * 2 + 4;
    if (kRows * (bb.Bi / 8) > kPiecesPerThread * kGatherThreads) return false;
    p.a_bytes = (uint32_t)(p.Kp / 8) * kRows * 16;
    p.b_bytes = (uint32_t)(p.Kp / 8) * bb.Bo * 16;
    const int nBo = p.L.nBo;
    p.BOG = 0;
    for (int g = 1; g <= nBo && g * bb.Bo <= 256; ++g) {
        if (nBo % g || (g * bb.Bo) % 32) continue;
        const uint32_t need = (uint32_t)g * p.nBi * p.b_bytes + 2 * kRows * p.xt_pitch + 2u * g * p.a_bytes +
                              (uint32_t)g * p.nBi * p.Kp + 4096;
        if (need <= kSmemLimit) p.BOG = g;
    }
    if (p.BOG == 0) return false;
    p.off_b = 0;
    p.off_xt = round_up((uint32_t)p.BOG * p.nBi * p.b_bytes, 128);
    p.off_a = round_up(p.off_xt + 2 * kRows * p.xt_pitch, 128);
    p.off_cols = p.off_a + 2 * p.BOG * p.a_bytes;
    p.off_bias = round_up(p.off_cols + p.BOG * p.nBi * p.Kp, 128);
    p.off_bar = round_up(p.off_bias + p.BOG * bb.Bo * 4, 128);
    p.smem_bytes = p.off_bar + sizeof(LinBars) + 1024;
    if (p.smem_bytes > kSmemLimit) return false;
    if (2u * p.BOG * p.a_bytes >= (1u << 18) || (uint32_t)p.BOG * p.nBi * p.b_bytes >= (1u << 18)) return false;
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < p.BOG * bb.Bo) p.tmem_cols *= 2;
    return true;
}

}  // namespace

bool linear_tc_supported(const npas_linear_desc &d, const npas_bb_desc &bb)
{
    LinTcParams p;
    return plan(d, bb, p);
}

npas_status linear_tc_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                             const void *blob, const float *bias, const void *res, void *y, uint32_t *ws,
                             cudaStream_t st)
{
    LinTcParams p;
    if (!plan(d, bb, p)) return NPAS_ERR_UNSUPPORTED;
    if (allow_dynamic_smem(reinterpret_cast<const void *>(linear_bb_tc_kernel), (int)kSmemLimit) != NPAS_OK) return NPAS_ERR_CUDA;
    const dim3 grid((d.M + kRows - 1) / kRows, p.L.nBo / p.BOG);
    if (grid.y > 65535) return NPAS_ERR_UNSUPPORTED;
    linear_bb_tc_kernel<<<grid, kThreads, p.smem_bytes, st>>>(p, static_cast<const uint16_t *>(x),
                                                              static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return launch_status();
}

}  // namespace npas
