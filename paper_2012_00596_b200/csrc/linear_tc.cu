// Block-based pruned GEMM on the sm_100a tensor cores (bf16 in, fp32 accumulation in TMEM).
//
// Per weight block (bo, bi) the pruned product keeps nc of the Bi input columns and nr of the Bo
// output rows.  The kept columns are a gather along K, which no operand descriptor can express at
// 2-byte granularity, so the CTA gathers them with plain shared-memory traffic:
//   A(bo,bi)[m][j] = X[m][bi*Bi + cols[j]]      (128 rows x Kp columns, Kp = nc rounded up to 16)
// written directly in the no-swizzle K-major operand layout ([K octet][row][8]).  The kept rows
// are NOT compacted: the B operand is the block's [Bo x Kp] kept-column matrix with zero rows
// where a row is pruned, so every column block accumulates into the same Bo TMEM columns and no
// scatter of partial results is needed.  MMAs are M = 128, N = Bo, K = 16.
//
// One CTA owns 128 rows of X and a group of row blocks; it walks the column blocks with two
// operand buffers so that the tensor core works on one column block while the threads gather the
// next.  The epilogue adds the fp32 bias, applies ReLU, rounds once and stores 16-byte words.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kThreads = 256;
constexpr int kRows = 128;
constexpr uint32_t kSmemLimit = 232448;

struct LinTcParams {
    int M, I, O, Bo, Bi, nBi, BOG;
    int relu, y_bf16;
    uint32_t xt_pitch;                    // bytes per staged X row (odd number of 32-bit words)
    uint32_t a_bytes, b_bytes, set_bytes; // per row block / per buffer set
    uint32_t off_xt, off_sets, off_idx, off_bar, smem_bytes, tmem_cols;
    BbLayout L;
};

struct LinBars {
    uint64_t done[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t touched;   // bit g set once row block g of the group has received an MMA
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    return (uint32_t)f32_bits_to_bf16(__float_as_uint(lo)) | ((uint32_t)f32_bits_to_bf16(__float_as_uint(hi)) << 16);
}

__global__ void __launch_bounds__(kThreads, 1)
linear_bb_tc_kernel(const LinTcParams p, const uint16_t *__restrict__ x, const uint8_t *__restrict__ blob,
                    const float *__restrict__ bias, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xt = smem + p.off_xt;
    uint8_t *sets = smem + p.off_sets;
    uint8_t *idx = smem + p.off_idx;      // per row block of the group: cols[Bi], rows[Bo], nr, nc
    LinBars *bars = reinterpret_cast<LinBars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kRows, bo0 = blockIdx.y * p.BOG;
    const int rows_here = min(kRows, p.M - m0);
    const uint32_t idx_stride = p.Bi + p.Bo + 16;
    const uint32_t *voff = reinterpret_cast<const uint32_t *>(blob + p.L.off_voff);
    const uint16_t *vals = reinterpret_cast<const uint16_t *>(blob + p.L.off_values);

    if (tid == 0) {
        mbar_init(&bars->done[0], 1);
        mbar_init(&bars->done[1], 1);
        bars->abort_flag = 0;
        bars->touched = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(&bars->tmem_base, p.tmem_cols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const uint32_t idesc = idesc_bf16_f32(128, p.Bo);
    bool ok = true;
    uint32_t touched = 0;   // meaningful in thread 0 only

    for (int bi = 0; bi < p.nBi; ++bi) {
        const int buf = bi & 1;
        // the MMAs that read this buffer set two column blocks ago must have completed
        if (bi >= 2 && !mbar_wait(&bars->done[buf], ((bi >> 1) - 1) & 1, abort_flag, ws, 0x600 + bi)) ok = false;
        // ---- stage X[m0.., bi*Bi..] with an odd word pitch (conflict-free column reads) ----------
        {
            const int chunks_per_row = p.Bi / 8;                  // 16-byte pieces per row
            for (int e = tid; e < kRows * chunks_per_row; e += kThreads) {
                const int r = e / chunks_per_row, ch = e % chunks_per_row;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (r < rows_here) v = *reinterpret_cast<const uint4 *>(x + (size_t)(m0 + r) * p.I + bi * p.Bi + ch * 8);
                uint32_t *dst = reinterpret_cast<uint32_t *>(xt + r * p.xt_pitch + ch * 16);
                dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
            }
            for (int e = tid; e < p.BOG * (int)idx_stride; e += kThreads) {
                const int g = e / idx_stride, o = e % idx_stride;
                const uint32_t b = (bo0 + g) * p.nBi + bi;
                uint8_t v = 0;
                if (o < p.Bi) v = blob[p.L.off_cols + (size_t)b * p.Bi + o];
                else if (o < p.Bi + p.Bo) v = blob[p.L.off_rows + (size_t)b * p.Bo + (o - p.Bi)];
                else if (o == p.Bi + p.Bo) v = blob[p.L.off_cnt + 2 * b];
                else if (o == p.Bi + p.Bo + 1) v = blob[p.L.off_cnt + 2 * b + 1];
                idx[e] = v;
            }
        }
        __syncthreads();
        // ---- gather the kept columns and lay out the zero-row-expanded weights --------------------
        uint8_t *set = sets + (size_t)buf * p.set_bytes;
        for (int g = 0; g < p.BOG; ++g) {
            const uint8_t *ix = idx + g * idx_stride;
            const int nr = ix[p.Bi + p.Bo], nc = ix[p.Bi + p.Bo + 1];
            const int kp8 = ((nc + 15) / 16) * 2;                 // K octets after padding to 16
            uint8_t *A = set + (size_t)g * (p.a_bytes + p.b_bytes), *B = A + p.a_bytes;
            for (int e = tid; e < kRows * kp8; e += kThreads) {
                const int m = e % kRows, h = e / kRows;
                const uint16_t *row = reinterpret_cast<const uint16_t *>(xt + m * p.xt_pitch);
                uint32_t w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int j0 = h * 8 + 2 * q;
                    const uint32_t lo = j0 < nc ? row[ix[j0]] : 0u;
                    const uint32_t hi = j0 + 1 < nc ? row[ix[j0 + 1]] : 0u;
                    w[q] = lo | (hi << 16);
                }
                *reinterpret_cast<uint4 *>(A + (size_t)h * (kRows * 16) + m * 16) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            for (int e = tid; e < kp8 * p.Bo; e += kThreads)
                *reinterpret_cast<uint4 *>(B + (size_t)e * 16) = make_uint4(0, 0, 0, 0);
        }
        __syncthreads();
        for (int g = 0; g < p.BOG; ++g) {
            const uint8_t *ix = idx + g * idx_stride;
            const int nr = ix[p.Bi + p.Bo], nc = ix[p.Bi + p.Bo + 1];
            uint8_t *B = set + (size_t)g * (p.a_bytes + p.b_bytes) + p.a_bytes;
            const uint16_t *v = vals + voff[(bo0 + g) * p.nBi + bi];
            for (int e = tid; e < nr * nc; e += kThreads) {
                const int r = e / nc, j = e % nc;
                *reinterpret_cast<uint16_t *>(B + (size_t)(j / 8) * (p.Bo * 16) + ix[p.Bi + r] * 16 + (j % 8) * 2) = v[e];
            }
        }
        fence_proxy_async_smem();
        __syncthreads();
        // ---- one thread issues this column block's MMAs ----------------------------------------------
        if (tid == 0 && ok) {
            tc_fence_after_sync();
            for (int g = 0; g < p.BOG; ++g) {
                const uint8_t *ix = idx + g * idx_stride;
                const int nc = ix[p.Bi + p.Bo + 1];
                const uint32_t A = smem_u32(set + (size_t)g * (p.a_bytes + p.b_bytes)), B = A + p.a_bytes;
                for (int s = 0; s < (nc + 15) / 16; ++s) {
                    const uint64_t ad = smem_desc_kmajor(A + 2 * s * (kRows * 16), kRows * 16, 128);
                    const uint64_t bd = smem_desc_kmajor(B + 2 * s * (p.Bo * 16), p.Bo * 16, 128);
                    mma_bf16_ss(tmem_base + g * p.Bo, ad, bd, idesc, (touched >> g) & 1u);
                    touched |= 1u << g;
                }
            }
            mma_commit(&bars->done[buf]);
            bars->touched = touched;
        }
        // idx is rewritten by the next iteration only after its first __syncthreads... the issuing
        // thread reads idx above, so hold everyone until it is done with it
        __syncthreads();
    }

    // ---- epilogue: wait for the last MMAs of both buffer sets -------------------------------------
    {
        const int last = p.nBi - 1;
        if (ok && !mbar_wait(&bars->done[last & 1], (last >> 1) & 1, abort_flag, ws, 0x700)) ok = false;
        if (ok && last >= 1 && !mbar_wait(&bars->done[(last - 1) & 1], ((last - 1) >> 1) & 1, abort_flag, ws, 0x701)) ok = false;
        tc_fence_after_sync();
        const int quarter = warp & 3, half = warp >> 2, m = quarter * 32 + lane;
        const int ncol = p.BOG * p.Bo, c_begin = half * (ncol / 2), c_end = c_begin + ncol / 2;
        const bool valid = m < rows_here;
        const size_t o0 = (size_t)(m0 + m) * p.O + (size_t)bo0 * p.Bo;
        if (ok) {
            for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                uint32_t r[16];
                __syncwarp();
                tmem_ld_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_ld_wait();
                if (valid) {
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        // a row block that kept no column anywhere never received an MMA
                        v[i] = ((bars->touched >> (c0 / p.Bo)) & 1u) ? __uint_as_float(r[i]) : 0.f;
                        if (bias) v[i] += __ldg(bias + bo0 * p.Bo + c0 + i);
                        if (p.relu) v[i] = fmaxf(v[i], 0.f);
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
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

bool plan(const npas_linear_desc &d, const npas_bb_desc &bb, LinTcParams &p)
{
    if (d.x_dtype != NPAS_BF16 || bb.w_packed != NPAS_BF16) return false;
    if (bb.Bo % 16 || bb.Bi % 8 || d.I % 8 || d.O % 8) return false;
    p.M = d.M; p.I = d.I; p.O = d.O; p.Bo = bb.Bo; p.Bi = bb.Bi;
    p.L = bb_layout(bb);
    p.nBi = p.L.nBi;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    p.xt_pitch = bb.Bi * 2 + 4;
    const uint32_t kp8max = ((bb.Bi + 15) / 16) * 2;
    p.a_bytes = kp8max * kRows * 16;
    p.b_bytes = kp8max * bb.Bo * 16;
    const int nBo = p.L.nBo;
    p.BOG = 1;
    for (int g = 1; g <= nBo && g * bb.Bo <= 256; ++g) {
        if (nBo % g || (g * bb.Bo) % 32) continue;
        const uint32_t need = 2u * g * (p.a_bytes + p.b_bytes) + kRows * p.xt_pitch + 4096;
        if (need <= kSmemLimit) p.BOG = g;
    }
    if ((p.BOG * bb.Bo) % 32) return false;
    p.set_bytes = p.BOG * (p.a_bytes + p.b_bytes);
    p.off_xt = 0;
    p.off_sets = round_up(kRows * p.xt_pitch, 128);
    p.off_idx = p.off_sets + 2 * p.set_bytes;
    p.off_bar = round_up(p.off_idx + p.BOG * (bb.Bi + bb.Bo + 16), 128);
    p.smem_bytes = p.off_bar + sizeof(LinBars) + 1024;
    if (p.smem_bytes > kSmemLimit) return false;
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
                             const void *blob, const float *bias, void *y, uint32_t *ws,
                             cudaStream_t st)
{
    LinTcParams p;
    if (!plan(d, bb, p)) return NPAS_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(linear_bb_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess)
        return NPAS_ERR_CUDA;
    const dim3 grid((d.M + kRows - 1) / kRows, p.L.nBo / p.BOG);
    if (grid.y > 65535) return NPAS_ERR_UNSUPPORTED;
    linear_bb_tc_kernel<<<grid, kThreads, p.smem_bytes, st>>>(p, static_cast<const uint16_t *>(x),
                                                              static_cast<const uint8_t *>(blob), bias, y, ws);
    count_launch();
    return launch_status();
}

}  // namespace npas
