// Block-punched convolution on the sm_100a tensor cores (bf16 in, fp32 accumulation in TMEM).
//
// Formulation.  A packed block (Mb filters x Nb channels, one kept tap) is a dense [pixels x Nb] x
// [Nb x Mb] product, so the layer is a sum of small dense contractions, one per kept (channel
// block, tap) pair.  One CTA owns a tile of up to 128 output positions of one image (whole output
// rows, taken as a run of consecutive positions of the zero-padded image, "padded-linear" order)
// and a group of FG filter blocks whose fp32 accumulators live side by side in tensor memory.
//
// Shared-memory layout of the activations: [channel octet][padded-linear position][8 channels],
// i.e. one 16-byte row per position, written by ONE 5-D TMA box per pipeline stage (out-of-image
// rows and columns are zero-filled by the TMA unit and are the convolution's padding).  In this
// layout 8 consecutive positions are one 128-byte core matrix of the no-swizzle K-major operand
// format, so selecting a kept tap is pure descriptor arithmetic: the tap (r, s) only moves the
// operand's start address by (r*Wp + s) * 16 bytes and the channel block picks the plane; no
// activation is ever copied or gathered.  The two 16-byte halves of a 32-byte K slice may sit at
// any distance (the descriptor's K-direction offset), so with Nb = 8 two arbitrary kept pairs of
// a filter block form one K = 16 MMA.
//
// Roles (7 warps): warp 0 streams activation stages (TMA tensor copies), warp 1 streams packed
// weights (1-D bulk copies straight from the blob: the blob's value order IS the operand layout),
// warp 2 reads each segment's pair words with one coalesced load, broadcasts them by shuffle and
// has one lane issue the MMAs, warps 3..6 run the fused epilogue (TMEM -> registers -> bias,
// residual, ReLU -> one rounding -> 16-byte stores).  Every wait is bounded.
#include <cstdlib>

#include "common.cuh"
#include "tc_common.cuh"

#include <mutex>

namespace npas {

using namespace tc;

namespace {

constexpr int kThreads = 224;
constexpr int kMaxStages = 8;
constexpr uint32_t kSmemLimit = 232448;  // 227 KB of dynamic shared memory per CTA

struct ConvTcParams {
    int N, H, W, C, K, R, S, pad, P, Q;
    int Wp, TR, tiles_per_img, slab_rows;
    int Mb, Nb, nCB, FG, q8;
    int CBS, nChunks, PPS;
    uint32_t plane_bytes, act_stage_bytes, act_tx_bytes;
    int SA, SW;
    uint32_t wstage_bytes, wmaxp, pair_bytes;
    uint32_t tmem_cols;
    int relu, y_bf16;
    // shared-memory offsets from the 1024-aligned base
    uint32_t off_act, off_w, off_zero, off_sched, off_bar, smem_bytes;
};

struct Bars {
    uint64_t act_full[kMaxStages], act_empty[kMaxStages], w_full[kMaxStages], w_empty[kMaxStages];
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    return cvt_bf16x2(lo, hi);
}

__global__ void __launch_bounds__(kThreads, 2)
conv_bp_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const ConvTcParams p,
                  const uint8_t *__restrict__ blob, const float *__restrict__ bias,
                  const void *__restrict__ res, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *act = smem + p.off_act;
    uint8_t *wring = smem + p.off_w;
    uint32_t *zero = reinterpret_cast<uint32_t *>(smem + p.off_zero);
    uint32_t *sched = reinterpret_cast<uint32_t *>(smem + p.off_sched);
    Bars *bars = reinterpret_cast<Bars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, n = tile / p.tiles_per_img, y0 = (tile % p.tiles_per_img) * p.TR;
    const int fb0 = blockIdx.y * p.FG;

    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_BLK]);
    const uint32_t *pairs = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
    const uint8_t *values = blob + hdr[BP_OFF_VALUES];

    // ---- set-up ------------------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < p.SA; ++s) { mbar_init(&bars->act_full[s], 1); mbar_init(&bars->act_empty[s], 1); }
        for (int s = 0; s < p.SW; ++s) { mbar_init(&bars->w_full[s], 1); mbar_init(&bars->w_empty[s], 1); }
        mbar_init(&bars->acc_full, 1);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
    }
    // first pair index of every (filter block of the group, channel chunk)
    for (int i = tid; i < p.FG * (p.nChunks + 1); i += kThreads) {
        const int g = i / (p.nChunks + 1), c = i % (p.nChunks + 1);
        sched[i] = blk_off[(size_t)(fb0 + g) * p.nCB + min(c * p.CBS, p.nCB)];
    }
    for (int i = tid; i < (int)(p.Mb * 16 / 4); i += kThreads) zero[i] = 0u;
    fence_proxy_async_smem();
    if (warp == 2) tmem_alloc(&bars->tmem_base, p.tmem_cols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ---- activation producer ---------------------------------------------------------------
        if (lane == 0) {
            for (int c = 0; c < p.nChunks; ++c) {
                const int s = c % p.SA, k = c / p.SA;
                if (k >= 1 && !mbar_wait(&bars->act_empty[s], (k & 1) ^ 1, abort_flag, ws, 0x100 + c)) break;
                mbar_arrive_expect_tx(&bars->act_full[s], p.act_tx_bytes);
                tma_load_5d(act + (size_t)s * p.act_stage_bytes, &tmap_x, &bars->act_full[s], 0, -p.pad,
                            y0 - p.pad, c * p.PPS, n);
            }
        }
    } else if (warp == 1) {
        // ---- weight producer -------------------------------------------------------------------
        if (lane == 0) {
            uint32_t seg = 0;
            bool ok = true;
            for (int c = 0; c < p.nChunks && ok; ++c)
                for (int g = 0; g < p.FG && ok; ++g) {
                    const uint32_t lo = sched[g * (p.nChunks + 1) + c], hi = sched[g * (p.nChunks + 1) + c + 1];
                    for (uint32_t s0 = lo; s0 < hi; s0 += p.wmaxp, ++seg) {
                        const uint32_t np = min(p.wmaxp, hi - s0), st = seg % p.SW, k = seg / p.SW;
                        if (k >= 1 && !mbar_wait(&bars->w_empty[st], (k & 1) ^ 1, abort_flag, ws, 0x200)) { ok = false; break; }
                        mbar_arrive_expect_tx(&bars->w_full[st], np * p.pair_bytes);
                        bulk_load_1d(wring + (size_t)st * p.wstage_bytes, values + (size_t)s0 * p.pair_bytes,
                                     np * p.pair_bytes, &bars->w_full[st]);
                    }
                }
        }
    } else if (warp == 2) {
        // ---- MMA issue ---------------------------------------------------------------------------
        const uint32_t idesc = idesc_bf16_f32(128, p.Mb);
        const uint32_t act_u32 = smem_u32(act), w_u32 = smem_u32(wring), zero_u32 = smem_u32(zero);
        uint32_t seg = 0, touched = 0;
        bool ok = true;
        for (int c = 0; c < p.nChunks && ok; ++c) {
            const int s = c % p.SA;
            if (!mbar_wait(&bars->act_full[s], (c / p.SA) & 1, abort_flag, ws, 0x300 + c)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t a_stage = act_u32 + s * p.act_stage_bytes;
            for (int g = 0; g < p.FG && ok; ++g) {
                const uint32_t lo = sched[g * (p.nChunks + 1) + c], hi = sched[g * (p.nChunks + 1) + c + 1];
                const uint32_t d_tmem = tmem_base + g * p.Mb;
                for (uint32_t s0 = lo; s0 < hi; s0 += p.wmaxp, ++seg) {
                    const uint32_t np = min(p.wmaxp, hi - s0), st = seg % p.SW;
                    // one coalesced read of the segment's pair words; wmaxp <= 32
                    uint32_t a_off = 0;
                    if ((uint32_t)lane < np) {
                        const uint32_t pw = pairs[s0 + lane];
                        const uint32_t cbl = (pw & 0xFFFFu) - c * p.CBS, tap = pw >> 16;
                        a_off = cbl * p.q8 * p.plane_bytes + ((tap / p.S) * p.Wp + (tap % p.S)) * 16u;
                    }
                    if (!mbar_wait(&bars->w_full[st], (seg / p.SW) & 1, abort_flag, ws, 0x400)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t b_stage = w_u32 + st * p.wstage_bytes;
                    if (p.Nb == 8) {
                        for (uint32_t i = 0; i < np; i += 2) {
                            const bool two = i + 1 < np;
                            const uint32_t a0 = __shfl_sync(0xFFFFFFFFu, a_off, i);
                            const uint32_t a1 = __shfl_sync(0xFFFFFFFFu, a_off, two ? i + 1 : i);
                            if (lane == 0) {
                                const uint32_t b0 = b_stage + i * p.pair_bytes;
                                const uint64_t ad = smem_desc_kmajor(a_stage + a0, a1 - a0, 128);
                                const uint64_t bd = smem_desc_kmajor(b0, two ? p.pair_bytes : zero_u32 - b0, 128);
                                mma_bf16_ss(d_tmem, ad, bd, idesc, (touched >> g) & 1u);
                            }
                            touched |= 1u << g;
                        }
                    } else {
                        for (uint32_t i = 0; i < np; ++i) {
                            const uint32_t a0 = __shfl_sync(0xFFFFFFFFu, a_off, i);
                            if (lane == 0) {
                                for (int kk = 0; kk < p.q8 / 2; ++kk) {
                                    const uint64_t ad = smem_desc_kmajor(a_stage + a0 + 2 * kk * p.plane_bytes, p.plane_bytes, 128);
                                    const uint64_t bd = smem_desc_kmajor(b_stage + i * p.pair_bytes + 2 * kk * p.Mb * 16, p.Mb * 16, 128);
                                    mma_bf16_ss(d_tmem, ad, bd, idesc, ((touched >> g) & 1u) | (kk > 0));
                                }
                            }
                            touched |= 1u << g;
                        }
                    }
                    if (lane == 0) mma_commit(&bars->w_empty[st]);
                    __syncwarp();
                }
            }
            if (ok && lane == 0) mma_commit(&bars->act_empty[s]);
            __syncwarp();
        }
        if (ok && lane == 0) mma_commit(&bars->acc_full);
        __syncwarp();
    } else {
        // ---- epilogue --------------------------------------------------------------------------------
        const int quarter = warp & 3, m = quarter * 32 + lane;
        const int oy = m / p.Wp, ox = m % p.Wp, yy = y0 + oy;
        const bool valid = oy < p.TR && yy < p.P && ox < p.Q;
        const int k0 = fb0 * p.Mb;
        const size_t o0 = (((size_t)n * p.P + yy) * p.Q + ox) * p.K + k0;
        if (mbar_wait(&bars->acc_full, 0, abort_flag, ws, 0x500)) {
            tc_fence_after_sync();
            for (int c0 = 0; c0 < p.FG * p.Mb; c0 += 16) {
                const int g = c0 / p.Mb;
                uint32_t r[16];
                __syncwarp();
                tmem_ld_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_ld_wait();
                if (!valid) continue;
                const bool has = sched[g * (p.nChunks + 1) + p.nChunks] > sched[g * (p.nChunks + 1)];
                float v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    v[i] = has ? __uint_as_float(r[i]) : 0.f;
                    if (bias) v[i] += __ldg(bias + k0 + c0 + i);
                }
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
                    yp[0] = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
                    yp[1] = make_uint4(pack_bf16x2(v[8], v[9]), pack_bf16x2(v[10], v[11]), pack_bf16x2(v[12], v[13]), pack_bf16x2(v[14], v[15]));
                } else {
                    float4 *yp = reinterpret_cast<float4 *>(static_cast<float *>(y) + o0 + c0);
#pragma unroll
                    for (int h = 0; h < 4; ++h) yp[h] = make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]);
                }
            }
        }
    }

    // ---- tear-down ---------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        // a role gave up: leave time for copies still in flight to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) { }
        __syncthreads();
    }
    if (warp == 2) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

bool plan(const npas_conv_desc &d, const npas_bp_desc &bp, ConvTcParams &p)
{
    if (d.x_dtype != NPAS_BF16 || bp.w_packed != NPAS_BF16) return false;
    if (d.stride != 1 || d.pad < 0 || d.pad >= d.R + 1) return false;
    if (bp.Nb % 8 || bp.Mb % 16 || bp.Mb > 256 || d.C % 8 || d.K % 8) return false;
    if (bp.Nb != 8 && bp.Nb % 16) return false;
    p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C; p.K = d.K; p.R = d.R; p.S = d.S; p.pad = d.pad;
    p.P = d.H + 2 * d.pad - d.R + 1; p.Q = d.W + 2 * d.pad - d.S + 1;
    if (p.P < 1 || p.Q < 1) return false;
    p.Wp = d.W + 2 * d.pad;
    if (p.Wp > 128) return false;
    p.TR = min(p.P, 128 / p.Wp);
    p.tiles_per_img = (p.P + p.TR - 1) / p.TR;
    p.slab_rows = p.TR + d.R - 1;
    if (p.slab_rows > 256 || p.TR * p.Wp <= d.S - 1) return false;
    p.Mb = bp.Mb; p.Nb = bp.Nb; p.nCB = d.C / bp.Nb; p.q8 = bp.Nb / 8;
    const int nFB = d.K / bp.Mb;
    p.FG = 1;
    for (int f = 1; f <= nFB && f <= 32; ++f)
        if (nFB % f == 0 && f * bp.Mb <= 256) p.FG = f;
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < p.FG * p.Mb) p.tmem_cols *= 2;
    p.CBS = max(1, 8 / p.q8);
    p.PPS = p.CBS * p.q8;
    if (p.PPS > 256) return false;
    p.nChunks = (p.nCB + p.CBS - 1) / p.CBS;
    if (p.FG * (p.nChunks + 1) > 4096) return false;
    p.plane_bytes = (uint32_t)p.slab_rows * p.Wp * 16u;
    p.act_tx_bytes = p.plane_bytes * p.PPS;
    p.act_stage_bytes = round_up(p.act_tx_bytes, 128);
    p.pair_bytes = (uint32_t)bp.Mb * bp.Nb * 2u;
    p.wstage_bytes = max(8192u, p.pair_bytes);
    if (p.wstage_bytes > 65536) return false;
    p.wmaxp = min(32u, p.wstage_bytes / p.pair_bytes);
    if (bp.Nb == 8 && (p.wmaxp & 1)) return false;
    p.SW = 4;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    // rows 0..127 of an operand may reach this far past the start of the last plane of a stage
    const uint32_t reach = (128u + (d.R - 1) * p.Wp + d.S) * 16u;
    const uint32_t slack = reach > p.plane_bytes ? round_up(reach - p.plane_bytes, 128) : 0u;
    for (p.SA = min(4, p.nChunks); p.SA >= 1; --p.SA) {
        p.off_act = 0;
        p.off_w = round_up(p.off_act + p.SA * p.act_stage_bytes + slack, 128);
        p.off_zero = p.off_w + p.SW * p.wstage_bytes;
        p.off_sched = p.off_zero + round_up(p.Mb * 16, 128);
        p.off_bar = round_up(p.off_sched + 4 * p.FG * (p.nChunks + 1), 128);
        p.smem_bytes = p.off_bar + sizeof(Bars) + 1024;
        // two CTAs per SM when they fit, so that one CTA's epilogue overlaps the other's main loop
        if (p.smem_bytes <= kSmemLimit / 2 || (p.SA <= 2 && p.smem_bytes <= kSmemLimit)) break;
    }
    if (p.SA < 1 || p.smem_bytes > kSmemLimit) return false;
    // the K-direction offsets of the descriptors are 14-bit counts of 16 bytes
    if (p.plane_bytes * (uint32_t)p.PPS >= (1u << 18) || p.SW * p.wstage_bytes + 4096 >= (1u << 18)) return false;
    return true;
}

}  // namespace

bool conv_tc_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvTcParams p;
    return plan(d, bp, p);
}

npas_status conv_tc_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st)
{
    ConvTcParams p;
    if (!plan(d, bp, p)) return NPAS_ERR_UNSUPPORTED;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return NPAS_ERR_CUDA;
    // X[N][H][W][C] bf16 seen as (8 channels, W, H, C/8, N): a box is then written to shared
    // memory as [octet][row][column][8 channels]
    CUtensorMap tmap;
    const cuuint64_t dims[5] = {8, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)(d.C / 8), (cuuint64_t)d.N};
    const cuuint64_t strides[4] = {(cuuint64_t)d.C * 2, (cuuint64_t)d.W * d.C * 2, 16, (cuuint64_t)d.H * d.W * d.C * 2};
    const cuuint32_t box[5] = {8, (cuuint32_t)p.Wp, (cuuint32_t)p.slab_rows, (cuuint32_t)p.PPS, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return NPAS_ERR_CUDA;
    if (allow_dynamic_smem(reinterpret_cast<const void *>(conv_bp_tc_kernel), (int)kSmemLimit) != NPAS_OK) return NPAS_ERR_CUDA;
    const dim3 grid(d.N * p.tiles_per_img, (d.K / bp.Mb) / p.FG);
    if (grid.y > 65535) return NPAS_ERR_UNSUPPORTED;
    conv_bp_tc_kernel<<<grid, kThreads, p.smem_bytes, st>>>(tmap, p, static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return launch_status();
}

}  // namespace npas
