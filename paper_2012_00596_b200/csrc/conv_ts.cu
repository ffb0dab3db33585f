// Block-punched convolution on the sm_100a tensor cores with the activation operand in TENSOR
// MEMORY (bf16 in, fp32 accumulation).
//
// Why: one packed block is an M=128 (pixels) x N=Mb (filters) x K=16 MMA.  With both operands in
// shared memory such an MMA cannot retire faster than its 4 KB activation operand is fetched
// (measured on B200: ~39 cycles for N=16 against 8 cycles of tensor math).  But the activation
// slice of a (16-channel chunk, tap) is the SAME for every filter block that keeps the tap.  So
// this kernel copies each slice ONCE from shared memory into tensor memory (tcgen05.cp; the copy
// applies the tap shift and picks the channel planes through its descriptor) and every filter
// block's MMA then reads A from TMEM and only its small packed-weight tile from shared memory
// (measured: 13 cycles per N=16 MMA with four issuing warps, full math rate from N=32 on).
//
// Tile / layout: as in the shared-memory-operand kernel, a CTA owns up to 128 consecutive
// "padded-linear" output positions of one image and FG filter blocks (<= 256 fp32 accumulator
// columns); activations are staged by one 5-D TMA box per 64 channels as
// [channel octet][padded position][8 channels] with the TMA unit's zero fill as padding.
//
// Pipeline (7 warps): warp 0 streams activation stages; warp 1 streams packed weights (1-D bulk
// copies of each (chunk, filter block) run of pairs straight from the blob); warp 2 copies the
// kept-tap slices of one 16/32-channel chunk into one of two TMEM staging buffers; warps 3..6
// issue the MMAs from a per-CTA list of MMA records (built once in shared memory from the blob's
// pair list: staging column, weight offsets), filter block g by warp g mod 4, because one thread
// can issue only one MMA per ~51 cycles; the same four warps then run the fused epilogue.  With Nb = 8 a
// K=16 MMA spans two channel blocks at one tap; a block that does not keep the tap contributes a
// zero weight tile for its half.  Accumulators are zeroed up front (tcgen05.st), so every MMA
// accumulates.  Every wait is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kThreads = 224;
constexpr int kMaxStages = 8;
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kZeroFlag = 0x8000u;

struct ConvTsParams {
    int N, H, W, C, K, R, S, pad, P, Q;
    int Wp, TR, tiles_per_img, slab_rows;
    int Mb, Nb, nCB, FG, RS;
    int CCH, KS, nChunks, chunks_per_stage, nStages, PPS, cbs_per_chunk;
    int GS, nSlotsPerChunk, maxrec, maxpairs;
    uint32_t plane_bytes, act_stage_bytes, act_tx_bytes;
    int SA, NW;
    uint32_t pair_bytes, seg_bytes, wslot_bytes, bufcols;
    int relu, y_bf16;
    uint32_t off_act, off_zero_lo, off_w, off_zero_hi, off_sched, off_mask, off_cnt, off_rec, off_bar, smem_bytes;
};

struct Bars {
    uint64_t act_full[kMaxStages], act_empty[kMaxStages], w_full[kMaxStages], w_empty[kMaxStages];
    uint64_t a_full[2], a_empty[2];
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

struct __align__(8) Rec { uint16_t a_col, pad, b0, b1; };

__device__ __forceinline__ void tmem_cp_128x256b(uint32_t taddr, uint64_t sdesc)
{
    asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// D[tmem] += A[tmem] * B[smem]
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc) : "memory");
}
__device__ __forceinline__ void tmem_st_zero_x16(uint32_t taddr)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                 ::"r"(taddr), "r"(0u) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    return (uint32_t)f32_bits_to_bf16(__float_as_uint(lo)) | ((uint32_t)f32_bits_to_bf16(__float_as_uint(hi)) << 16);
}

__global__ void __launch_bounds__(kThreads, 1)
conv_bp_ts_kernel(const __grid_constant__ CUtensorMap tmap_x, const ConvTsParams p,
                  const uint8_t *__restrict__ blob, const float *__restrict__ bias,
                  const void *__restrict__ res, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *act = smem + p.off_act;
    uint8_t *wring = smem + p.off_w;
    uint32_t *sched = reinterpret_cast<uint32_t *>(smem + p.off_sched);   // [FG][nCB+1] first pair of each block
    uint32_t *tmask = reinterpret_cast<uint32_t *>(smem + p.off_mask);    // [FG][nCB] kept-tap bitsets
    uint8_t *cnt = smem + p.off_cnt;                                      // [nChunks][FG] MMA records per segment
    Rec *recs = reinterpret_cast<Rec *>(smem + p.off_rec);                // [nChunks][FG][maxrec]
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
        for (int s = 0; s < p.NW; ++s) { mbar_init(&bars->w_full[s], 1); mbar_init(&bars->w_empty[s], min(p.GS, 4)); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bars->a_full[b], 1); mbar_init(&bars->a_empty[b], 4); }
        mbar_init(&bars->acc_full, 4);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
    }
    for (int i = tid; i < (int)(p.Mb * 16 / 4); i += kThreads) {
        reinterpret_cast<uint32_t *>(smem + p.off_zero_lo)[i] = 0u;
        reinterpret_cast<uint32_t *>(smem + p.off_zero_hi)[i] = 0u;
    }
    // kept-tap bitset and first pair index of every block of this CTA's filter group
    for (int i = tid; i < p.FG * p.nCB; i += kThreads) {
        const int g = i / p.nCB, cb = i % p.nCB;
        const uint32_t lo = blk_off[(size_t)(fb0 + g) * p.nCB + cb], hi = blk_off[(size_t)(fb0 + g) * p.nCB + cb + 1];
        uint32_t bits = 0;
        for (uint32_t j = lo; j < hi; ++j) bits |= 1u << (pairs[j] >> 16);
        tmask[i] = bits;
        sched[g * (p.nCB + 1) + cb] = lo;
        if (cb == p.nCB - 1) sched[g * (p.nCB + 1) + p.nCB] = hi;
    }
    fence_proxy_async_smem();
    if (warp == 2) tmem_alloc(&bars->tmem_base, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    // MMA records of every (chunk, filter block) segment
    for (int i = tid; i < p.nChunks * p.FG; i += kThreads) {
        const int c = i / p.FG, g = i % p.FG;
        Rec *out = recs + (size_t)i * p.maxrec;
        const uint32_t pb16 = p.pair_bytes / 16;
        int r = 0;
        if (p.Nb == 8) {
            const uint32_t T0 = tmask[g * p.nCB + 2 * c], T1 = tmask[g * p.nCB + 2 * c + 1], n0 = __popc(T0);
            for (uint32_t U = T0 | T1; U; U &= U - 1) {
                const uint32_t t = __ffs(U) - 1, below = (1u << t) - 1u;
                Rec rec;
                rec.a_col = (uint16_t)(t * 8); rec.pad = 0;
                rec.b0 = (T0 >> t) & 1u ? (uint16_t)(__popc(T0 & below) * pb16) : (uint16_t)kZeroFlag;
                rec.b1 = (T1 >> t) & 1u ? (uint16_t)((n0 + __popc(T1 & below)) * pb16) : (uint16_t)kZeroFlag;
                out[r++] = rec;
            }
        } else {
            const uint32_t T = tmask[g * p.nCB + c];
            for (uint32_t U = T; U; U &= U - 1) {
                const uint32_t t = __ffs(U) - 1, idx = __popc(T & ((1u << t) - 1u));
                for (int ks = 0; ks < p.KS; ++ks) {
                    Rec rec;
                    rec.a_col = (uint16_t)((t * p.KS + ks) * 8); rec.pad = 0;
                    rec.b0 = (uint16_t)(idx * pb16 + ks * 2 * p.Mb);
                    rec.b1 = (uint16_t)(rec.b0 + p.Mb);
                    out[r++] = rec;
                }
            }
        }
        cnt[i] = (uint8_t)r;
    }
    // zero the accumulators (warps 3..6 own the four lane quarters)
    if (warp >= 3) {
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        for (int c0 = 0; c0 < p.FG * p.Mb; c0 += 16) tmem_st_zero_x16(tmem_base + lane_base + c0);
        tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    if (warp == 0) {
        // ---- activation producer ---------------------------------------------------------------
        if (lane == 0) {
            for (int s = 0; s < p.nStages; ++s) {
                const int st = s % p.SA, k = s / p.SA;
                if (k >= 1 && !mbar_wait(&bars->act_empty[st], (k & 1) ^ 1, abort_flag, ws, 0x1100 + s)) break;
                mbar_arrive_expect_tx(&bars->act_full[st], p.act_tx_bytes);
                tma_load_5d(act + (size_t)st * p.act_stage_bytes, &tmap_x, &bars->act_full[st], 0, -p.pad,
                            y0 - p.pad, s * p.PPS, n);
            }
        }
    } else if (warp == 1) {
        // ---- weight producer: one ring slot per (chunk, GS filter blocks) ------------------------
        if (lane == 0) {
            uint32_t slot = 0;
            bool ok = true;
            for (int c = 0; c < p.nChunks && ok; ++c) {
                const int cb_lo = c * p.cbs_per_chunk, cb_hi = cb_lo + p.cbs_per_chunk;
                for (int q = 0; q < p.nSlotsPerChunk; ++q, ++slot) {
                    const uint32_t st = slot % p.NW, k = slot / p.NW;
                    if (k >= 1 && !mbar_wait(&bars->w_empty[st], (k & 1) ^ 1, abort_flag, ws, 0x1200)) { ok = false; break; }
                    uint32_t total = 0;
                    for (int gi = 0; gi < p.GS; ++gi) {
                        const int g = q * p.GS + gi;
                        total += (sched[g * (p.nCB + 1) + cb_hi] - sched[g * (p.nCB + 1) + cb_lo]) * p.pair_bytes;
                    }
                    if (total == 0) { mbar_arrive(&bars->w_full[st]); continue; }
                    mbar_arrive_expect_tx(&bars->w_full[st], total);
                    for (int gi = 0; gi < p.GS; ++gi) {
                        const int g = q * p.GS + gi;
                        const uint32_t lo = sched[g * (p.nCB + 1) + cb_lo], hi = sched[g * (p.nCB + 1) + cb_hi];
                        if (hi > lo)
                            bulk_load_1d(wring + (size_t)st * p.wslot_bytes + (size_t)gi * p.seg_bytes,
                                         values + (size_t)lo * p.pair_bytes, (hi - lo) * p.pair_bytes, &bars->w_full[st]);
                    }
                }
            }
        }
    } else if (warp == 2) {
        // ---- stager: copy the tap-shifted slices of each chunk from shared memory into TMEM ------
        if (lane == 0) {
            const uint32_t act_u32 = smem_u32(act);
            bool ok = true;
            for (int c = 0; c < p.nChunks && ok; ++c) {
                const int s = c / p.chunks_per_stage, st = s % p.SA, b = c & 1, kb = c >> 1;
                if (c % p.chunks_per_stage == 0) {
                    if (!mbar_wait(&bars->act_full[st], (s / p.SA) & 1, abort_flag, ws, 0x1300 + s)) { ok = false; break; }
                }
                if (kb >= 1 && !mbar_wait(&bars->a_empty[b], (kb & 1) ^ 1, abort_flag, ws, 0x1400 + c)) { ok = false; break; }
                tc_fence_after_sync();
                // taps that at least one filter block of the group keeps in this chunk
                uint32_t used = 0;
                for (int g = 0; g < p.FG; ++g)
                    for (int q = 0; q < p.cbs_per_chunk; ++q) used |= tmask[g * p.nCB + c * p.cbs_per_chunk + q];
                const uint32_t plane0 = act_u32 + st * p.act_stage_bytes +
                                        (uint32_t)(c % p.chunks_per_stage) * (p.CCH / 8) * p.plane_bytes;
                const uint32_t tbuf = tmem_base + 256 + b * p.bufcols;
                for (; used; used &= used - 1) {
                    const uint32_t t = __ffs(used) - 1;
                    const uint32_t shift = ((t / p.S) * p.Wp + (t % p.S)) * 16u;
                    for (int ks = 0; ks < p.KS; ++ks)
                        tmem_cp_128x256b(tbuf + (t * p.KS + ks) * 8,
                                         smem_desc_kmajor(plane0 + 2 * ks * p.plane_bytes + shift, p.plane_bytes, 128));
                }
                mma_commit(&bars->a_full[b]);
                if (c % p.chunks_per_stage == p.chunks_per_stage - 1 || c == p.nChunks - 1) mma_commit(&bars->act_empty[st]);
            }
        }
    } else {
        // ---- MMA issue: filter block g belongs to warp g mod 4, so every accumulator receives its
        // MMAs from one thread in program order (bitwise reproducible results) ----------------------
        const int wq = warp - 3;
        const uint32_t idesc = idesc_bf16_f32(128, p.Mb);
        const uint32_t w_u32 = smem_u32(wring), zlo = smem_u32(smem + p.off_zero_lo), zhi = smem_u32(smem + p.off_zero_hi);
        uint32_t slot = 0;
        bool ok = true;
        for (int c = 0; c < p.nChunks && ok; ++c) {
            const int b = c & 1;
            if (!mbar_wait(&bars->a_full[b], (c >> 1) & 1, abort_flag, ws, 0x1500 + c)) { ok = false; break; }
            const uint32_t tbuf = tmem_base + 256 + b * p.bufcols;
            for (int q = 0; q < p.nSlotsPerChunk && ok; ++q, ++slot) {
                // first filter block of this slot that is mine (slots hold GS consecutive blocks)
                const int gi0 = (wq - q * p.GS) & 3;
                if (gi0 >= p.GS) continue;
                const uint32_t st = slot % p.NW;
                if (!mbar_wait(&bars->w_full[st], (slot / p.NW) & 1, abort_flag, ws, 0x1600)) { ok = false; break; }
                tc_fence_after_sync();
                if (lane == 0) {
                    for (int gi = gi0; gi < p.GS; gi += 4) {
                        const int g = q * p.GS + gi;
                        const int nrec = cnt[c * p.FG + g];
                        const Rec *rr = recs + (size_t)(c * p.FG + g) * p.maxrec;
                        const uint32_t seg = w_u32 + st * p.wslot_bytes + gi * p.seg_bytes;
                        const uint32_t d_tmem = tmem_base + g * p.Mb;
                        for (int r = 0; r < nrec; ++r) {
                            const Rec rec = rr[r];
                            const uint32_t h0 = rec.b0 & kZeroFlag ? zlo : seg + (uint32_t)rec.b0 * 16u;
                            const uint32_t h1 = rec.b1 & kZeroFlag ? zhi : seg + (uint32_t)rec.b1 * 16u;
                            mma_bf16_ts(d_tmem, tbuf + rec.a_col, smem_desc_kmajor(h0, h1 - h0, 128), idesc);
                        }
                    }
                    mma_commit(&bars->w_empty[st]);
                }
                __syncwarp();
            }
            if (ok && lane == 0) mma_commit(&bars->a_empty[b]);
            __syncwarp();
        }
        if (ok && lane == 0) mma_commit(&bars->acc_full);
        __syncwarp();

        // ---- fused epilogue ------------------------------------------------------------------------
        const int quarter = warp & 3, m = quarter * 32 + lane;
        const int oy = m / p.Wp, ox = m % p.Wp, yy = y0 + oy;
        const bool valid = oy < p.TR && yy < p.P && ox < p.Q;
        const int k0 = fb0 * p.Mb;
        const size_t o0 = (((size_t)n * p.P + yy) * p.Q + ox) * p.K + k0;
        if (ok && mbar_wait(&bars->acc_full, 0, abort_flag, ws, 0x1700)) {
            tc_fence_after_sync();
            for (int c0 = 0; c0 < p.FG * p.Mb; c0 += 16) {
                uint32_t r[16];
                __syncwarp();
                tmem_ld_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_ld_wait();
                if (!valid) continue;
                float v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    v[i] = __uint_as_float(r[i]);
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
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) { }
        __syncthreads();
    }
    if (warp == 2) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

bool plan(const npas_conv_desc &d, const npas_bp_desc &bp, ConvTsParams &p)
{
    if (d.x_dtype != NPAS_BF16 || bp.w_packed != NPAS_BF16) return false;
    if (d.stride != 1 || d.pad < 0) return false;
    if (bp.Nb != 8 && bp.Nb != 16 && bp.Nb != 32) return false;
    if (bp.Mb % 16 || bp.Mb > 256 || d.C % 16 || d.K % 8) return false;
    p.RS = d.R * d.S;
    p.CCH = bp.Nb < 16 ? 16 : bp.Nb;
    p.KS = p.CCH / 16;
    if (p.RS * p.KS > 16 || d.C % p.CCH) return false;
    p.bufcols = (uint32_t)p.RS * p.KS * 8;
    p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C; p.K = d.K; p.R = d.R; p.S = d.S; p.pad = d.pad;
    p.P = d.H + 2 * d.pad - d.R + 1; p.Q = d.W + 2 * d.pad - d.S + 1;
    if (p.P < 1 || p.Q < 1) return false;
    p.Wp = d.W + 2 * d.pad;
    if (p.Wp > 128) return false;
    p.TR = min(p.P, 128 / p.Wp);
    p.tiles_per_img = (p.P + p.TR - 1) / p.TR;
    p.slab_rows = p.TR + d.R - 1;
    if (p.slab_rows > 256 || p.TR * p.Wp <= d.S - 1) return false;
    p.Mb = bp.Mb; p.Nb = bp.Nb; p.nCB = d.C / bp.Nb;
    p.cbs_per_chunk = bp.Nb == 8 ? 2 : 1;
    p.nChunks = d.C / p.CCH;
    p.chunks_per_stage = max(1, 64 / p.CCH);
    p.PPS = p.chunks_per_stage * p.CCH / 8;
    p.nStages = (p.nChunks + p.chunks_per_stage - 1) / p.chunks_per_stage;
    p.maxpairs = p.RS * p.cbs_per_chunk;
    p.maxrec = p.RS * p.KS;
    p.pair_bytes = (uint32_t)bp.Mb * bp.Nb * 2u;
    p.seg_bytes = (uint32_t)p.maxpairs * p.pair_bytes;
    const int nFB = d.K / bp.Mb;
    const int tiles = d.N * p.tiles_per_img;
    // filter blocks per CTA: as many as the accumulator columns allow, fewer when that leaves SMs idle
    int best = 0;
    double best_cost = 0;
    for (int f = 1; f <= nFB; ++f) {
        if (nFB % f || f * bp.Mb > 256 || (uint32_t)(f * bp.Mb) + 2 * p.bufcols > 512u) continue;
        const double per_chunk = fmax(p.RS * p.KS * 40.0, f * (p.RS * p.KS / 2.5) * 14.0);
        const double cta = 4000.0 + p.nChunks * per_chunk + f * bp.Mb * 12.0;
        const double waves = ceil((double)tiles * (nFB / f) / 148.0);
        const double cost = waves * cta;
        if (!best || cost < best_cost) { best = f; best_cost = cost; }
    }
    if (!best) return false;
    p.FG = best;
    p.GS = 1;
    for (int g = 1; g <= p.FG; ++g)
        if (p.FG % g == 0 && (uint32_t)g * p.seg_bytes <= 20480u) p.GS = g;
    p.nSlotsPerChunk = p.FG / p.GS;
    p.wslot_bytes = round_up((uint32_t)p.GS * p.seg_bytes, 128);
    if (p.wslot_bytes > 65536u || p.wslot_bytes / 16 >= kZeroFlag) return false;
    p.plane_bytes = (uint32_t)p.slab_rows * p.Wp * 16u;
    p.act_tx_bytes = p.plane_bytes * p.PPS;
    p.act_stage_bytes = round_up(p.act_tx_bytes, 128);
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    if ((uint32_t)p.FG * (p.nCB + 1) > 8192u || (uint32_t)p.nChunks * p.FG * p.maxrec * 8u > 80u * 1024u) return false;
    const uint32_t reach = (128u + (d.R - 1) * p.Wp + d.S) * 16u;
    const uint32_t slack = reach > p.plane_bytes ? round_up(reach - p.plane_bytes, 128) : 0u;
    p.NW = 4;
    for (p.SA = min(3, p.nStages); p.SA >= 1; --p.SA) {
        p.off_act = 0;
        p.off_zero_lo = round_up(p.off_act + p.SA * p.act_stage_bytes + slack, 128);
        p.off_w = p.off_zero_lo + round_up(p.Mb * 16, 128);
        p.off_zero_hi = p.off_w + p.NW * p.wslot_bytes;
        p.off_sched = p.off_zero_hi + round_up(p.Mb * 16, 128);
        p.off_mask = round_up(p.off_sched + 4 * p.FG * (p.nCB + 1), 128);
        p.off_cnt = round_up(p.off_mask + 4 * p.FG * p.nCB, 128);
        p.off_rec = round_up(p.off_cnt + p.nChunks * p.FG, 128);
        p.off_bar = round_up(p.off_rec + (uint32_t)p.nChunks * p.FG * p.maxrec * 8u, 128);
        p.smem_bytes = p.off_bar + sizeof(Bars) + 1024;
        if (p.smem_bytes <= kSmemLimit) break;
    }
    if (p.SA < 1 || p.smem_bytes > kSmemLimit) return false;
    if (p.plane_bytes * (uint32_t)p.PPS >= (1u << 18) || p.off_zero_hi - p.off_zero_lo + 4096 >= (1u << 18)) return false;
    return true;
}

}  // namespace

bool conv_ts_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvTsParams p;
    return plan(d, bp, p);
}

npas_status conv_ts_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st)
{
    ConvTsParams p;
    if (!plan(d, bp, p)) return NPAS_ERR_UNSUPPORTED;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return NPAS_ERR_CUDA;
    CUtensorMap tmap;
    const cuuint64_t dims[5] = {8, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)(d.C / 8), (cuuint64_t)d.N};
    const cuuint64_t strides[4] = {(cuuint64_t)d.C * 2, (cuuint64_t)d.W * d.C * 2, 16, (cuuint64_t)d.H * d.W * d.C * 2};
    const cuuint32_t box[5] = {8, (cuuint32_t)p.Wp, (cuuint32_t)p.slab_rows, (cuuint32_t)p.PPS, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return NPAS_ERR_CUDA;
    if (cudaFuncSetAttribute(conv_bp_ts_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess)
        return NPAS_ERR_CUDA;
    const dim3 grid(d.N * p.tiles_per_img, (d.K / bp.Mb) / p.FG);
    if (grid.y > 65535) return NPAS_ERR_UNSUPPORTED;
    conv_bp_ts_kernel<<<grid, kThreads, p.smem_bytes, st>>>(tmap, p, static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return launch_status();
}

}  // namespace npas
