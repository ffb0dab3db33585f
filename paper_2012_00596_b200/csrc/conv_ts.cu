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
// (measured: ~9 cycles per N=16 MMA with eight issuing warps, full math rate from N=32 on).
//
// Tile / layout: as in the shared-memory-operand kernel, a CTA owns up to 128 consecutive
// "padded-linear" output positions of one image and FG filter blocks (<= 256 fp32 accumulator
// columns); activations are staged by one 5-D TMA box per 64 channels as
// [channel octet][padded position][8 channels] with the TMA unit's zero fill as padding.
//
// Pipeline (11 warps): warp 0 streams activation stages; warp 1 streams packed weights, one ring
// slot per (chunk, run of filter blocks), every lane issuing the 1-D bulk copy of one filter
// block's run of pairs straight from the blob (the blob's value order IS the operand layout);
// warp 2 copies the kept-tap slices of one 16/32-channel chunk into one of up to three TMEM
// staging buffers; warps 3..10 issue the MMAs.  Scalar work in a single thread is the scarce
// resource here (an integer division or a dependent shared-memory load costs 50..70 cycles, one
// thread issues at most one MMA per ~51 cycles), so everything data dependent is computed ONCE
// per CTA, in parallel, before the main loop: per-block tap bitsets, the packing of each chunk's
// weight runs into ring slots, the set of taps each chunk needs, and one 8-byte record per MMA
// (staging column + ready-made low descriptor word relative to the ring slot).  The main loops
// only add a base to a table entry.  Filter block g is always issued by warp g mod 8, so each
// accumulator gets its MMAs from one thread in program order and results are bitwise
// reproducible.  With Nb = 8 a K=16 MMA spans two channel blocks at one tap; a block that does
// not keep the tap contributes the zero tile kept at the head / tail of every weight slot.
// Accumulators are zeroed up front, so every MMA accumulates.  The eight MMA warps then run the
// fused epilogue.  Every wait is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kMmaWarps = 8;
constexpr int kThreads = (3 + kMmaWarps) * 32;
constexpr int kMaxStages = 8;
constexpr int kMaxABufs = 3;
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kDescHi = (128u >> 4) | (1u << 14);   // SBO = 128 bytes, descriptor version bit

struct ConvTsParams {
    int N, H, W, C, K, R, S, pad, P, Q;
    int Wp, TR, tiles_per_img, slab_rows;
    int Mb, Nb, nCB, FG, RS;
    int CCH, KS, nChunks, chunks_per_stage, nStages, PPS, cbs_per_chunk;
    int maxrec, nabuf;
    uint32_t plane_bytes, act_stage_bytes, act_tx_bytes;
    int SA, NW;
    uint32_t pair_bytes, zb, wcap, bufcols;
    int relu, y_bf16;
    uint32_t off_act, off_w, off_sched, off_mask, off_segoff, off_segslot, off_slotbase, off_used, off_cnt, off_rec,
        off_tap, off_bar, smem_bytes;
};

struct Bars {
    uint64_t act_full[kMaxStages], act_empty[kMaxStages], w_full[kMaxStages], w_empty[kMaxStages];
    uint64_t a_full[kMaxABufs], a_empty[kMaxABufs];
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

// One MMA: lo = low word of the B descriptor relative to the ring slot (start >> 4 in bits 0..13,
// K-direction offset >> 4 in bits 16..29), a_col = column of the A slice inside the staging buffer.
struct __align__(8) Rec { uint32_t lo; uint32_t a_col; };

__device__ __forceinline__ void tmem_cp_128x256b(uint32_t taddr, uint32_t desc_lo)
{
    asm volatile(
        "{\n\t.reg .b64 d;\n\tmov.b64 d, {%1, %2};\n\t"
        "tcgen05.cp.cta_group::1.128x256b [%0], d;\n\t}" ::"r"(taddr), "r"(desc_lo), "r"(kDescHi));
}
// D[tmem] += A[tmem] * B[smem]
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 d;\n\tsetp.ne.b32 p, 1, 0;\n\tmov.b64 d, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], d, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(kDescHi), "r"(idesc));
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
    uint32_t *sched = reinterpret_cast<uint32_t *>(smem + p.off_sched);       // [FG][nCB+1] first pair of each block
    uint32_t *tmask = reinterpret_cast<uint32_t *>(smem + p.off_mask);        // [FG][nCB] kept-tap bitsets
    uint16_t *segoff = reinterpret_cast<uint16_t *>(smem + p.off_segoff);     // [nChunks][FG] offset/16 in its slot
    uint8_t *segslot = smem + p.off_segslot;                                  // [nChunks][FG] slot within the chunk
    uint16_t *slotbase = reinterpret_cast<uint16_t *>(smem + p.off_slotbase); // [nChunks+1] first slot of each chunk
    uint32_t *used = reinterpret_cast<uint32_t *>(smem + p.off_used);         // [nChunks] taps kept by any block
    uint8_t *cnt = smem + p.off_cnt;                                          // [nChunks][FG] records per segment
    Rec *recs = reinterpret_cast<Rec *>(smem + p.off_rec);                    // [nChunks][FG][maxrec]
    uint32_t *tapoff = reinterpret_cast<uint32_t *>(smem + p.off_tap);        // [RS] tap shift in 16-byte units
    Bars *bars = reinterpret_cast<Bars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, n = tile / p.tiles_per_img, y0 = (tile % p.tiles_per_img) * p.TR;
    const int fb0 = blockIdx.y * p.FG;

    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_BLK]);
    const uint32_t *pairs = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
    const uint8_t *values = blob + hdr[BP_OFF_VALUES];

    // ---- set-up, phase 1: barriers, TMEM, kept-tap bitsets and first pair of every block --------
    if (tid == 0) {
        for (int s = 0; s < p.SA; ++s) { mbar_init(&bars->act_full[s], 1); mbar_init(&bars->act_empty[s], 1); }
        for (int s = 0; s < p.NW; ++s) { mbar_init(&bars->w_full[s], 1); mbar_init(&bars->w_empty[s], kMmaWarps); }
        for (int b = 0; b < p.nabuf; ++b) { mbar_init(&bars->a_full[b], 1); mbar_init(&bars->a_empty[b], kMmaWarps); }
        mbar_init(&bars->acc_full, kMmaWarps);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
    }
    if (warp == 2) tmem_alloc(&bars->tmem_base, 512);
    // zero tiles at the head and the tail of every weight slot
    for (int i = tid; i < p.NW * (int)(p.zb / 4); i += kThreads) {
        const int s = i / (p.zb / 4), o = i % (p.zb / 4);
        reinterpret_cast<uint32_t *>(wring + (size_t)s * p.wcap)[o] = 0u;
        reinterpret_cast<uint32_t *>(wring + (size_t)s * p.wcap + p.wcap - p.zb)[o] = 0u;
    }
    if (tid < p.RS) tapoff[tid] = (uint32_t)((tid / p.S) * p.Wp + (tid % p.S));
    for (int i = tid; i < p.FG * p.nCB; i += kThreads) {
        const int g = i / p.nCB, cb = i - g * p.nCB;
        const uint32_t *bo = blk_off + (size_t)(fb0 + g) * p.nCB + cb;
        const uint32_t lo = bo[0], hi = bo[1];
        uint32_t bits = 0;
        for (uint32_t j = lo; j < hi; ++j) bits |= 1u << (pairs[j] >> 16);
        tmask[i] = bits;
        sched[g * (p.nCB + 1) + cb] = lo;
        if (cb == p.nCB - 1) sched[g * (p.nCB + 1) + p.nCB] = hi;
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    // the first activation stages can already be on their way while the tables are built
    if (warp == 0 && lane == 0) {
        for (int s = 0; s < p.SA && s < p.nStages; ++s) {
            mbar_arrive_expect_tx(&bars->act_full[s], p.act_tx_bytes);
            tma_load_5d(act + (size_t)s * p.act_stage_bytes, &tmap_x, &bars->act_full[s], 0, -p.pad, y0 - p.pad,
                        s * p.PPS, n);
        }
    }
    // ---- phase 2: pack every chunk's runs into weight slots (greedy, in filter-block order) -----
    for (int c = tid; c < p.nChunks; c += kThreads) {
        const int cb_lo = c * p.cbs_per_chunk, cb_hi = cb_lo + p.cbs_per_chunk;
        uint32_t off = p.zb, slot = 0, u = 0;
        for (int g = 0; g < p.FG; ++g) {
            const uint32_t bytes = (sched[g * (p.nCB + 1) + cb_hi] - sched[g * (p.nCB + 1) + cb_lo]) * p.pair_bytes;
            if (off + bytes + p.zb > p.wcap) { ++slot; off = p.zb; }
            segoff[c * p.FG + g] = (uint16_t)(off >> 4);
            segslot[c * p.FG + g] = (uint8_t)slot;
            off += bytes;
            u |= tmask[g * p.nCB + cb_lo];
            if (p.cbs_per_chunk == 2) u |= tmask[g * p.nCB + cb_lo + 1];
        }
        used[c] = u;
        slotbase[c + 1] = (uint16_t)(slot + 1);       // count for now, prefix-summed below
    }
    // zero the accumulators: two MMA warps per lane quarter split the columns
    if (warp >= 3) {
        const int ncol = p.FG * p.Mb, mid = ((ncol / 2 + 15) / 16) * 16, half = (warp - 3) >> 2;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        for (int c0 = half ? mid : 0; c0 < (half ? ncol : mid); c0 += 16) tmem_st_zero_x16(tmem_base + lane_base + c0);
        tmem_st_wait();
    }
    __syncthreads();

    // ---- phase 3: slot numbering (warp scan) and the MMA records of every segment ---------------
    if (warp == 0) {
        uint32_t carry = 0;
        for (int c0 = 0; c0 < p.nChunks; c0 += 32) {
            const int c = c0 + lane;
            uint32_t v = c < p.nChunks ? slotbase[c + 1] : 0u;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
                if (lane >= d) v += o;
            }
            if (c < p.nChunks) slotbase[c + 1] = (uint16_t)(carry + v);
            carry += __shfl_sync(0xFFFFFFFFu, v, 31);
        }
        if (lane == 0) slotbase[0] = 0;
    } else {
        for (int i = tid - 32; i < p.nChunks * p.FG; i += kThreads - 32) {
            const int c = i / p.FG, g = i - c * p.FG;
            Rec *out = recs + (size_t)i * p.maxrec;
            const uint32_t pb16 = p.pair_bytes >> 4, so = segoff[i], tail = (p.wcap - p.zb) >> 4;
            int r = 0;
            if (p.Nb == 8) {
                const uint32_t T0 = tmask[g * p.nCB + 2 * c], T1 = tmask[g * p.nCB + 2 * c + 1], n0 = __popc(T0);
                for (uint32_t U = T0 | T1; U; U &= U - 1) {
                    const uint32_t t = __ffs(U) - 1, below = (1u << t) - 1u;
                    const uint32_t h0 = (T0 >> t) & 1u ? so + __popc(T0 & below) * pb16 : 0u;
                    const uint32_t h1 = (T1 >> t) & 1u ? so + (n0 + __popc(T1 & below)) * pb16 : tail;
                    out[r].lo = h0 | ((h1 - h0) << 16);
                    out[r].a_col = t * 8;
                    ++r;
                }
            } else {
                const uint32_t T = tmask[g * p.nCB + c];
                for (uint32_t U = T; U; U &= U - 1) {
                    const uint32_t t = __ffs(U) - 1, idx = __popc(T & ((1u << t) - 1u));
                    for (int ks = 0; ks < p.KS; ++ks) {
                        out[r].lo = (so + idx * pb16 + ks * 2 * p.Mb) | ((uint32_t)p.Mb << 16);
                        out[r].a_col = (t * p.KS + ks) * 8;
                        ++r;
                    }
                }
            }
            cnt[i] = (uint8_t)r;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    if (warp == 0) {
        // ---- activation producer (the first SA stages were issued during set-up) ----------------
        if (lane == 0) {
            int st = 0, k = 1;
            for (int s = p.SA; s < p.nStages; ++s) {
                if (!mbar_wait(&bars->act_empty[st], (k & 1) ^ 1, abort_flag, ws, 0x1100 + s)) break;
                mbar_arrive_expect_tx(&bars->act_full[st], p.act_tx_bytes);
                tma_load_5d(act + (size_t)st * p.act_stage_bytes, &tmap_x, &bars->act_full[st], 0, -p.pad,
                            y0 - p.pad, s * p.PPS, n);
                if (++st == p.SA) { st = 0; ++k; }
            }
        }
    } else if (warp == 1) {
        // ---- weight producer: ring slot = (chunk, run of filter blocks); lane g copies block g ----
        bool ok = true;
        uint32_t st = 0, k = 0;
        for (int c = 0; c < p.nChunks && ok; ++c) {
            const int cb_lo = c * p.cbs_per_chunk, cb_hi = cb_lo + p.cbs_per_chunk;
            const uint32_t nslots = slotbase[c + 1] - slotbase[c];
            for (uint32_t local = 0; local < nslots && ok; ++local) {
                if (k >= 1) ok = mbar_wait(&bars->w_empty[st], (k & 1) ^ 1, abort_flag, ws, 0x1200);
                if (!ok) break;
                // FG <= 32: lane g owns filter block g
                uint32_t lo = 0, bytes = 0, so = 0;
                if (lane < p.FG && segslot[c * p.FG + lane] == local) {
                    lo = sched[lane * (p.nCB + 1) + cb_lo];
                    bytes = (sched[lane * (p.nCB + 1) + cb_hi] - lo) * p.pair_bytes;
                    so = segoff[c * p.FG + lane];
                }
                uint32_t total = bytes;
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, d);
                if (lane == 0) mbar_arrive_expect_tx(&bars->w_full[st], total);
                __syncwarp();
                if (bytes)
                    bulk_load_1d(wring + (size_t)st * p.wcap + ((size_t)so << 4), values + (size_t)lo * p.pair_bytes,
                                 bytes, &bars->w_full[st]);
                if (++st == (uint32_t)p.NW) { st = 0; ++k; }
            }
        }
    } else if (warp == 2) {
        // ---- stager: copy the tap-shifted slices of each chunk from shared memory into TMEM ------
        if (lane == 0) {
            const uint32_t act16 = smem_u32(act) >> 4, plane16 = p.plane_bytes >> 4;
            const uint32_t lbo16 = plane16 << 16, chunk16 = (uint32_t)(p.CCH / 8) * plane16;
            int st = 0, ks_stage = 0, in_stage = 0, b = 0, kb = 0;
            for (int c = 0; c < p.nChunks; ++c) {
                if (in_stage == 0 && !mbar_wait(&bars->act_full[st], ks_stage & 1, abort_flag, ws, 0x1300 + c)) break;
                if (kb >= 1 && !mbar_wait(&bars->a_empty[b], (kb & 1) ^ 1, abort_flag, ws, 0x1400 + c)) break;
                tc_fence_after_sync();
                const uint32_t base16 = (act16 + (uint32_t)st * (p.act_stage_bytes >> 4) + (uint32_t)in_stage * chunk16) | lbo16;
                const uint32_t tbuf = tmem_base + 256 + b * p.bufcols;
                for (uint32_t u = used[c]; u; u &= u - 1) {
                    const uint32_t t = __ffs(u) - 1;
                    const uint32_t lo = base16 + tapoff[t];
                    if (p.KS == 1) {
                        tmem_cp_128x256b(tbuf + t * 8, lo);
                    } else {
                        for (int ks = 0; ks < p.KS; ++ks) tmem_cp_128x256b(tbuf + (t * p.KS + ks) * 8, lo + ks * 2 * plane16);
                    }
                }
                mma_commit(&bars->a_full[b]);
                if (++in_stage == p.chunks_per_stage || c == p.nChunks - 1) {
                    mma_commit(&bars->act_empty[st]);
                    in_stage = 0;
                    if (++st == p.SA) { st = 0; ++ks_stage; }
                }
                if (++b == p.nabuf) { b = 0; ++kb; }
            }
        }
    } else {
        // ---- MMA issue: filter block g belongs to warp g mod 8.  The whole warp walks the loop (so
        // that the index arithmetic stays in the uniform datapath); lane 0 issues ------------------
        const int wq = warp - 3;
        const uint32_t idesc = idesc_bf16_f32(128, p.Mb);
        const uint32_t w16 = smem_u32(wring) >> 4, wcap16 = p.wcap >> 4;
        bool ok = true;
        uint32_t st = 0, k = 0;
        int b = 0, kb = 0;
        for (int c = 0; c < p.nChunks && ok; ++c) {
            if (!mbar_wait(&bars->a_full[b], kb & 1, abort_flag, ws, 0x1500 + c)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t tbuf = tmem_base + 256 + b * p.bufcols;
            const uint32_t nslots = slotbase[c + 1] - slotbase[c];
            const uint8_t *ss = segslot + c * p.FG;
            const uint8_t *cc = cnt + c * p.FG;
            for (uint32_t local = 0; local < nslots; ++local) {
                if (!mbar_wait(&bars->w_full[st], k & 1, abort_flag, ws, 0x1600)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t base16 = w16 + st * wcap16;
                for (int g = wq; g < p.FG; g += kMmaWarps) {
                    if (ss[g] != local) continue;
                    const int nrec = cc[g];
                    const Rec *rr = recs + (size_t)(c * p.FG + g) * p.maxrec;
                    const uint32_t d_tmem = tmem_base + g * p.Mb;
                    for (int r = 0; r < nrec; ++r) {
                        const Rec rec = rr[r];
                        if (lane == 0) mma_bf16_ts(d_tmem, tbuf + rec.a_col, base16 + rec.lo, idesc);
                    }
                }
                if (lane == 0) mma_commit(&bars->w_empty[st]);
                __syncwarp();
                if (++st == (uint32_t)p.NW) { st = 0; ++k; }
            }
            if (ok && lane == 0) mma_commit(&bars->a_empty[b]);
            __syncwarp();
            if (++b == p.nabuf) { b = 0; ++kb; }
        }
        if (ok && lane == 0) mma_commit(&bars->acc_full);
        __syncwarp();

        // ---- fused epilogue: two warps per TMEM lane quarter split the filter columns --------------
        const int quarter = warp & 3, half = wq >> 2, m = quarter * 32 + lane;
        const int oy = m / p.Wp, ox = m % p.Wp, yy = y0 + oy;
        const bool valid = oy < p.TR && yy < p.P && ox < p.Q;
        const int k0 = fb0 * p.Mb;
        const size_t o0 = (((size_t)n * p.P + yy) * p.Q + ox) * p.K + k0;
        const int ncol = p.FG * p.Mb, mid = ((ncol / 2 + 15) / 16) * 16;
        if (ok && mbar_wait(&bars->acc_full, 0, abort_flag, ws, 0x1700)) {
            tc_fence_after_sync();
            for (int c0 = half ? mid : 0; c0 < (half ? ncol : mid); c0 += 16) {
                uint32_t r[16];
                __syncwarp();
                tmem_ld_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_ld_wait();
                if (!valid) continue;
                float v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
                if (bias) {
                    const float4 *bp4 = reinterpret_cast<const float4 *>(bias + k0 + c0);
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const float4 u = __ldg(bp4 + h);
                        v[4 * h] += u.x; v[4 * h + 1] += u.y; v[4 * h + 2] += u.z; v[4 * h + 3] += u.w;
                    }
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
    p.nabuf = min(kMaxABufs, (int)(256u / p.bufcols));
    if (p.nabuf < 2) return false;
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
    p.maxrec = p.RS * p.KS;
    p.pair_bytes = (uint32_t)bp.Mb * bp.Nb * 2u;
    p.zb = (uint32_t)bp.Mb * 16u;
    const uint32_t seg_max = (uint32_t)p.RS * p.cbs_per_chunk * p.pair_bytes;
    const int nFB = d.K / bp.Mb;
    const int tiles = d.N * p.tiles_per_img;
    // filter blocks per CTA: as many as the accumulator columns allow, fewer when that leaves SMs idle
    int best = 0;
    double best_cost = 0;
    for (int f = 1; f <= nFB && f <= 32; ++f) {
        if (nFB % f || f * bp.Mb > 256) continue;
        const double per_chunk = fmax(p.RS * p.KS * 90.0, f * (p.RS * p.KS / 2.5) * fmax(10.0, bp.Mb / 2.0)) + 300.0;
        const double cta = 8000.0 + p.nChunks * per_chunk + f * bp.Mb * 10.0;
        const double waves = ceil((double)tiles * (nFB / f) / 148.0);
        const double cost = waves * cta;
        if (!best || cost < best_cost) { best = f; best_cost = cost; }
    }
    if (!best) return false;
    p.FG = best;
    p.plane_bytes = (uint32_t)p.slab_rows * p.Wp * 16u;
    p.act_tx_bytes = p.plane_bytes * p.PPS;
    p.act_stage_bytes = round_up(p.act_tx_bytes, 128);
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    if ((uint32_t)p.FG * (p.nCB + 1) > 8192u || (uint32_t)p.nChunks * p.FG * p.maxrec * 8u > 80u * 1024u) return false;
    const uint32_t reach = (128u + (d.R - 1) * p.Wp + d.S) * 16u;
    const uint32_t slack = reach > p.plane_bytes ? round_up(reach - p.plane_bytes, 128) : 0u;
    // weight slots: large enough for the biggest single run, otherwise about a third of what a
    // chunk of dense blocks would need (chunks that need more simply take several slots)
    p.wcap = round_up(max(seg_max + 2 * p.zb, min(16384u, (uint32_t)p.FG * seg_max / 3 + 2 * p.zb)), 128);
    if (p.wcap > 65536u) return false;
    const uint32_t n_seg = (uint32_t)p.nChunks * p.FG;
    const uint32_t tables = round_up(4 * p.FG * (p.nCB + 1), 128) + round_up(4 * p.FG * p.nCB, 128) + round_up(2 * n_seg, 128) +
                            round_up(n_seg, 128) * 2 + round_up(2 * (p.nChunks + 1), 128) + round_up(4 * p.nChunks, 128) +
                            round_up(n_seg * p.maxrec * 8u, 128) + round_up(4 * p.RS, 128) + (uint32_t)sizeof(Bars) + 1024u + 256u;
    bool fits = false;
    for (p.SA = min(3, p.nStages); p.SA >= 1; --p.SA) {
        const uint32_t act_bytes = round_up(p.SA * p.act_stage_bytes + slack, 128);
        if (act_bytes + tables + 2 * p.wcap > kSmemLimit) continue;
        p.NW = (int)min((uint32_t)kMaxStages, (kSmemLimit - act_bytes - tables) / p.wcap);
        p.off_act = 0;
        p.off_w = act_bytes;
        p.off_sched = p.off_w + p.NW * p.wcap;
        p.off_mask = round_up(p.off_sched + 4 * p.FG * (p.nCB + 1), 128);
        p.off_segoff = round_up(p.off_mask + 4 * p.FG * p.nCB, 128);
        p.off_segslot = round_up(p.off_segoff + 2 * n_seg, 128);
        p.off_slotbase = round_up(p.off_segslot + n_seg, 128);
        p.off_used = round_up(p.off_slotbase + 2 * (p.nChunks + 1), 128);
        p.off_cnt = round_up(p.off_used + 4 * p.nChunks, 128);
        p.off_rec = round_up(p.off_cnt + n_seg, 128);
        p.off_tap = round_up(p.off_rec + n_seg * p.maxrec * 8u, 128);
        p.off_bar = round_up(p.off_tap + 4 * p.RS, 128);
        p.smem_bytes = p.off_bar + sizeof(Bars) + 1024;
        if (p.smem_bytes <= kSmemLimit) { fits = true; break; }
    }
    if (!fits) return false;
    if (p.plane_bytes * (uint32_t)p.PPS >= (1u << 18)) return false;
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
    // X[N][H][W][C] bf16 seen as (8 channels, W, H, C/8, N): a box lands in shared memory as
    // [octet][row][column][8 channels]
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
