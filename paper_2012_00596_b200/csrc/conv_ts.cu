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
// Pipeline (24 warps, persistent CTA: a CTA keeps its filter group and walks over tiles): warp 0
// streams activation stages; warps 1..4 stream packed weights, one ring slot per chunk, as 1-D
// bulk copies of each filter block's run of pairs straight from the blob (the blob's value order
// IS the operand layout); warps 5..7 copy the kept-tap slices of one 16-channel chunk into one
// of three TMEM staging buffers (taps t with t % 3 == i); warps 8..23 issue the MMAs and then
// run the fused epilogue.  Scalar work in a single thread is the scarce
// resource here (an integer division or a dependent shared-memory load costs 50..70 cycles, one
// thread issues one MMA per ~51..67 cycles, a tcgen05.commit ~190), so everything data dependent
// is computed ONCE per CTA, in parallel, before the main loop: per-block tap bitsets, where each
// block's weights go in the slot, the set of taps each chunk needs, and - because chunk c always
// uses weight slot / staging buffer c & 1 and a fixed activation stage - every tcgen05.cp and
// every MMA as a ready-made (descriptor word, TMEM address) pair stored in the order the issuing
// thread reads it.  Per chunk an MMA warp does two waits, its MMAs and ONE commit: the `done` barrier frees the
// chunk's TMEM staging buffer and its weight slot at once.  Filter block g is always issued by
// warp g mod 16, so each accumulator gets its MMAs from one thread in program order and results
// are bitwise reproducible.  With Nb = 8 a K=16 MMA spans two channel blocks at one tap; a block
// that does not keep the tap contributes the zero tile kept at the head / tail of every weight
// slot.  Accumulators are zeroed per tile, so every MMA accumulates.  Every wait is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kMmaWarps = 16;
constexpr int kWProducers = 4;                  // warps 1..4 stream weights
constexpr int kStagers = 3;                     // warps 5..7 stage activation slices into TMEM
constexpr int kFirstStager = 1 + kWProducers;
constexpr int kFirstMmaWarp = kFirstStager + kStagers;   // warps 8..23 issue MMAs, then run the epilogue
constexpr int kThreads = (kFirstMmaWarp + kMmaWarps) * 32;
constexpr int kMaxStages = 4;
constexpr int kABufs = 3;                       // at most this many TMEM staging buffers
constexpr int kMaxRing = 4;                     // weight slots and `done` barriers: chunk c uses c % n
constexpr int kMaxTaps = 16;
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kDescHi = (128u >> 4) | (1u << 14);   // SBO = 128 bytes, descriptor version bit

struct ConvTsParams {
    int N, H, W, C, K, R, S, pad, P, Q;       // P, Q: output positions at stride 1
    int stride, Po, Qo;                       // the stride asked for and its output size
    int Wp, TR, tiles_per_img, n_tiles, slab_rows;
    int Mb, Nb, nCB, FG, RS;
    int CCH, nChunks, chunks_per_stage, nStages, PPS, cbs_per_chunk;
    int NA, gpw, maxrec, blk_words, cpd_words, NWS, nabuf, max_pairs;
    uint32_t plane_bytes, act_stage_bytes, act_tx_bytes;
    int SA;
    uint32_t pair_bytes, zb, wcap, bufcols;
    int relu, y_bf16;
    uint32_t off_act, off_w, off_first, off_mask, off_used, off_wtot, off_wsrc, off_blk, off_cpd, off_bar, smem_bytes;
};

struct Bars {
    uint64_t act_full[kMaxStages], act_empty[kMaxStages];
    uint64_t w_full[kMaxRing], done[kMaxRing];
    uint64_t a_full[kABufs];
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
    float bias[256];                 // the CTA's filters' biases (zeros when the layer has none)
};

// Source of one filter block's run of pairs for one chunk (read by one lane of the weight warp).
struct __align__(8) WSrc { uint32_t pair_lo; uint16_t bytes16, so16; };

// Ring position that advances by one per use: index in [0, n) plus the number of completed laps.
struct Ring {
    int idx, lap;
    __device__ __forceinline__ void next(int n) { if (++idx == n) { idx = 0; ++lap; } }
};

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
// barrier among the threads of the MMA / epilogue warps only
__device__ __forceinline__ void mma_warps_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kMmaWarps * 32) : "memory"); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    return cvt_bf16x2(lo, hi);
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
    uint32_t *first = reinterpret_cast<uint32_t *>(smem + p.off_first);   // [FG][nCB] first pair of each block
    uint32_t *tmask = reinterpret_cast<uint32_t *>(smem + p.off_mask);    // [FG][nCB] kept-tap bitsets
    uint32_t *used = reinterpret_cast<uint32_t *>(smem + p.off_used);     // [nChunks] taps kept by any block
    uint32_t *wtot = reinterpret_cast<uint32_t *>(smem + p.off_wtot);     // [nChunks] weight bytes of the chunk
    WSrc *wsrc = reinterpret_cast<WSrc *>(smem + p.off_wsrc);             // [nChunks][FG]
    uint32_t *blks = reinterpret_cast<uint32_t *>(smem + p.off_blk);      // [NA][nChunks][gpw][blk_words]
    uint32_t *cpd = reinterpret_cast<uint32_t *>(smem + p.off_cpd);       // [stager][nChunks][cpd_words]
    Bars *bars = reinterpret_cast<Bars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int fb0 = blockIdx.y * p.FG;
    const int tile0 = blockIdx.x, tile_step = gridDim.x;     // this CTA's tiles: tile0, tile0 + step, ...

    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_BLK]);
    const uint32_t *pairs = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
    const uint8_t *values = blob + hdr[BP_OFF_VALUES];

    // ---- set-up (once per CTA), phase 1: barriers, TMEM, kept-tap bitset and first pair per block --
    if (tid == 0) {
        for (int s = 0; s < p.SA; ++s) { mbar_init(&bars->act_full[s], 1); mbar_init(&bars->act_empty[s], kStagers); }
        for (int b = 0; b < kABufs; ++b) mbar_init(&bars->a_full[b], kStagers);
        for (int b = 0; b < kMaxRing; ++b) { mbar_init(&bars->w_full[b], kWProducers); mbar_init(&bars->done[b], p.NA); }   // `done` is a ring of 4
        mbar_init(&bars->acc_full, p.NA);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
    }
    if (warp == 1) tmem_alloc(&bars->tmem_base, 512);
    // zero tiles at the head and the tail of every weight slot
    for (int i = tid; i < p.NWS * (int)(p.zb / 4); i += kThreads) {
        const int s = i / (int)(p.zb / 4), o = i - s * (int)(p.zb / 4);
        reinterpret_cast<uint32_t *>(wring + (size_t)s * p.wcap)[o] = 0u;
        reinterpret_cast<uint32_t *>(wring + (size_t)s * p.wcap + p.wcap - p.zb)[o] = 0u;
    }
    for (int i = tid; i < p.nChunks; i += kThreads) { used[i] = 0u; wtot[i] = 0u; }
    for (int i = tid; i < p.FG * p.Mb; i += kThreads) bars->bias[i] = bias ? bias[fb0 * p.Mb + i] : 0.f;
    for (int i = tid; i < p.FG * p.nCB; i += kThreads) {
        const int g = i / p.nCB, cb = i - g * p.nCB;
        const uint32_t *bo = blk_off + (size_t)(fb0 + g) * p.nCB + cb;
        const uint32_t lo = bo[0], hi = bo[1];
        uint32_t bits = 0;
#pragma unroll
        for (int j = 0; j < kMaxTaps; ++j)            // independent loads: one memory latency, not hi - lo
            if (lo + j < hi) bits |= 1u << (pairs[lo + j] >> 16);
        tmask[i] = bits;
        first[i] = lo;
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    // the first activation stages can already be on their way while the tables are built
    if (warp == 0 && lane == 0) {
        const int n = tile0 / p.tiles_per_img, y0 = (tile0 - n * p.tiles_per_img) * p.TR;
        for (int s = 0; s < p.SA && s < p.nStages; ++s) {
            mbar_arrive_expect_tx(&bars->act_full[s], p.act_tx_bytes);
            tma_load_5d(act + (size_t)s * p.act_stage_bytes, &tmap_x, &bars->act_full[s], 0, -p.pad, y0 - p.pad,
                        s * p.PPS, n);
        }
    }
    // ---- phase 2: one thread per (chunk, filter block): where its weights go and its MMA records.
    // Descriptors are stored relative to the weight slot / staging buffer / activation stage the
    // chunk will use, so that issuing one is a single add. -----------------------------------------
    for (int i = tid; i < p.nChunks * p.FG; i += kThreads) {
        const int c = i / p.FG, g = i - c * p.FG;
        const int cb = c * p.cbs_per_chunk;
        const uint32_t T0 = tmask[g * p.nCB + cb], T1 = p.cbs_per_chunk == 2 ? tmask[g * p.nCB + cb + 1] : 0u;
        const uint32_t n0 = __popc(T0), np = n0 + __popc(T1), pb16 = p.pair_bytes >> 4;
        // offset inside the chunk's slot: behind the head zero tile and the runs of the blocks before it
        uint32_t so = p.zb >> 4;
        for (int gg = 0; gg < g; ++gg)
            so += (__popc(tmask[gg * p.nCB + cb]) + (p.cbs_per_chunk == 2 ? __popc(tmask[gg * p.nCB + cb + 1]) : 0)) * pb16;
        WSrc e;
        e.pair_lo = first[g * p.nCB + cb]; e.bytes16 = (uint16_t)(np * pb16); e.so16 = (uint16_t)so;
        wsrc[i] = e;
        if (np) { atomicOr(&used[c], T0 | T1); atomicAdd(&wtot[c], np * p.pair_bytes); }
        // MMA block of warp (g mod NA): {count, accumulator address} then {B descriptor low word, A address}
        const int w = g & (p.NA - 1), k = g / p.NA;
        uint32_t *blk = blks + ((size_t)(w * p.nChunks + c) * p.gpw + k) * p.blk_words;
        const uint32_t tail = (p.wcap - p.zb) >> 4;
        if (np > (uint32_t)p.max_pairs) bars->abort_flag = 2;     // more kept taps than the descriptor promised
        int r = 0;
        if (p.Nb == 8) {
            for (uint32_t U = T0 | T1; U; U &= U - 1) {
                const uint32_t t = __ffs(U) - 1, below = (1u << t) - 1u;
                const uint32_t h0 = (T0 >> t) & 1u ? so + __popc(T0 & below) * pb16 : 0u;
                const uint32_t h1 = (T1 >> t) & 1u ? so + (n0 + __popc(T1 & below)) * pb16 : tail;
                blk[2 + 2 * r] = h0 | ((h1 - h0) << 16);
                blk[3 + 2 * r] = t * 8;
                ++r;
            }
        } else {
            for (uint32_t U = T0; U; U &= U - 1) {
                const uint32_t t = __ffs(U) - 1, idx = __popc(T0 & ((1u << t) - 1u));
                blk[2 + 2 * r] = (so + idx * pb16) | ((uint32_t)p.Mb << 16);
                blk[3 + 2 * r] = t * 8;
                ++r;
            }
        }
        blk[0] = (uint32_t)r;
        blk[1] = tmem_base + g * p.Mb;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const bool bad_blob = *abort_flag != 0;
    if (bad_blob && tid == 0) { if (atomicCAS(ws, 0u, 6u /* NPAS_ERR_BLOB */) == 0u) ws[1] = 0x1001; }
    // ---- phase 3: per chunk and stager, the list of tcgen05.cp operations in final form ---------
    for (int i = tid; i < kStagers * p.nChunks; i += kThreads) {
        const int me = i % kStagers, c = i / kStagers;
        const int stage = c / p.chunks_per_stage, in_stage = c - stage * p.chunks_per_stage;
        const uint32_t plane16 = p.plane_bytes >> 4;
        const uint32_t base16 = ((uint32_t)in_stage * 2u * plane16) | (plane16 << 16);   // relative to the stage
        uint32_t *out = cpd + ((size_t)me * p.nChunks + c) * p.cpd_words;
        int r = 0;
        for (uint32_t U = used[c]; U; U &= U - 1) {
            const uint32_t t = __ffs(U) - 1;
            if ((int)(t % kStagers) != me) continue;
            out[2 + 2 * r] = base16 + (t / p.S) * p.Wp + (t % p.S);
            out[3 + 2 * r] = t * 8;
            ++r;
        }
        // control word: count | first chunk of its stage << 16 | last chunk of its stage << 17
        const bool last = in_stage == p.chunks_per_stage - 1 || c == p.nChunks - 1;
        out[0] = (uint32_t)r | ((in_stage == 0 ? 1u : 0u) << 16) | ((last ? 1u : 0u) << 17);
        out[1] = 0;
    }
    __syncthreads();

    if (bad_blob) {
        // nothing may be copied: a run of pairs could overflow its slot
    } else if (warp == 0) {
        // ---- activation producer (the first SA stages of the first tile were issued during set-up) --
        if (lane == 0) {
            Ring ring{0, 0};
            bool ok = true;
            int skip = min(p.SA, p.nStages);
            for (int tile = tile0; tile < p.n_tiles && ok; tile += tile_step) {
                const int n = tile / p.tiles_per_img, y0 = (tile - n * p.tiles_per_img) * p.TR;
                for (int s = 0; s < p.nStages; ++s, ring.next(p.SA)) {
                    if (skip > 0) { --skip; continue; }
                    if (ring.lap >= 1 && !mbar_wait(&bars->act_empty[ring.idx], (ring.lap & 1) ^ 1, abort_flag, ws, 0x1100 + s)) { ok = false; break; }
                    mbar_arrive_expect_tx(&bars->act_full[ring.idx], p.act_tx_bytes);
                    tma_load_5d(act + (size_t)ring.idx * p.act_stage_bytes, &tmap_x, &bars->act_full[ring.idx], 0, -p.pad,
                                y0 - p.pad, s * p.PPS, n);
                }
            }
        }
    } else if (warp < kFirstStager) {
        // ---- weight producers: chunk c goes to slot c % NWS.  Issuing a bulk copy costs the issuing
        // warp ~80 cycles, so the copies of a chunk (one per filter block: a block's run of pairs is
        // contiguous in the blob) are spread over four warps, each announcing its own byte count.  A
        // slot is free again once the MMA warps have committed the chunk that used it (the barrier
        // that also frees the TMEM staging buffer) ---------------------------------------------------
        const int pw = warp - 1, g = lane * kWProducers + pw;
        bool ok = true;
        uint32_t use = 0;                               // chunks issued so far
        const uint32_t nd_mask = kMaxRing - 1, nd_shift = 2;
        for (int tile = tile0; tile < p.n_tiles && ok; tile += tile_step) {
            const WSrc *src = wsrc + g;
            for (int c = 0; c < p.nChunks && ok; ++c, src += p.FG, ++use) {
                WSrc e;
                e.pair_lo = 0; e.bytes16 = 0; e.so16 = 0;
                if (g < p.FG) e = *src;
                uint32_t total = (uint32_t)e.bytes16 << 4;
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, d);
                const uint32_t slot = use & (p.NWS - 1);
                if (lane == 0) {
                    if (use >= (uint32_t)p.NWS) {
                        const uint32_t prev = use - p.NWS;
                        ok = mbar_wait(&bars->done[prev & nd_mask], (prev >> nd_shift) & 1u, abort_flag, ws, 0x1200 + c);
                    }
                    if (ok) mbar_arrive_expect_tx(&bars->w_full[slot], total);
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                if (ok && e.bytes16)
                    bulk_load_1d(wring + (size_t)slot * p.wcap + ((size_t)e.so16 << 4), values + (size_t)e.pair_lo * p.pair_bytes,
                                 (uint32_t)e.bytes16 << 4, &bars->w_full[slot]);
            }
        }
    } else if (warp < kFirstMmaWarp) {
        // ---- three stagers: copy the tap-shifted slices of each chunk from shared memory into
        // TMEM, stager i taking the taps t with t % 3 == i.  All descriptors come ready-made --------
        if (lane == 0) {
            const uint32_t *mine = cpd + (size_t)(warp - kFirstStager) * p.nChunks * p.cpd_words;
            const uint32_t nd_mask = kMaxRing - 1, nd_shift = 2;
            const uint32_t act16 = smem_u32(act) >> 4, stage16 = p.act_stage_bytes >> 4;
            uint32_t use = 0;                           // chunks staged so far
            Ring ar{0, 0};                              // activation stage
            Ring br{0, 0};                              // TMEM staging buffer
            bool ok = true;
            for (int tile = tile0; tile < p.n_tiles && ok; tile += tile_step) {
                const uint32_t *e = mine;
                for (int c = 0; c < p.nChunks; ++c, e += p.cpd_words, ++use) {
                    const uint4 v0 = *reinterpret_cast<const uint4 *>(e);
                    const uint4 v1 = *reinterpret_cast<const uint4 *>(e + 4);
                    const uint4 v2 = *reinterpret_cast<const uint4 *>(e + 8);
                    const uint4 v3 = *reinterpret_cast<const uint4 *>(e + 12);
                    const uint32_t cnt = v0.x & 0xFFu;
                    if ((v0.x >> 16) & 1u) {
                        if (!mbar_wait(&bars->act_full[ar.idx], ar.lap & 1, abort_flag, ws, 0x1300 + c)) { ok = false; break; }
                    }
                    if (use >= (uint32_t)p.nabuf) {
                        const uint32_t prev = use - p.nabuf;
                        if (!mbar_wait(&bars->done[prev & nd_mask], (prev >> nd_shift) & 1u, abort_flag, ws, 0x1400 + c)) { ok = false; break; }
                    }
                    const uint32_t sb = act16 + (uint32_t)ar.idx * stage16, tb = tmem_base + 256 + br.idx * p.bufcols;
                    tc_fence_after_sync();
                    if (cnt > 0) tmem_cp_128x256b(tb + v0.w, sb + v0.z);
                    if (cnt > 1) tmem_cp_128x256b(tb + v1.y, sb + v1.x);
                    if (cnt > 2) tmem_cp_128x256b(tb + v1.w, sb + v1.z);
                    if (cnt > 3) tmem_cp_128x256b(tb + v2.y, sb + v2.x);
                    if (cnt > 4) tmem_cp_128x256b(tb + v2.w, sb + v2.z);
                    if (cnt > 5) tmem_cp_128x256b(tb + v3.y, sb + v3.x);
                    mma_commit(&bars->a_full[br.idx]);
                    if ((v0.x >> 17) & 1u) { mma_commit(&bars->act_empty[ar.idx]); ar.next(p.SA); }
                    br.next(p.nabuf);
                }
            }
        }
    } else {
        // ---- MMA issue + epilogue.  Filter block g belongs to warp g mod NA; the whole warp walks
        // the loop (index arithmetic stays in the uniform datapath), lane 0 issues -------------------
        const int wq = warp - kFirstMmaWarp;
        // kMmaWarps / 4 warps share a TMEM lane quarter and split the filter columns between them
        const int quarter = warp & 3, part = wq >> 2;
        const int ncol = p.FG * p.Mb, per_part = ((ncol + kMmaWarps / 4 - 1) / (kMmaWarps / 4) + 15) / 16 * 16;
        const int col_lo = min(ncol, part * per_part), col_hi = min(ncol, col_lo + per_part);
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t idesc = idesc_bf16_f32(128, p.Mb);
        const uint32_t *blk_base = blks + (size_t)wq * p.nChunks * p.gpw * p.blk_words;
        const uint32_t w16 = smem_u32(wring) >> 4, wcap16 = p.wcap >> 4;
        Ring br{0, 0};                                  // TMEM staging buffer
        const int k0 = fb0 * p.Mb;
        const int m = quarter * 32 + lane, oy = m / p.Wp, ox = m - oy * p.Wp;
        uint32_t use = 0;                               // chunks consumed so far
        bool ok = true;
        int it = 0;
        for (int tile = tile0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
            // zero this tile's accumulators (every MMA accumulates), then let no MMA start early
            for (int c0 = col_lo; c0 < col_hi; c0 += 16) tmem_st_zero_x16(tmem_base + lane_base + c0);
            tmem_st_wait();
            tc_fence_before_sync();
            mma_warps_sync();
            tc_fence_after_sync();
            if (wq < p.NA) {
                const uint32_t *blk = blk_base;
                for (int c = 0; c < p.nChunks && ok; ++c, ++use) {
                    const uint32_t slot = use & (p.NWS - 1), dn = use & (kMaxRing - 1);
                    const uint32_t wb = w16 + slot * wcap16, ab = tmem_base + 256 + br.idx * p.bufcols;
                    // the first records do not depend on the barriers: fetch them while waiting
                    const uint4 v0 = *reinterpret_cast<const uint4 *>(blk);
                    const uint4 v1 = *reinterpret_cast<const uint4 *>(blk + 4);
                    if (!mbar_wait(&bars->a_full[br.idx], br.lap & 1, abort_flag, ws, 0x1500 + c)) { ok = false; break; }
                    if (!mbar_wait(&bars->w_full[slot], (use >> (p.NWS == 4 ? 2 : 1)) & 1u, abort_flag, ws, 0x1600 + c)) { ok = false; break; }
                    tc_fence_after_sync();
                    {
                        const uint32_t cnt = v0.x, d_tmem = v0.y;
                        if (lane == 0) {
                            if (cnt > 0) mma_bf16_ts(d_tmem, ab + v0.w, wb + v0.z, idesc);
                            if (cnt > 1) mma_bf16_ts(d_tmem, ab + v1.y, wb + v1.x, idesc);
                            if (cnt > 2) mma_bf16_ts(d_tmem, ab + v1.w, wb + v1.z, idesc);
                        }
                        for (uint32_t r = 3; r < cnt; ++r) {
                            const uint2 rec = *reinterpret_cast<const uint2 *>(blk + 2 + 2 * r);
                            if (lane == 0) mma_bf16_ts(d_tmem, ab + rec.y, wb + rec.x, idesc);
                        }
                        blk += p.blk_words;
                    }
                    for (int k = 1; k < p.gpw; ++k, blk += p.blk_words) {
                        const uint4 u0 = *reinterpret_cast<const uint4 *>(blk);
                        const uint4 u1 = *reinterpret_cast<const uint4 *>(blk + 4);
                        const uint32_t cnt = u0.x, d_tmem = u0.y;
                        if (lane == 0) {
                            if (cnt > 0) mma_bf16_ts(d_tmem, ab + u0.w, wb + u0.z, idesc);
                            if (cnt > 1) mma_bf16_ts(d_tmem, ab + u1.y, wb + u1.x, idesc);
                            if (cnt > 2) mma_bf16_ts(d_tmem, ab + u1.w, wb + u1.z, idesc);
                        }
                        for (uint32_t r = 3; r < cnt; ++r) {
                            const uint2 rec = *reinterpret_cast<const uint2 *>(blk + 2 + 2 * r);
                            if (lane == 0) mma_bf16_ts(d_tmem, ab + rec.y, wb + rec.x, idesc);
                        }
                    }
                    if (lane == 0) mma_commit(&bars->done[dn]);
                    __syncwarp();
                    br.next(p.nabuf);
                }
                if (ok && lane == 0) mma_commit(&bars->acc_full);
                __syncwarp();
            }
            ok = ok && !*abort_flag;

            // fused epilogue: two warps per TMEM lane quarter split the filter columns
            const int n = tile / p.tiles_per_img, y0 = (tile - n * p.tiles_per_img) * p.TR;
            const int yy = y0 + oy;
            // with a stride the tile is computed at every position and only the strided ones are stored
            const bool valid = oy < p.TR && yy < p.P && ox < p.Q && yy % p.stride == 0 && ox % p.stride == 0;
            const size_t o0 = (((size_t)n * p.Po + yy / p.stride) * p.Qo + ox / p.stride) * p.K + k0;
            if (ok && mbar_wait(&bars->acc_full, it & 1, abort_flag, ws, 0x1700)) {
                tc_fence_after_sync();
                for (int c0 = col_lo; c0 < col_hi; c0 += 16) {
                    uint32_t r[16];
                    __syncwarp();
                    tmem_ld_x16(tmem_base + lane_base + c0, r);
                    tmem_ld_wait();
                    if (!valid) continue;
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) + bars->bias[c0 + i];
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
            } else {
                ok = false;
            }
            // all epilogue reads of this tile are done before any warp zeroes / reuses the accumulators
            tc_fence_before_sync();
            mma_warps_sync();
            tc_fence_after_sync();
            ok = ok && !*abort_flag;
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
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

bool plan(const npas_conv_desc &d, const npas_bp_desc &bp, ConvTsParams &p, dim3 &grid)
{
    if (d.x_dtype != NPAS_BF16 || bp.w_packed != NPAS_BF16) return false;
    if ((d.stride != 1 && d.stride != 2) || d.pad < 0) return false;
    if (bp.Nb != 8 && bp.Nb != 16) return false;
    if (bp.Mb % 16 || bp.Mb > 256 || d.C % 16 || d.K % 8) return false;
    p.RS = d.R * d.S;
    p.CCH = 16;
    if (p.RS > kMaxTaps) return false;
    p.bufcols = (uint32_t)p.RS * 8;
    p.nabuf = min(kABufs, (int)(256u / p.bufcols));
    if (p.nabuf < 2) return false;
    p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C; p.K = d.K; p.R = d.R; p.S = d.S; p.pad = d.pad;
    p.P = d.H + 2 * d.pad - d.R + 1; p.Q = d.W + 2 * d.pad - d.S + 1;     // positions at stride 1
    if (p.P < 1 || p.Q < 1) return false;
    p.stride = d.stride;
    p.Po = (p.P - 1) / d.stride + 1; p.Qo = (p.Q - 1) / d.stride + 1;
    p.Wp = d.W + 2 * d.pad;
    if (p.Wp > 128) return false;
    p.TR = min(p.P, 128 / p.Wp);
    p.tiles_per_img = (p.P + p.TR - 1) / p.TR;
    p.n_tiles = d.N * p.tiles_per_img;
    p.slab_rows = p.TR + d.R - 1;
    if (p.slab_rows > 256 || p.TR * p.Wp <= d.S - 1) return false;
    p.Mb = bp.Mb; p.Nb = bp.Nb; p.nCB = d.C / bp.Nb;
    p.cbs_per_chunk = bp.Nb == 8 ? 2 : 1;
    p.nChunks = d.C / p.CCH;
    p.maxrec = p.RS;
    p.blk_words = (2 + 2 * p.maxrec + 3) & ~3;
    p.cpd_words = 16;                                        // header pair + up to 6 operations per stager
    if ((p.RS + kStagers - 1) / kStagers > 6) return false;
    if (p.blk_words < 8) p.blk_words = 8;
    p.pair_bytes = (uint32_t)bp.Mb * bp.Nb * 2u;
    p.zb = (uint32_t)bp.Mb * 16u;
    p.plane_bytes = (uint32_t)p.slab_rows * p.Wp * 16u;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    // kept taps per block: the descriptor's promise when it makes one, else all of them
    const int max_taps = bp.max_taps > 0 ? min(bp.max_taps, p.RS) : p.RS;
    p.max_pairs = max_taps * p.cbs_per_chunk;
    const uint32_t seg_max = (uint32_t)p.max_pairs * p.pair_bytes;

    const uint32_t reach = (128u + (d.R - 1) * p.Wp + d.S) * 16u;
    const uint32_t slack = reach > p.plane_bytes ? round_up(reach - p.plane_bytes, 128) : 0u;
    const int nFB = d.K / bp.Mb;
    // Filter blocks per CTA (a power of two).  More blocks per CTA reuse every staged activation
    // slice more often but need a larger weight slot; fewer blocks give more CTAs.  Among the
    // choices that fit in shared memory take the one with the lowest estimated time.
    bool found = false;
    double best_cost = 0;
    ConvTsParams best = p;
    dim3 best_grid;
    for (int f = 1; f <= nFB && f <= 32; f *= 2) {
        if (nFB % f || f * bp.Mb > 256) continue;
        ConvTsParams q = p;
        q.FG = f;
        q.NA = min(f, kMmaWarps);
        q.gpw = f / q.NA;
        q.wcap = round_up((uint32_t)f * seg_max + 2 * q.zb, 128);
        if (q.wcap > 100000u) continue;
        const uint32_t n_seg = (uint32_t)q.nChunks * f;
        const uint32_t blk_bytes = 4u * q.NA * q.nChunks * q.gpw * q.blk_words;
        if ((uint32_t)f * q.nCB > 8192u) continue;
        const uint32_t cpd_bytes = 4u * kStagers * q.nChunks * q.cpd_words;
        const uint32_t tables = 2 * round_up(4 * f * q.nCB, 128) + 2 * round_up(4 * q.nChunks, 128) + round_up(8 * n_seg, 128) +
                                round_up(blk_bytes, 128) + round_up(cpd_bytes, 128) + (uint32_t)sizeof(Bars) + 1024u + 256u;
        bool fits = false;
        for (int nws = kMaxRing; nws >= 2 && !fits; nws /= 2)
        for (int cps = 4; cps >= 1 && !fits; cps /= 2) {
            q.NWS = nws;
            q.chunks_per_stage = min(cps, q.nChunks);
            q.PPS = q.chunks_per_stage * 2;
            q.nStages = (q.nChunks + q.chunks_per_stage - 1) / q.chunks_per_stage;
            q.act_tx_bytes = q.plane_bytes * q.PPS;
            q.act_stage_bytes = round_up(q.act_tx_bytes, 128);
            for (q.SA = 3; q.SA >= 2 && !fits; --q.SA) {
                const uint32_t act_bytes = round_up(q.SA * q.act_stage_bytes + slack, 128);
                q.off_act = 0;
                q.off_w = act_bytes;
                q.off_first = q.off_w + q.NWS * q.wcap;
                q.off_mask = round_up(q.off_first + 4 * f * q.nCB, 128);
                q.off_used = round_up(q.off_mask + 4 * f * q.nCB, 128);
                q.off_wtot = round_up(q.off_used + 4 * q.nChunks, 128);
                q.off_wsrc = round_up(q.off_wtot + 4 * q.nChunks, 128);
                q.off_blk = round_up(q.off_wsrc + 8 * n_seg, 128);
                q.off_cpd = round_up(q.off_blk + blk_bytes, 128);
                q.off_bar = round_up(q.off_cpd + cpd_bytes, 128);
                q.smem_bytes = q.off_bar + sizeof(Bars) + 1024;
                fits = q.smem_bytes <= kSmemLimit && q.plane_bytes * (uint32_t)q.PPS < (1u << 18);
                if (fits) break;
            }
        }
        if (!fits) continue;
        const int groups = nFB / f;
        const int ctas_x = min(q.n_tiles, max(1, 148 / groups));
        const double tiles_per_cta = ceil((double)q.n_tiles / ctas_x);
        const double mma_per_blk = q.RS / 3.0 * (q.Nb == 8 ? 1.67 : 1.0);
        const double per_chunk = fmax((q.RS + 1) / 2 * 70.0 + 350.0, q.gpw * mma_per_blk * 67.0 + 340.0);
        const double cost = 6000.0 + tiles_per_cta * (q.nChunks * per_chunk + 800.0 + f * bp.Mb * 8.0);
        if (!found || cost < best_cost) { found = true; best_cost = cost; best = q; best_grid = dim3(ctas_x, groups); }
    }
    if (!found || best_grid.y > 65535) return false;
    p = best;
    grid = best_grid;
    return true;
}

}  // namespace

bool conv_ts_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvTsParams p;
    dim3 grid;
    return plan(d, bp, p, grid);
}

npas_status conv_ts_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st)
{
    ConvTsParams p;
    dim3 grid;
    if (!plan(d, bp, p, grid)) return NPAS_ERR_UNSUPPORTED;
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
    conv_bp_ts_kernel<<<grid, kThreads, p.smem_bytes, st>>>(tmap, p, static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return launch_status();
}

}  // namespace npas
