// Block-punched convolution on the sm_100a tensor cores that multiplies ONLY the kept (block, tap)
// pairs (paper Sec. 3: inside a block the kept kernel positions are shared by all kernels, so a kept
// pair is a dense [Mb filters x Nb channels] sub-contraction).  bf16 in, fp32 accumulation in TMEM.
//
// Mapping.  A CTA owns up to 128 consecutive "padded-linear" output positions of one image (M of
// the MMA) and one group of GS filter blocks (<= 256 filters = 256 fp32 accumulator columns).  For a
// 16-channel chunk and a tap, the activation operand (128 positions x 16 channels, shifted by the
// tap) is the same for every filter block that keeps the tap.  Measured on B200, what an MMA with
// a small N costs is the fetch of that operand, not the math: about 39 cycles from shared memory
// and about 24 from tensor memory, whatever N <= 48.  So
//   * each tap-shifted slice is written ONCE per chunk into tensor memory, by ordinary threads
//     (two 16-byte shared-memory loads and a share of a tcgen05.st per position; this runs on the
//     load/store path beside the MMAs, where the tcgen05.cp alternative queues with them), and
//   * neighbouring filter blocks that keep the same tap are covered by ONE MMA of N = run x Mb:
//     the blob's `kt` section stores the kept tiles of a (chunk, group) tap by tap with the blocks
//     in ascending order, in a layout in which consecutive tiles form one valid B operand.
// Accumulator columns are split into fixed segments of SEG filter blocks, one issuing warp per
// segment; runs are formed inside a segment only, so every accumulator column receives all its
// MMAs from one thread in program order (bitwise reproducible sums).
//
// Pipeline (18 warps, persistent CTA over the tiles of its filter group):
//   warp 0      activation slabs by TMA, [channel octet][padded position][8 channels], zero fill
//               outside the image = padding; a tap shift is an address offset of whole positions
//   warp 1      the chunk's tiles of the group: ONE bulk copy per chunk into a ring of weight slots
//   warps 2-9   stagers: slab -> registers -> TMEM staging buffer (ring of 2 or 3), one warp per
//               TMEM lane quarter, two sets of four warps taking alternate chunks
//   warps 10-17 MMA issue (one thread of each of the first NA warps, chosen with elect.sync) and
//               then the fused epilogue (bf16 output in whole 64-filter slabs: through shared
//               memory and tensor stores; otherwise straight from registers)
// The MMAs of every (issuing warp, chunk) are written into shared memory once per CTA as ready-made
// records (built by the issuing warps from the per-tap bitsets of keeping blocks, which come from the
// blob's index sections, while the producers already run).  Per chunk an issuing warp fetches its
// records, waits for the staging buffer and the weight slot, issues, and commits once: that commit
// frees both the staging buffer and the weight slot.
// Every wait is bounded; a blob that breaks the descriptor's promises is reported, not computed.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kStagerWarps = 8;
constexpr int kFirstStager = 2;
constexpr int kFirstMmaWarp = kFirstStager + kStagerWarps;
constexpr int kMmaWarps = 8;
constexpr int kThreads = (kFirstMmaWarp + kMmaWarps) * 32;
constexpr int kMaxStages = 4;
constexpr int kABufs = 3;
constexpr int kMaxRing = 4;            // weight slots and `done` barriers: chunk use u -> u % n
constexpr int kMaxTaps = 16;
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kDescHiB = (256u >> 4) | (1u << 14);   // B operand: 256 bytes between filter octets

struct ConvKrParams {
    int N, H, W, C, K, R, S, pad, P, Q;
    int Wp, TR, tiles_per_img, n_tiles, slab_rows;
    int Mb, GS, SEG, NA, RS, nGrp;
    int nChunks, cps, nStages, PPS, SA, NWS, nabuf, NP, cpb, nCB, max_taps;
    uint32_t plane_bytes, act_stage_bytes, act_tx_bytes, wcap, bufcols, tile_bytes;
    int relu, y_bf16;
    uint32_t off_act, off_w, off_cm, off_kto, off_rec, off_bar, smem_bytes;
    int RW;                      // words per (issuing warp, chunk) record list: count + MMAs, a multiple of 4
    int epi_tma;                 // bf16 output leaves through shared memory and tensor stores (64-filter slabs)
    uint32_t off_epi;
};

struct Bars {
    uint64_t act_full[kMaxStages], act_empty[kMaxStages];
    uint64_t w_full[kMaxRing], done[kMaxRing];
    uint64_t a_full[kABufs];
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t tapoff[kMaxTaps];       // byte offset of a tap's shift inside a slab plane
    float bias[256];
};

struct Ring {
    int idx, lap;
    __device__ __forceinline__ void next(int n) { if (++idx == n) { idx = 0; ++lap; } }
};

// D[tmem] += A[tmem] * B[smem]
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 d;\n\tsetp.ne.b32 p, 1, 0;\n\tmov.b64 d, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], d, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(kDescHiB), "r"(idesc));
}
__device__ __forceinline__ void tmem_st_zero_x16(uint32_t taddr)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                 ::"r"(taddr), "r"(0u) : "memory");
}
__device__ __forceinline__ void tmem_st_x8(uint32_t taddr, const uint4 &a, const uint4 &b)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}
// four taps (4 x 8 columns) in one instruction
__device__ __forceinline__ void tmem_st_x32(uint32_t taddr, const uint4 (&u)[8])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr),
          "r"(u[0].x), "r"(u[0].y), "r"(u[0].z), "r"(u[0].w), "r"(u[1].x), "r"(u[1].y), "r"(u[1].z), "r"(u[1].w),
          "r"(u[2].x), "r"(u[2].y), "r"(u[2].z), "r"(u[2].w), "r"(u[3].x), "r"(u[3].y), "r"(u[3].z), "r"(u[3].w),
          "r"(u[4].x), "r"(u[4].y), "r"(u[4].z), "r"(u[4].w), "r"(u[5].x), "r"(u[5].y), "r"(u[5].z), "r"(u[5].w),
          "r"(u[6].x), "r"(u[6].y), "r"(u[6].z), "r"(u[6].w), "r"(u[7].x), "r"(u[7].y), "r"(u[7].z), "r"(u[7].w)
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void mma_warps_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kMmaWarps * 32) : "memory"); }
// barrier among the four epilogue warps that share one half of the filter columns (ids 2 and 3)
__device__ __forceinline__ void part_sync(int part)
{
    if (part == 0) asm volatile("bar.sync 2, 128;" ::: "memory");
    else asm volatile("bar.sync 3, 128;" ::: "memory");
}
// the same barriers with a vote: true when `pred` holds in every thread that arrives (a group of warps then
// enters or skips a region with barriers inside as one)
template <int kId, int kCount>
__device__ __forceinline__ bool bar_all(bool pred)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %3, 0;\n\tbar.red.and.pred p, %1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r) : "n"(kId), "n"(kCount), "r"((uint32_t)pred) : "memory");
    return r != 0u;
}
// [rows][padded columns][64 filters] in shared memory (128-byte swizzled) -> Y[n][y0 + row][column][k0 ..]; what lies
// outside the tensor (the padding columns of a row, rows past the last) is not written
__device__ __forceinline__ void tma_store_4d(const CUtensorMap *m, uint32_t src, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
constexpr uint32_t kEpiBufBytes = 128u * 128u;          // 128 positions x 64 bf16 filters


// One MMA = one run of neighbouring kept blocks inside a segment at one tap: first tile of the
// chunk's weight slot (12 bits), tap (4 bits), N / 16 (8 bits), first accumulator column / 16 (8 bits).
__device__ __forceinline__ uint32_t make_rec(uint32_t tile, uint32_t tap, uint32_t n16, uint32_t d16)
{
    return tile | (tap << 12) | (n16 << 16) | (d16 << 24);
}

// Staged epilogue of one warp (bf16 output, whole 64-filter slabs): registers -> shared memory (one 128-byte line
// per position, 16-byte units swizzled by the line number) -> one tensor store per slab and column half, which writes
// whole lines where a thread's own stores would be 16-byte requests (measured: 2 k of the 4 k cycles of an epilogue
// over 256 filters).  A function of its own so that its registers do not weigh on the issue loop.
__device__ __forceinline__ void epilogue_staged(const CUtensorMap *tmap_y, uint32_t ebuf, const float *bias_s, const uint16_t *res_row,
                                             bool relu, uint32_t t_addr, int part, bool leader, int m, int col_lo, int col_hi,
                                             int k0, int y0, int n)
{
    const uint32_t line = ebuf + (uint32_t)m * 128u, sw = (uint32_t)(m & 7) << 4;
    auto finish16 = [&](const uint32_t *r, int c0, int u) {
        float v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
        if (bias_s) {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += bias_s[c0 + i];
        }
        if (res_row) {
            const uint4 *rp = reinterpret_cast<const uint4 *>(res_row + c0);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint4 q = rp[h];
                const uint32_t wv[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[8 * h + 2 * i] += __uint_as_float(wv[i] << 16);
                    v[8 * h + 2 * i + 1] += __uint_as_float(wv[i] & 0xFFFF0000u);
                }
            }
        }
        // one rounding, then ReLU on the packed pairs (max with +0 is exact on the rounded values)
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] = cvt_bf16x2(v[2 * i], v[2 * i + 1]);
        if (relu) {
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i] = relu_bf16x2(o[i]);
        }
        st_shared_v4(line + (((uint32_t)(2 * u) << 4) ^ sw), o[0], o[1], o[2], o[3]);
        st_shared_v4(line + (((uint32_t)(2 * u + 1) << 4) ^ sw), o[4], o[5], o[6], o[7]);
    };
    uint32_t ra[32];
    for (int c0 = col_lo; c0 < col_hi; c0 += 64) {
        if (leader) bulk_wait_read_all();            // the slab before this one has left the buffer
        part_sync(part);
#pragma unroll 1
        for (int u = 0; u < 2; ++u) {
            __syncwarp();
            tmem_ld_x32(t_addr + c0 + 32 * u, ra);
            tmem_ld_wait();
            finish16(ra, c0 + 32 * u, 2 * u);
            finish16(ra + 16, c0 + 32 * u + 16, 2 * u + 1);
        }
        fence_proxy_async_smem();
        part_sync(part);
        if (leader) { tma_store_4d(tmap_y, ebuf, k0 + c0, 0, y0, n); bulk_commit(); }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
conv_bp_kr_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_y, const ConvKrParams p,
                  const uint8_t *__restrict__ blob, const float *__restrict__ bias,
                  const void *__restrict__ res, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *act = smem + p.off_act;
    uint8_t *wring = smem + p.off_w;
    uint32_t *colmask = reinterpret_cast<uint32_t *>(smem + p.off_cm);    // [nChunks][16]: blocks of the group keeping (chunk, tap)
    uint32_t *kto = reinterpret_cast<uint32_t *>(smem + p.off_kto);       // [nChunks][2]: first tile, tile count of (chunk, group)
    uint32_t *recs = reinterpret_cast<uint32_t *>(smem + p.off_rec);      // [NA][nChunks][RW]: count, then one word per MMA
    Bars *bars = reinterpret_cast<Bars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int grp = blockIdx.y, fb0 = grp * p.GS;
    const int tile0 = blockIdx.x, tile_step = gridDim.x;

    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);

    // ---- set-up (once per CTA) ------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < p.SA; ++s) { mbar_init(&bars->act_full[s], 1); mbar_init(&bars->act_empty[s], 4 * p.NP); }
        for (int b = 0; b < kABufs; ++b) mbar_init(&bars->a_full[b], 4);
        for (int b = 0; b < kMaxRing; ++b) { mbar_init(&bars->w_full[b], 1); mbar_init(&bars->done[b], p.NA); }
        mbar_init(&bars->acc_full, p.NA);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
        if (p.epi_tma) prefetch_tensormap(&tmap_y);
    }
    if (warp == 1) tmem_alloc(&bars->tmem_base, 512);
    for (int i = tid; i < p.nChunks * 16; i += kThreads) colmask[i] = 0u;
    pdl_trigger();
    pdl_wait();                          // nothing above touches global memory
    for (int i = tid; i < p.GS * p.Mb; i += kThreads) bars->bias[i] = bias ? bias[fb0 * p.Mb + i] : 0.f;
    if (tid < kMaxTaps) bars->tapoff[tid] = tid < p.RS ? (uint32_t)((tid / p.S) * p.Wp + (tid % p.S)) * 16u : 0u;
    __syncthreads();
    // the blob must be what the descriptor says: version, the tile section and its grouping
    const bool hdr_ok = hdr[BP_MAGIC] == kMagicBP && hdr[BP_VERSION] == kVersion && hdr[BP_OFF_KT] != 0u &&
                        hdr[BP_GS] == (uint32_t)p.GS && hdr[BP_MB] == (uint32_t)p.Mb && hdr[BP_NCB] == (uint32_t)p.nCB;
    if (!hdr_ok) {
        if (tid == 0) bars->abort_flag = 2;
    } else {
        const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_BLK]);
        const uint32_t *pairs = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
        const uint32_t *kt_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_KTOFF]);
        // per (block of the group, channel block): its kept taps -> the chunk's per-tap block sets
        for (int i = tid; i < p.GS * p.nCB; i += kThreads) {
            const int g = i / p.nCB, cb = i - g * p.nCB;
            const uint32_t *bo = blk_off + (size_t)(fb0 + g) * p.nCB + cb;
            const uint32_t lo = bo[0], hi = bo[1];
            if (hi - lo > (uint32_t)p.max_taps) { bars->abort_flag = 2; continue; }     // more kept taps than promised
            uint32_t bits = 0;
#pragma unroll
            for (int j = 0; j < kMaxTaps; ++j)
                if (lo + j < hi) bits |= 1u << (pairs[lo + j] >> 16);
            if (bits >> p.RS) { bars->abort_flag = 2; continue; }
            for (uint32_t U = bits; U; U &= U - 1) {
                const uint32_t t = __ffs(U) - 1;
                for (int k = 0; k < p.cpb; ++k) atomicOr(&colmask[(cb * p.cpb + k) * 16 + t], 1u << g);
            }
        }
        for (int c = tid; c < p.nChunks; c += kThreads) {
            const uint32_t a = kt_off[c * p.nGrp + grp], b = kt_off[c * p.nGrp + grp + 1];
            kto[2 * c] = a; kto[2 * c + 1] = b - a;
            if (b < a || b - a > (uint32_t)(p.GS * p.max_taps)) bars->abort_flag = 2;   // would overflow a weight slot
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const bool bad_blob = *abort_flag != 0;
    if (bad_blob && tid == 0) { if (atomicCAS(ws, 0u, 6u /* NPAS_ERR_BLOB */) == 0u) ws[1] = 0x7001; }

    if (bad_blob) {
        // nothing is copied or computed
    } else if (warp == 0) {
        // ---- activation producer ------------------------------------------------------------------
        if (lane == 0) {
            Ring ring{0, 0};
            bool ok = true;
            for (int tile = tile0; tile < p.n_tiles && ok; tile += tile_step) {
                const int n = tile / p.tiles_per_img, y0 = (tile - n * p.tiles_per_img) * p.TR;
                for (int s = 0; s < p.nStages; ++s, ring.next(p.SA)) {
                    if (ring.lap >= 1 && !mbar_wait(&bars->act_empty[ring.idx], (ring.lap & 1) ^ 1, abort_flag, ws, 0x7100 + s)) { ok = false; break; }
                    mbar_arrive_expect_tx(&bars->act_full[ring.idx], p.act_tx_bytes);
                    tma_load_5d(act + (size_t)ring.idx * p.act_stage_bytes, &tmap_x, &bars->act_full[ring.idx], 0, -p.pad,
                                y0 - p.pad, s * p.PPS, n);
                }
            }
        }
    } else if (warp == 1) {
        // ---- weight producer: the group's tiles of a chunk are one contiguous run of the blob ------
        if (lane == 0) {
            const uint8_t *kt = blob + hdr[BP_OFF_KT];
            bool ok = true;
            uint32_t use = 0;
            for (int tile = tile0; tile < p.n_tiles && ok; tile += tile_step) {
                for (int c = 0; c < p.nChunks; ++c, ++use) {
                    const uint32_t slot = use & (p.NWS - 1);
                    if (use >= (uint32_t)p.NWS) {
                        const uint32_t prev = use - p.NWS;
                        if (!mbar_wait(&bars->done[prev & (kMaxRing - 1)], (prev >> 2) & 1u, abort_flag, ws, 0x7200 + c)) { ok = false; break; }
                    }
                    const uint32_t first = kto[2 * c], bytes = kto[2 * c + 1] * p.tile_bytes;
                    mbar_arrive_expect_tx(&bars->w_full[slot], bytes);
                    if (bytes) bulk_load_1d(wring + (size_t)slot * p.wcap, kt + (size_t)first * p.tile_bytes, bytes, &bars->w_full[slot]);
                }
            }
        }
    } else if (warp < kFirstMmaWarp) {
        // ---- stagers ------------------------------------------------------------------------------
        const int quarter = warp & 3, phase = (warp - kFirstStager) >> 2;
        if (phase < p.NP) {
            const uint32_t m = (uint32_t)(quarter * 32 + lane);
            const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
            const int full_groups = p.RS >> 2;
            uint32_t tapoff[9];                            // shifts of a 3x3 kernel, in registers
#pragma unroll
            for (int k = 0; k < 9; ++k) tapoff[k] = bars->tapoff[k];
            bool ok = true;
            uint32_t use = 0;
            Ring ar{0, 0};                                 // activation stage
            uint32_t buf = 0;                              // TMEM staging buffer of chunk `use`
            for (int tile = tile0; tile < p.n_tiles && ok; tile += tile_step) {
                for (int st = 0; st < p.nStages && ok; ++st, ar.next(p.SA)) {
                    for (int in_stage = 0; in_stage < p.cps; ++in_stage, ++use, buf = buf + 1 == (uint32_t)p.nabuf ? 0u : buf + 1) {
                        if ((int)(use & (uint32_t)(p.NP - 1)) != phase) continue;
                        const int c = st * p.cps + in_stage;
                        if (!mbar_wait(&bars->act_full[ar.idx], ar.lap & 1, abort_flag, ws, 0x7300 + c)) { ok = false; break; }
                        if (use >= (uint32_t)p.nabuf) {
                            const uint32_t prev = use - p.nabuf;
                            if (!mbar_wait(&bars->done[prev & (kMaxRing - 1)], (prev >> 2) & 1u, abort_flag, ws, 0x7400 + c)) { ok = false; break; }
                        }
                        tc_fence_after_sync();
                        const uint8_t *src = act + (size_t)ar.idx * p.act_stage_bytes + (size_t)in_stage * 2u * p.plane_bytes + m * 16u;
                        const uint32_t tb = tmem_base + lane_base + 256 + buf * p.bufcols;
                        if (p.RS == 9) {
                            // 3x3 kernels: all eighteen loads in flight together, then three stores
                            uint4 u[8], v[8], w0, w1;
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint8_t *q = src + tapoff[k], *q2 = src + tapoff[4 + k];
                                u[2 * k] = *reinterpret_cast<const uint4 *>(q);
                                u[2 * k + 1] = *reinterpret_cast<const uint4 *>(q + p.plane_bytes);
                                v[2 * k] = *reinterpret_cast<const uint4 *>(q2);
                                v[2 * k + 1] = *reinterpret_cast<const uint4 *>(q2 + p.plane_bytes);
                            }
                            w0 = *reinterpret_cast<const uint4 *>(src + tapoff[8]);
                            w1 = *reinterpret_cast<const uint4 *>(src + tapoff[8] + p.plane_bytes);
                            tmem_st_x32(tb, u);
                            tmem_st_x32(tb + 32, v);
                            tmem_st_x8(tb + 64, w0, w1);
                        } else {
                        for (int g = 0; g < full_groups; ++g) {
                            uint4 u[8];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint8_t *q = src + bars->tapoff[4 * g + k];
                                u[2 * k] = *reinterpret_cast<const uint4 *>(q);
                                u[2 * k + 1] = *reinterpret_cast<const uint4 *>(q + p.plane_bytes);
                            }
                            tmem_st_x32(tb + g * 32, u);
                        }
                        for (int t = full_groups * 4; t < p.RS; ++t) {
                            const uint8_t *q = src + bars->tapoff[t];
                            const uint4 u0 = *reinterpret_cast<const uint4 *>(q);
                            const uint4 u1 = *reinterpret_cast<const uint4 *>(q + p.plane_bytes);
                            tmem_st_x8(tb + t * 8, u0, u1);
                        }
                        }
                        tmem_st_wait();
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive(&bars->a_full[buf]);
                            // last chunk of this stage that this set of warps handles: the slab may be refilled
                            if (in_stage + p.NP >= p.cps) mbar_arrive(&bars->act_empty[ar.idx]);
                        }
                    }
                }
            }
        }
    } else {
        // ---- MMA issue + epilogue ---------------------------------------------------------------
        const int wq = __shfl_sync(0xFFFFFFFFu, warp, 0) - kFirstMmaWarp;     // (warp-uniform for the compiler)
        // (built by these eight warps while the producers and the stagers already work on the first chunks; the
        // barrier after the zeroing of the first tile's accumulators publishes the lists)
        // every MMA of every (issuing warp, chunk) in the order it will be issued: taps ascending, runs of
        // neighbouring keeping blocks inside the warp's segment ascending
        for (int i = tid - kFirstMmaWarp * 32; i < p.NA * p.nChunks; i += kMmaWarps * 32) {
            const int rw = i / p.nChunks, c = i - rw * p.nChunks;
            uint32_t *out = recs + (size_t)i * p.RW;
            const uint32_t seg_lo = (uint32_t)(rw * p.SEG), seg_mask = (1u << p.SEG) - 1u, mb16 = (uint32_t)p.Mb >> 4;
            uint32_t n = 0, base = 0;
            for (int t = 0; t < p.RS; ++t) {
                const uint32_t cm = colmask[c * 16 + t];
                uint32_t seg = (cm >> seg_lo) & seg_mask;
                while (seg) {
                    const uint32_t s1 = __ffs(seg) - 1, l1 = __ffs(~(seg >> s1)) - 1;
                    out[1 + n++] = make_rec(base + __popc(cm & ((1u << (seg_lo + s1)) - 1u)), (uint32_t)t, l1 * mb16, (seg_lo + s1) * mb16);
                    seg &= ~(((1u << l1) - 1u) << s1);
                }
                base += __popc(cm);
            }
            out[0] = n;
        }
        const int quarter = warp & 3, part = wq >> 2;
        const int ncol = p.GS * p.Mb, per_part = ((ncol + kMmaWarps / 4 - 1) / (kMmaWarps / 4) + 15) / 16 * 16;
        const int col_lo = min(ncol, part * per_part), col_hi = min(ncol, col_lo + per_part);
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t idesc0 = idesc_bf16_f32(128, 0);
        const uint32_t w16 = smem_u32(wring) >> 4, wcap16 = p.wcap >> 4, tile16 = p.tile_bytes >> 4;
        const uint32_t *rec_base = recs + (size_t)wq * p.nChunks * p.RW;
        const uint32_t tmem_base_ = tmem_base;
        auto issue = [&](uint32_t r, uint32_t wb, uint32_t ab) {
            mma_bf16_ts(tmem_base_ + ((r >> 24) << 4), ab + ((r >> 12) & 15u) * 8u, wb + (r & 0xFFFu) * tile16,
                        idesc0 | (((r >> 16) & 0xFFu) << 18));
        };
        const int k0 = fb0 * p.Mb;
        const int m = quarter * 32 + lane, oy = m / p.Wp, ox = m - oy * p.Wp;
        uint32_t use = 0;
        Ring br{0, 0};                                  // TMEM staging buffer
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
                for (int c = 0; c < p.nChunks && ok; ++c, ++use, br.next(p.nabuf)) {
                    const uint32_t slot = use & (p.NWS - 1), buf = (uint32_t)br.idx;
                    // the chunk's MMAs come ready-made; fetch them while the operands may still be on their way
                    const uint32_t *rp = rec_base + (size_t)c * p.RW;
                    const uint4 v0 = *reinterpret_cast<const uint4 *>(rp);
                    const uint4 v1 = *reinterpret_cast<const uint4 *>(rp + 4);
                    {
                        // poll both barriers together: most of the time both have completed already
                        const uint32_t wpar = (use >> (p.NWS == 4 ? 2 : 1)) & 1u;
                        const bool a_ok = mbar_try_wait(&bars->a_full[buf], br.lap & 1), w_ok = mbar_try_wait(&bars->w_full[slot], wpar);
                        // (the decision is the whole warp's, so that elect.sync below always meets all its lanes)
                        bool rdy = a_ok || mbar_wait(&bars->a_full[buf], br.lap & 1, abort_flag, ws, 0x7500 + c);
                        rdy = rdy && (w_ok || mbar_wait(&bars->w_full[slot], wpar, abort_flag, ws, 0x7600 + c));
                        if (!__all_sync(0xFFFFFFFFu, rdy)) { ok = false; break; }
                    }
                    tc_fence_after_sync();
                    const uint32_t wb = (w16 + slot * wcap16) | (8u << 16);          // 128 bytes between the two channel octets
                    const uint32_t ab = tmem_base + 256 + buf * p.bufcols;
                    const uint32_t n = v0.x;
                    if (elect_one()) {
                        if (n > 0) issue(v0.y, wb, ab);
                        if (n > 1) issue(v0.z, wb, ab);
                        if (n > 2) issue(v0.w, wb, ab);
                        if (n > 3) issue(v1.x, wb, ab);
                        if (n > 4) issue(v1.y, wb, ab);
                        if (n > 5) issue(v1.z, wb, ab);
                        if (n > 6) issue(v1.w, wb, ab);
                        for (uint32_t k = 7; k < n; ++k) issue(rp[1 + k], wb, ab);
                        mma_commit(&bars->done[use & (kMaxRing - 1)]);
                    }
                    __syncwarp();
                }
                if (ok && elect_one()) mma_commit(&bars->acc_full);
                __syncwarp();
            }
            ok = __all_sync(0xFFFFFFFFu, ok && !*abort_flag);      // the warp goes on, or stops, as one (elect.sync needs all its lanes)

            // fused epilogue: the warps that share a TMEM lane quarter split the filter columns
            const int n = tile / p.tiles_per_img, y0 = (tile - n * p.tiles_per_img) * p.TR;
            const int yy = y0 + oy;
            const bool valid = oy < p.TR && yy < p.P && ox < p.Q;
            const size_t o0 = (((size_t)n * p.P + yy) * p.Q + ox) * p.K + k0;
            bool go = __all_sync(0xFFFFFFFFu, ok && mbar_wait(&bars->acc_full, it & 1, abort_flag, ws, 0x7700));    // (tcgen05.ld needs the whole warp)
            if (p.epi_tma) go = part == 0 ? bar_all<2, 128>(go) : bar_all<3, 128>(go);        // (the staged epilogue has barriers among the four warps of a column half)
            if (go) {
                tc_fence_after_sync();
                if (p.epi_tma) {
                    epilogue_staged(&tmap_y, smem_u32(smem + p.off_epi) + (uint32_t)part * kEpiBufBytes, bias ? bars->bias : nullptr,
                                    (res && valid) ? static_cast<const uint16_t *>(res) + o0 : nullptr, p.relu != 0,
                                    tmem_base + lane_base, part, (wq & 3) == 0 && lane == 0, m, col_lo, col_hi, k0, y0, n);
                } else
                for (int c0 = col_lo; c0 < col_hi; c0 += 16) {
                    uint32_t r[16];
                    __syncwarp();
                    tmem_ld_x16(tmem_base + lane_base + c0, r);
                    tmem_ld_wait();
                    if (!valid) continue;
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
                    if (bias) {                                  // (an fp32 sum with +0 would be exact too, but costs sixteen loads and adds)
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] += bars->bias[c0 + i];
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
                    if (p.y_bf16) {
                        // one rounding, then ReLU on the packed pairs (max with +0 is exact on the rounded values)
                        uint32_t o[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) o[i] = cvt_bf16x2(v[2 * i], v[2 * i + 1]);
                        if (p.relu) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) o[i] = relu_bf16x2(o[i]);
                        }
                        uint4 *yp = reinterpret_cast<uint4 *>(static_cast<uint16_t *>(y) + o0 + c0);
                        yp[0] = make_uint4(o[0], o[1], o[2], o[3]);
                        yp[1] = make_uint4(o[4], o[5], o[6], o[7]);
                    } else {
                        if (p.relu) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
                        }
                        float4 *yp = reinterpret_cast<float4 *>(static_cast<float *>(y) + o0 + c0);
#pragma unroll
                        for (int h = 0; h < 4; ++h) yp[h] = make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]);
                    }
                }
            } else {
                ok = false;
            }
            // (at the top of the loop every warp zeroes exactly the lanes and columns it has just read.)  All eight warps go
            // on, or stop, as one: there are barriers among them in the loop
            ok = bar_all<1, kMmaWarps * 32>(ok && !*abort_flag);
        }
        if (p.epi_tma && (wq & 3) == 0 && lane == 0) bulk_wait_all();    // the staging buffers stay valid until the stores have read them
    }

    // ---- tear-down ---------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag == 1) {
        // a wait ran out: leave time for copies still in flight to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

bool plan(const npas_conv_desc &d, const npas_bp_desc &bp, ConvKrParams &p, dim3 &grid)
{
    if (d.x_dtype != NPAS_BF16 || bp.w_packed != NPAS_BF16) return false;
    if (d.stride != 1 || d.pad < 0) return false;
    const BpLayout L = bp_layout(bp, 0);
    if (!L.off_kt) return false;                         // Mb, Nb multiples of 16, R*S <= 16, Mb divides the group width
    p.RS = d.R * d.S;
    if (p.RS > kMaxTaps || d.C % 16) return false;
    p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C; p.K = d.K; p.R = d.R; p.S = d.S; p.pad = d.pad;
    p.P = d.H + 2 * d.pad - d.R + 1; p.Q = d.W + 2 * d.pad - d.S + 1;
    if (p.P < 1 || p.Q < 1) return false;
    p.Wp = d.W + 2 * d.pad;
    if (p.Wp > 128) return false;
    p.TR = min(p.P, 128 / p.Wp);
    p.tiles_per_img = (p.P + p.TR - 1) / p.TR;
    p.n_tiles = d.N * p.tiles_per_img;
    p.slab_rows = p.TR + d.R - 1;
    if (p.slab_rows > 256 || p.TR * p.Wp <= d.S - 1) return false;
    p.Mb = bp.Mb; p.GS = (int)L.GS; p.nGrp = (int)L.nGrp; p.nCB = d.C / bp.Nb; p.cpb = bp.Nb / 16;
    if (p.GS > 32 || p.GS * p.Mb > 256) return false;
    p.max_taps = bp.max_taps > 0 ? min(bp.max_taps, d.R * d.S) : d.R * d.S;
    // segments (blocks per issuing warp): as many issuing warps as there are, at most eight
    p.SEG = 1;
    while (p.GS / p.SEG > kMmaWarps) p.SEG *= 2;
    if (p.SEG > 4 || p.GS % p.SEG) return false;
    p.NA = p.GS / p.SEG;
    p.nChunks = d.C / 16;
    p.tile_bytes = (uint32_t)bp.Mb * 32u;
    p.wcap = round_up((uint32_t)p.GS * p.max_taps * p.tile_bytes, 128);
    p.bufcols = (uint32_t)p.RS * 8u;
    p.nabuf = min(kABufs, (int)(256u / p.bufcols));
    if (p.nabuf < 2) return false;
    p.NP = p.nChunks % 2 == 0 ? 2 : 1;
    // per (issuing warp, chunk): a count and at most (SEG + 1) / 2 runs per tap
    p.RW = (1 + p.RS * ((p.SEG + 1) / 2) + 3) & ~3;
    if (p.RW < 8) p.RW = 8;
    p.plane_bytes = (uint32_t)p.slab_rows * p.Wp * 16u;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    const uint32_t reach = (128u + (d.R - 1) * p.Wp + d.S) * 16u;
    const uint32_t slack = reach > p.plane_bytes ? round_up(reach - p.plane_bytes, 128) : 0u;
    bool fits = false;
    for (int nws = kMaxRing; nws >= 2 && !fits; nws /= 2)
        for (int cps = 4; cps >= p.NP && !fits; cps /= 2) {
            if (cps % p.NP || p.nChunks % min(cps, p.nChunks)) continue;
            p.NWS = nws;
            p.cps = min(cps, p.nChunks);
            p.PPS = p.cps * 2;
            p.nStages = (p.nChunks + p.cps - 1) / p.cps;
            p.act_tx_bytes = p.plane_bytes * p.PPS;
            p.act_stage_bytes = round_up(p.act_tx_bytes, 128);
            for (p.SA = 3; p.SA >= 2 && !fits; --p.SA) {
                p.off_act = 0;
                p.off_w = round_up(p.SA * p.act_stage_bytes + slack, 128);
                p.off_cm = p.off_w + p.NWS * p.wcap;
                p.off_kto = p.off_cm + round_up(64u * p.nChunks, 128);
                p.off_rec = p.off_kto + round_up(8u * p.nChunks, 128);
                p.off_bar = p.off_rec + round_up(4u * p.NA * p.nChunks * p.RW, 128);
                // bf16 output in whole 64-filter slabs per column half: staged for tensor stores when there is room
                const bool want_epi = p.y_bf16 && (p.GS * p.Mb) % 128 == 0;
                for (p.epi_tma = want_epi ? 1 : 0; p.epi_tma >= 0 && !fits; --p.epi_tma) {
                    p.off_epi = round_up(p.off_bar + (uint32_t)sizeof(Bars), 1024);
                    p.smem_bytes = (p.epi_tma ? p.off_epi + 2u * kEpiBufBytes : p.off_bar + (uint32_t)sizeof(Bars)) + 1024u;
                    fits = p.smem_bytes <= kSmemLimit && p.plane_bytes * (uint32_t)p.PPS < (1u << 18);
                    if (fits) break;
                }
                if (fits) break;
            }
        }
    if (!fits) return false;
    const int ctas_x = min(p.n_tiles, max(1, sm_count() / p.nGrp));
    if (p.nGrp > 65535) return false;
    grid = dim3(ctas_x, p.nGrp);
    return true;
}

}  // namespace

bool conv_kr_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvKrParams p;
    dim3 grid;
    return plan(d, bp, p, grid);
}

// Where this kernel was measured faster than the dense-image kernels (64x28x28x512 -> 512 with random
// tap sets): up to three taps in nine kept at blocks of 16 filters, up to four in nine at blocks of 32
// filters or more; and only when there is at least one item per SM.
bool conv_kr_preferred(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvKrParams p;
    dim3 grid;
    if (bp.max_taps <= 0 || !plan(d, bp, p, grid)) return false;
    if (p.n_tiles * p.nGrp < sm_count()) return false;
    return bp.Mb >= 32 ? 9 * bp.max_taps <= 4 * p.RS : 3 * bp.max_taps <= p.RS;
}

npas_status conv_kr_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st)
{
    ConvKrParams p;
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
    // Y[N][P][Q][K] bf16 seen as (K, Q, P, N): a box of 64 filters x Wp columns x TR rows is the tile's positions
    // in the order the accumulator lanes hold them; the padding columns fall outside the tensor
    CUtensorMap tmy = tmap;
    if (p.epi_tma) {
        const cuuint64_t ydims[4] = {(cuuint64_t)d.K, (cuuint64_t)p.Q, (cuuint64_t)p.P, (cuuint64_t)d.N};
        const cuuint64_t ystr[3] = {(cuuint64_t)d.K * 2, (cuuint64_t)p.Q * d.K * 2, (cuuint64_t)p.P * p.Q * d.K * 2};
        const cuuint32_t ybox[4] = {64, (cuuint32_t)p.Wp, (cuuint32_t)p.TR, 1};
        const cuuint32_t yes[4] = {1, 1, 1, 1};
        if (enc(&tmy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, y, ydims, ystr, ybox, yes, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return NPAS_ERR_CUDA;
    }
    if (allow_dynamic_smem(reinterpret_cast<const void *>(conv_bp_kr_kernel), (int)kSmemLimit) != NPAS_OK) return NPAS_ERR_CUDA;
    const cudaError_t e = launch_pdl(conv_bp_kr_kernel, grid, dim3(kThreads), p.smem_bytes, st, tmap, tmy, p,
                                     static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return e == cudaSuccess ? launch_status() : NPAS_ERR_CUDA;
}

}  // namespace npas
