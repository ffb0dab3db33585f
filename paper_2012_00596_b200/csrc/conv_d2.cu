// Block-punched convolution from the blob's dense operand image on CTA pairs (tcgen05 cta_group::2).
//
// Same formulation as conv_dn.cu (per 16-channel chunk and tap one MMA over the masked dense
// weights, taps nobody keeps skipped through the tap-union table), with two changes that let the
// tensor pipe run near its rate:
//
// * The activation slab is a 128-byte-swizzled tile, one 128-byte row (64 channels) per padded
//   position, loaded by a 4-D TMA (64 channels, Wp columns, rows, 1 image).  A tap shift is then a
//   start-address offset of whole 128-byte rows, so every operand row the MMA fetches is one
//   aligned line.  In the 16-byte-per-position layout of conv_dn.cu seven of nine tap shifts start in the
//   middle of a line and the A operand costs two shared-memory cycles per eight rows.
// * Two CTAs of a cluster share every MMA: M = 256 positions (each CTA supplies the 128 rows of its
//   own position tile from its own shared memory), N = NT filters of which each CTA holds one half
//   of the B operand (the blob's image, unswizzled [octet][filter][8] tiles as in conv_dn.cu).  A
//   pair halves the weight bytes every SM stages and reads per MMA, and every weight byte fetched
//   from L2 serves twice the positions.
//
// Roles per CTA (384 threads): warp 0 loads the slabs (ring of 64-channel stages), warp 2 loads this CTA's
// half of the weight tiles through a 2-D tensor map laid over the blob (ring of 16- or 32-channel stages),
// warps 1 and 3 of the pair's leader (cluster rank 0) issue the MMAs, one warp per position tile and
// accumulator, and, when they retire, signal the "empty" barriers and at the end of an item the
// "accumulator full" barrier of BOTH CTAs (multicast commit).  Both CTAs' tensor copies complete on the
// LEADER's "full" barriers (the cta_group::2 form of the copy), so no thread tells the leader that the
// other CTA's stage has landed.  Eight warps per CTA run the epilogue on the CTA's own 128 TMEM lanes (bias,
// residual, ReLU, one rounding); the peer's first epilogue warp then hands the accumulator back to the
// leader with ONE arrival that has release semantics at cluster scope, matched by the leader's acquire at
// cluster scope.  Every wait is bounded; a role that gives up raises the abort flag of both CTAs.
#include <cstdio>
#include <cstdlib>

#include "common.cuh"
#include "tc_pair.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kEpiWarps = 8;
constexpr int kParts = kEpiWarps / 4;            // epilogue warps per TMEM lane quarter
constexpr int kFirstEpiWarp = 4;                 // warp 0: slabs, warps 1 and 3: MMA issue (leader), warp 2: weights
constexpr int kThreads = (kFirstEpiWarp + kEpiWarps) * 32;
constexpr int kMaxStages = 8;                    // weight ring
constexpr int kMaxSlabStages = 3;
constexpr int kMaxTapsD2 = 16;
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kDescHiB = (128u >> 4) | (1u << 14);                      // B: no swizzle, SBO = 128 bytes, version bit
constexpr uint32_t kDescHiA = (1024u >> 4) | (1u << 14) | (2u << 29);        // A: 128-byte swizzle, SBO = 1024 bytes, version bit

struct ConvD2Params {
    int N, H, W, C, K, R, S, pad, stride, P, Q, Po, Qo;      // P, Q: the grid of positions the tiles walk
    int nph, sh;                                              // input phases per slab (1, or 4: stride 2 by parity); store shift
    int Wp, TR, tiles_per_img, n_tiles, slab_rows;
    int IT, img_pitch;                                        // small maps: IT whole images per tile, img_pitch positions apart
    int RS, nCh, nBlk, GH, NT, MT, CPW, n_fsets, n_items, SA, SB, nacc, dcols;   // GH: filters per CTA, NT = 2 GH per item; CPW: chunks per weight stage
    int GI;                                                   // filters per group of the blob's operand image (128, or 64 when 128 does not divide K)
    int relu, y_bf16;
    uint32_t slab_bytes, act_stride, a_stage_bytes, w_bytes, off_w, off_tapu, off_bias, off_bar, smem_bytes, tmem_cols;
    uint32_t shift16[kMaxTapsD2];                             // operand start of every tap inside a tile's slabs, 16-byte units
    uint32_t w_box_rows;                                      // 128-byte rows of the blob per weight copy (the weight map's box)
};

struct ConvD2Bars {
    uint64_t a_full[kMaxSlabStages], a_empty[kMaxSlabStages];     // slab ring
    uint64_t w_full[kMaxStages], w_empty[kMaxStages];             // weight ring
    uint64_t acc_full[2], acc_empty[2];
    uint64_t acc_done[2];                                         // peer only: its epilogue warps have read the accumulator
    uint32_t tmem_base;
    uint32_t abort_flag;
};

// A operand (the slab): the swizzle is a function of the shared-memory address itself (bits 4..6 ^= bits
// 7..9, what TMA applied when it wrote the slab), so an operand may start at any 128-byte row of the
// 1024-byte-aligned slab with the descriptor's base-offset field left at zero (checked tap by tap
// against the oracle).
// The MMAs of one 16-channel chunk: tap t (bit t of `taps`) multiplies the slab at a_lo + shift[t] by the
// weight tile at b_lo + t * b_step (both low descriptor words, the high words are constants); the first
// MMA of an item (tap 0 of chunk 0) overwrites the accumulator.  One thread issues all of them and an
// MMA costs it about 80 cycles by itself, so everything else per MMA is two additions; when every tap
// is present (any mask that is not structured) there are no tests either.
template <int NTAPS>
__device__ __forceinline__ void issue_taps(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t b_step,
                                           const uint32_t (&shift)[kMaxTapsD2], uint32_t taps, uint32_t idesc, bool accumulate0)
{
    constexpr uint64_t hi_a = (uint64_t)kDescHiA << 32, hi_b = (uint64_t)kDescHiB << 32;
    if (NTAPS == 9 && taps == 0x1FFu) {
#pragma unroll
        for (int t = 0; t < NTAPS; ++t, b_lo += b_step)
            mma_bf16_ss_pair(d_tmem, hi_a | (a_lo + shift[t]), hi_b | b_lo, idesc, (t > 0 || accumulate0) ? 1u : 0u);
        return;
    }
#pragma unroll
    for (int t = 0; t < NTAPS; ++t, b_lo += b_step)
        if ((taps >> t) & 1u)
            mma_bf16_ss_pair(d_tmem, hi_a | (a_lo + shift[t]), hi_b | b_lo, idesc, (t > 0 || accumulate0) ? 1u : 0u);
}
// the same, completing on a barrier of the pair's leader (cluster address): the cta_group::2 form of the copy
__device__ __forceinline__ void tma_load_4d_pair(void *dst, const CUtensorMap *m, uint32_t bar_cluster_addr, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// barrier among all warps but the two producers
__device__ __forceinline__ void consumers_sync() { asm volatile("bar.sync 3, %0;" ::"n"(kThreads - 64) : "memory"); }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
conv_bp_d2_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, const ConvD2Params p,
                  const uint8_t *__restrict__ blob, const float *__restrict__ bias,
                  const void *__restrict__ res, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint32_t *tapu_s = reinterpret_cast<uint32_t *>(smem + p.off_tapu);     // [K / GI][nCh]
    float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);           // [K]
    ConvD2Bars *bars = reinterpret_cast<ConvD2Bars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                  // 0: leader (issues the MMAs), 1: its peer
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    const uint32_t peer_abort = map_to_cta(smem_u32(&bars->abort_flag), rank ^ 1u);

    if (tid == 0) {
        // The tensor copies of both CTAs (slabs, and the weights through a tensor map laid over the blob)
        // complete on the LEADER's "full" barriers, for which the leader's producers announce the bytes of
        // both: nothing is relayed by a thread.  One issuing warp per position tile commits on the "empty"
        // and "accumulator full" barriers; an accumulator is free again when the leader's epilogue warps and
        // the peer's single relayed arrival have come in.
        for (int s = 0; s < p.SA; ++s) { mbar_init(&bars->a_full[s], 1); mbar_init(&bars->a_empty[s], p.MT); }
        for (int s = 0; s < p.SB; ++s) { mbar_init(&bars->w_full[s], 1); mbar_init(&bars->w_empty[s], p.MT); }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->acc_full[a], p.MT); mbar_init(&bars->acc_empty[a], kEpiWarps + 1); mbar_init(&bars->acc_done[a], kEpiWarps);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) tmem_alloc_pair(&bars->tmem_base, p.tmem_cols);      // both CTAs; warp 1 also frees it
    pdl_trigger();
    tc_fence_before_sync();
    cluster_sync_all();                 // barriers of both CTAs exist before anything arrives on them
    tc_fence_after_sync();
    pdl_wait();                         // nothing above touches global memory
    const uint32_t tmem_base = bars->tmem_base;
    // the two producers start at once; the other warps first stage the biases and the tap unions
    if (warp != 0 && warp != 2) {
        const int t = tid < 64 ? tid - 32 : tid - 64;         // 0 .. kThreads - 65 over warps 1, 3, 4, ...
        for (int i = t; i < p.K; i += kThreads - 64) bias_s[i] = bias ? bias[i] : 0.f;
        const uint32_t off_tapu = hdr[BP_OFF_TAPU];
        const uint32_t *tapu = reinterpret_cast<const uint32_t *>(blob + off_tapu);
        for (int i = t; i < (p.K / p.GI) * p.nCh; i += kThreads - 64) tapu_s[i] = off_tapu ? tapu[i] : 0xFFFFFFFFu;
        if (p.IT > 1 && p.act_stride > p.slab_bytes) {
            // several images per tile: the last image's bottom-right taps read just past the slab, where no copy
            // ever writes: zeros, once, in every buffer of the ring (read by the tensor core: async proxy)
            const uint32_t tail = p.act_stride - p.slab_bytes, nbuf = (uint32_t)(p.SA * p.MT * p.nph);
            for (uint32_t i = (uint32_t)t * 16u; i < nbuf * tail; i += (kThreads - 64) * 16u) {
                const uint32_t b = i / tail, o = i - b * tail;
                *reinterpret_cast<uint4 *>(smem + (size_t)(b / (uint32_t)(p.MT * p.nph)) * p.a_stage_bytes +
                                           (size_t)(b % (uint32_t)(p.MT * p.nph)) * p.act_stride + p.slab_bytes + o) = make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async_smem();
        }
        consumers_sync();
    }

    if (warp == 0) {
        // ---- slab producer: this CTA's position tiles, one 64-channel block per stage ----------------------
        if (lane == 0) {
            uint32_t n = 0;                                   // stages issued so far
            bool ok = true;
            const uint32_t a_full0 = map_to_cta(smem_u32(&bars->a_full[0]), 0u);      // the leader's barriers
            for (int item = pair; item < p.n_items && ok; item += n_pairs) {
                const int ts = item / p.n_fsets;
                for (int blk = 0; blk < p.nBlk; ++blk, ++n) {
                    const uint32_t s = n % (uint32_t)p.SA, k = n / (uint32_t)p.SA;
                    if (k >= 1 && !pair_wait(&bars->a_empty[s], (k - 1u) & 1u, abort_flag, peer_abort, ws, 0x7100)) { ok = false; break; }
                    uint8_t *st = smem + (size_t)s * p.a_stage_bytes;
                    if (rank == 0) mbar_arrive_expect_tx(&bars->a_full[s], 2u * (uint32_t)(p.MT * p.nph) * p.slab_bytes);
                    for (int mt = 0; mt < p.MT; ++mt) {
                        const int tile = min((ts * 2 + (int)rank) * p.MT + mt, p.n_tiles - 1);   // a missing tile repeats the last one
                        const int img = p.IT > 1 ? tile * p.IT : tile / p.tiles_per_img;
                        const int y0 = p.IT > 1 ? 0 : (tile - img * p.tiles_per_img) * p.TR;
                        uint8_t *dst = st + (size_t)(mt * p.nph) * p.act_stride;
                        if (p.nph == 1) {
                            tma_load_4d_pair(dst, &tmap_x, a_full0 + s * 8u, blk * 64, -p.pad, y0 - p.pad, img);
                        } else {
                            // phase (a, b) = the input pixels (2 i + a, 2 j + b), i from y0 - 1, j from -1; the tensor
                            // map steps by two pixels in both directions
                            for (int ph = 0; ph < 4; ++ph)
                                tma_load_4d_pair(dst + (size_t)ph * p.act_stride, &tmap_x, a_full0 + s * 8u, blk * 64,
                                            (ph & 1) - 2, 2 * (y0 - 1) + (ph >> 1), img);
                        }
                    }
                }
            }
            // do not leave while the leader's commits may still arrive on this CTA's barriers
            for (uint32_t e = n; e < n + (uint32_t)p.SA && ok; ++e) {
                const uint32_t s = e % (uint32_t)p.SA, k = e / (uint32_t)p.SA;
                if (k >= 1 && !pair_wait(&bars->a_empty[s], (k - 1u) & 1u, abort_flag, peer_abort, ws, 0x7110)) break;
            }
        }
    } else if (warp == 2) {
        // ---- weight producer: this CTA's half of the weight tile of every 16-channel chunk ----------------
        const uint32_t off_image = hdr[BP_OFF_IMAGE];
        bool ok = true;
        // the blob must carry the operand image in the groups the plan assumed; if not, nothing is requested
        // and the other roles leave their waits through the abort flag
        if (off_image == 0u || (off_image & 2047u) || hdr[BP_GI] != (uint32_t)p.GI) {
            if (lane == 0) {
                bars->abort_flag = 2;
                st_remote_u32(peer_abort, 2u);
                if (atomicCAS(ws, 0u, 6u /* NPAS_ERR_BLOB */) == 0u) ws[1] = 0x7001;
            }
            ok = false;
        }
        // A CTA holding 128 filters fetches the whole tile of its image group, one contiguous run, in a few
        // large copies (boxes of 128-byte rows).  One holding 64 fetches its half of every (tap, octet) row of
        // 2048 bytes: the weight map is then four-dimensional (128 bytes, 8 lines of a half, 2 halves, rows of
        // 2048 bytes) and ONE box (128, 8, 1, rows of the stage) brings the stage's halves back to back (36
        // separate 1 KB copies per stage cost the issuing warp 2.5 k cycles, more than the stage's MMAs take).
        const int rows_st = 2 * p.RS * p.CPW;                 // weight rows (chunk, tap, octet) of a stage
        const uint32_t copy_bytes = p.w_box_rows * 128u;      // 128 filters: one copy = one box of the weight map
        const int n_copies = p.GH == 128 ? (int)(p.w_bytes / copy_bytes) : 1;
        const uint32_t grow = (uint32_t)p.GI * 16u;           // bytes of a (tap, octet) row of the image: GI filters x 8 channels
        const uint32_t w_full0 = map_to_cta(smem_u32(&bars->w_full[0]), 0u);      // the leader's barriers
        const uint32_t image_row0 = off_image >> 7;           // the weight map counts the blob in 128-byte rows
        uint32_t n = 0;
        for (int item = pair; item < p.n_items && ok; item += n_pairs) {
            const int fs = item % p.n_fsets;
            const int f0 = fs * p.NT + (int)rank * p.GH;      // first filter of this CTA's half
            const uint32_t wsrc = image_row0 + (uint32_t)(((size_t)(f0 / p.GI) * p.nCh * (2u * p.RS * grow) + (size_t)(f0 % p.GI) * 16u) >> 7);
            for (int wst = 0; wst < p.nCh / p.CPW; ++wst, ++n) {
                const uint32_t s = n % (uint32_t)p.SB, k = n / (uint32_t)p.SB;
                if (lane == 0) {
                    if (k >= 1 && !pair_wait(&bars->w_empty[s], (k - 1u) & 1u, abort_flag, peer_abort, ws, 0x7120)) ok = false;
                    if (ok && rank == 0) mbar_arrive_expect_tx(&bars->w_full[s], 2u * p.w_bytes);
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                uint8_t *wdst = smem + p.off_w + (size_t)s * p.w_bytes;
                const uint32_t src = wsrc + (uint32_t)wst * (uint32_t)rows_st * (grow >> 7);     // rows of the image, in 128-byte map rows
                if (p.GH == 128) {
                    for (int i = lane; i < n_copies; i += 32)
                        tma_load_2d_pair(wdst + (size_t)i * copy_bytes, &tmap_w, w_full0 + s * 8u, 0, (int)(src + (uint32_t)i * p.w_box_rows));
                } else if (lane == 0) {
                    tma_load_4d_pair(wdst, &tmap_w, w_full0 + s * 8u, 0, 0, (int)rank, (int)(src / (grow >> 7)));    // (src counts 128-byte rows)
                }
            }
        }
        if (lane == 0 && ok) {
            for (uint32_t e = n; e < n + (uint32_t)p.SB; ++e) {
                const uint32_t s = e % (uint32_t)p.SB, k = e / (uint32_t)p.SB;
                if (k >= 1 && !pair_wait(&bars->w_empty[s], (k - 1u) & 1u, abort_flag, peer_abort, ws, 0x7130)) break;
            }
        }
    } else if (warp == 1 || warp == 3) {
        const int wst_blk = 4 / p.CPW;                        // weight stages per 64-channel block
        // (the peer has no part in this role: its copies complete on the leader's barriers by themselves)
        if (rank == 0 && (warp >> 1) < p.MT) {
            // ---- leader: MMA issue for the pair; this warp owns the accumulator of position tile mt, so the
            // order of summation is fixed ----------------------------------------------------------------
            // (one thread; its own instructions are on the critical path, so ring positions and operand
            // addresses are carried along instead of being divided out per stage)
            if (elect_one()) {
                const int mt = warp >> 1;
                const uint32_t idesc = idesc_bf16_f32(256, p.NT);
                const uint32_t base16 = smem_u32(smem) >> 4, a_stage16 = p.a_stage_bytes >> 4;
                const uint32_t tile16 = (uint32_t)p.nph * (p.act_stride >> 4), w16 = p.w_bytes >> 4;
                uint32_t shift[kMaxTapsD2];
#pragma unroll
                for (int t = 0; t < kMaxTapsD2; ++t) shift[t] = p.shift16[t];
                const uint32_t b_hi = (uint32_t)p.GH << 16, b_step = 2u * p.GH, chunk16 = (uint32_t)p.RS * b_step;
                const uint32_t a_base = (base16 + (uint32_t)mt * tile16) | (1u << 16), b_base = (base16 + (p.off_w >> 4)) | b_hi;
                const int ngrp = p.NT / p.GI;                   // groups of the image per item (1 or 2)
                uint32_t sa = 0, pha = 0, a_st = a_base, sb = 0, phb = 0, b_st = b_base, it = 0;
                bool ok = true;
                for (int item = pair; item < p.n_items && ok; item += n_pairs, ++it) {
                    const int fs = item % p.n_fsets;
                    const uint32_t acc = p.nacc == 2 ? (it & 1u) : 0u, lap_acc = p.nacc == 2 ? (it >> 1) : it;
                    if (lap_acc >= 1 && !pair_wait<true>(&bars->acc_empty[acc], (lap_acc & 1u) ^ 1u, abort_flag, peer_abort, ws, 0x7200)) break;
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + acc * p.dcols + (uint32_t)mt * p.NT;
                    const uint32_t *tu = tapu_s + (fs * ngrp) * p.nCh;
                    int ch = 0;
                    for (int blk = 0; blk < p.nBlk && ok; ++blk) {
                        if (!pair_wait(&bars->a_full[sa], pha, abort_flag, peer_abort, ws, 0x7300)) { ok = false; break; }
                        uint32_t a16 = a_st;                    // 16 channels = 32 bytes inside the swizzled 128-byte row
                        for (int q = 0; q < wst_blk; ++q) {
                            if (!pair_wait(&bars->w_full[sb], phb, abort_flag, peer_abort, ws, 0x7320)) { ok = false; break; }
                            tc_fence_after_sync();
                            uint32_t b_lo = b_st;
                            for (int cc = 0; cc < p.CPW; ++cc, ++ch, a16 += 2u, b_lo += chunk16) {
                                // a tap that no block of these (groups, chunk) keeps multiplies zeros: skipped, except
                                // the very first MMA, which initialises the accumulator
                                uint32_t m = tu[ch] | (ch == 0 ? 1u : 0u);
                                if (ngrp == 2) m |= tu[p.nCh + ch];
                                if (p.RS == 9) issue_taps<9>(d_tmem, a16, b_lo, b_step, shift, m, idesc, ch != 0);
                                else issue_taps<kMaxTapsD2>(d_tmem, a16, b_lo, b_step, shift, m & ((1u << p.RS) - 1u), idesc, ch != 0);
                            }
                            mma_commit_pair(&bars->w_empty[sb]);
                            b_st += w16;
                            if (++sb == (uint32_t)p.SB) { sb = 0; phb ^= 1u; b_st = b_base; }
                        }
                        if (!ok) break;
                        mma_commit_pair(&bars->a_empty[sa]);
                        if (blk == p.nBlk - 1) mma_commit_pair(&bars->acc_full[acc]);
                        a_st += a_stage16;
                        if (++sa == (uint32_t)p.SA) { sa = 0; pha ^= 1u; a_st = a_base; }
                    }
                }
            }
        }
    } else {
        // ---- epilogue: warp -> TMEM lane quarter (warp % 4) and every kParts-th 16-column chunk -----------
        const int quarter = warp & 3, part = (warp - kFirstEpiWarp) >> 2, m = quarter * 32 + lane;
        const int il = p.IT > 1 ? m / p.img_pitch : 0, mr = m - il * p.img_pitch;    // image of the tile, position inside it
        const int oy = mr / p.Wp, ox = mr - oy * p.Wp;
        const int cpt = p.NT / 16;                          // chunks per position tile
        const int sh = p.sh;                                // positions computed but not stored: divide by shifting
        const uint32_t acc_empty0 = map_to_cta(smem_u32(&bars->acc_empty[0]), 0u);   // the leader's
        uint32_t it = 0;
        bool ok = true;
        for (int item = pair; item < p.n_items && ok; item += n_pairs, ++it) {
            const int ts = item / p.n_fsets, fs = item - ts * p.n_fsets;
            const uint32_t acc = p.nacc == 2 ? (it & 1u) : 0u, lap_acc = p.nacc == 2 ? (it >> 1) : it;
            const int nch = p.MT * cpt;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * p.dcols;

            // where this thread's position of each tile goes (MT <= 2); with a stride the tile is computed
            // at every position and only the strided ones are stored (stride is 1 or 2)
            bool val[2];
            size_t obase[2];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const int tile_raw = (ts * 2 + (int)rank) * p.MT + mt, tile = min(tile_raw, p.n_tiles - 1);
                const int img = p.IT > 1 ? tile * p.IT + il : tile / p.tiles_per_img;
                const int yy = p.IT > 1 ? oy : (tile - img * p.tiles_per_img) * p.TR + oy;
                val[mt] = mt < p.MT && tile_raw < p.n_tiles && il < p.IT && img < p.N && oy < p.TR && yy < p.P && ox < p.Q && ((yy | ox) & sh) == 0;
                obase[mt] = (((size_t)img * p.Po + (yy >> sh)) * p.Qo + (ox >> sh)) * p.K;
            }
            auto finish = [&](const uint32_t (&r)[16], int j) {
                const int mt = j >= cpt ? 1 : 0, c0 = (j - mt * cpt) * 16;
                if (!(mt ? val[1] : val[0])) return;
                const int k0 = fs * p.NT + c0;
                const size_t o0 = (mt ? obase[1] : obase[0]) + k0;
                float v[16];
                const float4 *b4 = reinterpret_cast<const float4 *>(bias_s + k0);
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float4 u = b4[h];
                    v[4 * h] = __uint_as_float(r[4 * h]) + u.x; v[4 * h + 1] = __uint_as_float(r[4 * h + 1]) + u.y;
                    v[4 * h + 2] = __uint_as_float(r[4 * h + 2]) + u.z; v[4 * h + 3] = __uint_as_float(r[4 * h + 3]) + u.w;
                }
                if (res) {
                    if (p.y_bf16) {
                        const uint4 *rp = reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(res) + o0);
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
                        const float4 *rp = reinterpret_cast<const float4 *>(static_cast<const float *>(res) + o0);
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
                    uint4 *yp = reinterpret_cast<uint4 *>(static_cast<uint16_t *>(y) + o0);
                    yp[0] = make_uint4(o[0], o[1], o[2], o[3]);
                    yp[1] = make_uint4(o[4], o[5], o[6], o[7]);
                } else {
                    if (p.relu) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
                    }
                    float4 *yp = reinterpret_cast<float4 *>(static_cast<float *>(y) + o0);
#pragma unroll
                    for (int h = 0; h < 4; ++h) yp[h] = make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]);
                }
            };

            if (!pair_wait(&bars->acc_full[acc], lap_acc & 1u, abort_flag, peer_abort, ws, 0x7400)) { ok = false; break; }
            tc_fence_after_sync();
            // two register sets: the next chunk is on its way out of TMEM while this one is finished
            uint32_t ra[16], rb[16];
            int j = part;
            if (j < nch) tmem_ld_x16(t_addr + j * 16, ra);
            while (j < nch) {
                tmem_ld_wait();
                if (j + kParts < nch) tmem_ld_x16(t_addr + (j + kParts) * 16, rb);
                finish(ra, j);
                j += kParts;
                if (j >= nch) break;
                tmem_ld_wait();
                if (j + kParts < nch) tmem_ld_x16(t_addr + (j + kParts) * 16, ra);
                finish(rb, j);
                j += kParts;
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(rank == 0 ? &bars->acc_empty[acc] : &bars->acc_done[acc]);
            if (rank == 1 && warp == kFirstEpiWarp && lane == 0) {
                // peer: once all its epilogue warps have read the accumulator, ONE arrival on the leader's barrier
                // with release semantics at cluster scope (the leader needs the accumulator an item later)
                if (!mbar_wait(&bars->acc_done[acc], lap_acc & 1u, abort_flag, ws, 0x7520)) { ok = false; }
                else {
                    tc_fence_after_sync();
                    tc_fence_before_sync();
                    mbar_arrive_remote_release(acc_empty0 + acc * 8u);
                }
            }
            __syncwarp();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        // a role gave up: leave time for copies still in flight to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) { }
    }
    cluster_sync_all();                 // neither CTA retires (or frees TMEM) while the other may still use it
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, p.tmem_cols);
    }
}

int pairs_available() { return sm_count() / 2; }

bool plan(const npas_conv_desc &d, const npas_bp_desc &bp, ConvD2Params &p, int pairs)
{
    if (d.x_dtype != NPAS_BF16 || bp.w_packed != NPAS_BF16) return false;
    if ((d.stride != 1 && d.stride != 2) || d.pad < 0 || d.C % 64 || d.K % 64) return false;
    p.GI = (int)bp_layout(bp, 0).GI;                      // 128, or 64 when 128 does not divide K
    if (p.GI != 64 && p.GI != 128) return false;
    p.RS = d.R * d.S;
    if (p.RS > kMaxTapsD2) return false;
    p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C; p.K = d.K; p.R = d.R; p.S = d.S; p.pad = d.pad; p.stride = d.stride;
    p.P = d.H + 2 * d.pad - d.R + 1; p.Q = d.W + 2 * d.pad - d.S + 1;
    if (p.P < 1 || p.Q < 1) return false;
    p.Po = (p.P - 1) / d.stride + 1; p.Qo = (p.Q - 1) / d.stride + 1;
    // Stride 2 with a 3x3 kernel and pad 1: the input is taken apart by the parity of its coordinates
    // into four phase images, in each of which a tap is a stride-1 access, and only the wanted positions
    // are computed (output (p, q), tap (r, s) reads phase ((r - 1) & 1, (s - 1) & 1) at (p + dr, q + ds),
    // dr, ds = -1 for r, s = 0, else 0).  Any other strided geometry is computed at every stride-1
    // position and the epilogue stores every other one.
    const bool phases = d.stride == 2 && d.R == 3 && d.S == 3 && d.pad == 1;
    p.nph = phases ? 4 : 1;
    p.sh = phases ? 0 : d.stride - 1;
    uint32_t reach;
    if (phases) {
        p.P = p.Po; p.Q = p.Qo;                       // the tiles walk the output grid itself
        p.Wp = p.Qo + 1;                              // one column to the left (ds = -1)
        if (p.Wp > 128) return false;
        p.TR = min(p.P, 128 / p.Wp);
        p.slab_rows = p.TR + 1;                       // one row above (dr = -1)
        reach = (128u + (uint32_t)p.Wp + 1u) * 128u;
    } else {
        p.Wp = d.W + 2 * d.pad;
        if (p.Wp > 128) return false;
        p.TR = min(p.P, 128 / p.Wp);
        p.slab_rows = p.TR + d.R - 1;
        reach = (128u + (uint32_t)(d.R - 1) * p.Wp + d.S) * 128u;
    }
    p.tiles_per_img = (p.P + p.TR - 1) / p.TR;
    p.n_tiles = d.N * p.tiles_per_img;
    if (p.slab_rows > 128) return false;
    // Small maps (a whole image in less than half a tile): several images per tile, their slabs one behind the other
    // (one box over the image dimension).  Without phases the rows are W + pad positions wide instead of W + 2 pad: a
    // row's right border is the next row's left border, and the slab's last row the next image's first.
    p.IT = 1; p.img_pitch = 0;
    if (p.TR == p.P && (phases || (d.stride == 1 && d.R - 1 == 2 * d.pad && d.S - 1 == 2 * d.pad))) {
        const int Wq = phases ? p.Wp : d.W + d.pad, pitch = p.slab_rows * Wq;
        int it = 1 + (128 - ((p.P - 1) * Wq + p.Q)) / pitch;           // images whose stored positions fit into 128 lanes
        it = min(min(it, d.N), 16);
        if (it >= 2) {
            p.IT = it; p.Wp = Wq; p.img_pitch = pitch;
            p.tiles_per_img = 1;
            p.n_tiles = (d.N + it - 1) / it;
            if (!phases) reach = (128u + (uint32_t)(d.R - 1) * p.Wp + d.S) * 128u;
        }
    }
    p.nCh = d.C / 16; p.nBlk = d.C / 64;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    p.slab_bytes = (uint32_t)(p.IT * p.slab_rows) * p.Wp * 128u;
    // a shifted operand reads 128 rows from its start: room behind the slab (what lies there only reaches
    // positions that are not stored)
    p.act_stride = round_up(reach > p.slab_bytes ? reach : p.slab_bytes, 1024);
    for (int t = 0; t < kMaxTapsD2; ++t) p.shift16[t] = 0;
    for (int t = 0; t < p.RS; ++t) {
        const int r = t / d.S, sx = t % d.S;
        if (phases) {
            const int a = (r - 1) & 1, b = (sx - 1) & 1, dr = r == 0 ? -1 : 0, ds = sx == 0 ? -1 : 0;
            p.shift16[t] = (uint32_t)(a * 2 + b) * (p.act_stride >> 4) + (uint32_t)((dr + 1) * p.Wp + ds + 1) * 8u;
        } else {
            p.shift16[t] = (uint32_t)(r * p.Wp + sx) * 8u;
        }
    }
    const uint32_t fixed = round_up((uint32_t)(d.K / p.GI) * p.nCh * 4u, 128) + round_up((uint32_t)d.K * 4u, 128) +
                           (uint32_t)sizeof(ConvD2Bars) + 1024u + 256u;
    if (fixed >= kSmemLimit) return false;
    const uint32_t avail = kSmemLimit - fixed;
    // filters per item (NT) and position tiles per CTA (MT): the combination with the least modelled time,
    // rounds of items over the pairs x (MMA cycles of an item + its epilogue where that is not overlapped)
    // (the call descriptor's `variant`, NT + (MT << 16), restricts the choice to one combination)
    const int want_nt = d.variant & 0xFFFF, want_mt = (d.variant >> 16) & 0xFFFF;
    double best = 0.;
    bool found = false;
    for (int NT = 256; NT >= 64; NT >>= 1) {
        // an item is one or two groups of the image (with groups of 64 filters: one)
        if (d.K % NT || (want_nt && NT != want_nt) || NT < p.GI || (p.GI == 64 && NT != 64)) continue;
        for (int MT = 1; MT <= 2; ++MT) {
            if (MT * NT > 512 || (want_mt && MT != want_mt)) continue;
            if (MT > 1 && p.n_tiles < 4) continue;
            ConvD2Params q = p;
            q.NT = NT; q.GH = NT / 2; q.MT = MT; q.n_fsets = d.K / NT;
            const long long items = (long long)((p.n_tiles + 2 * MT - 1) / (2 * MT)) * q.n_fsets;
            if (items > 0x7FFFFFFF) return false;
            q.n_items = (int)items;
            q.a_stage_bytes = (uint32_t)(MT * p.nph) * p.act_stride;
            // a weight stage holds two chunks of a 64-filter half (32 KB at nine taps, as one chunk of a
            // 128-filter half), one where the slabs leave no room for two such stages
            q.CPW = q.GH == 64 ? 2 : q.GH == 32 ? 4 : 1;
            while (q.CPW > 1 && p.nCh % q.CPW) q.CPW /= 2;
            q.w_bytes = (uint32_t)q.CPW * p.RS * 2u * q.GH * 16u;
            while (q.CPW > 1 && 2u * q.a_stage_bytes + 2u * q.w_bytes > avail) { q.CPW /= 2; q.w_bytes /= 2; }
            q.dcols = MT * NT;
            q.nacc = 2 * q.dcols <= 512 ? 2 : 1;
            // two slab stages, the rest of shared memory for weight stages; a third slab stage if at least
            // four weight stages remain
            if (2u * q.a_stage_bytes + 2u * q.w_bytes > avail) continue;
            q.SA = (p.nBlk >= 3 && 3u * q.a_stage_bytes + 4u * q.w_bytes <= avail) ? 3 : 2;
            q.SB = (int)((avail - (uint32_t)q.SA * q.a_stage_bytes) / q.w_bytes);
            if (q.SB > kMaxStages) q.SB = kMaxStages;
            if ((uint32_t)q.SA * q.a_stage_bytes + (uint32_t)q.SB * q.w_bytes >= (1u << 18)) continue;   // descriptor addresses are 14 bits of 16 bytes
            // An MMA of a pair takes the tensor pipe NT / 2 cycles, and its issuing thread 50 to 100.  The epilogue
            // of an item overlaps the next item's MMAs when two accumulators fit, and always costs once at the
            // end; measured on every shape tried (64 to 448 position tiles, 128 to 512 filters, stride 1 and 2),
            // 128 filters and one position tile per CTA is the fastest combination or within 1 % of it: more,
            // smaller items fill the pairs better and leave less epilogue exposed.
            const double rounds = (double)((items + pairs - 1) / pairs);
            const double per_mma = NT / 2 > 70 ? NT / 2 : 70.;
            // (two position tiles have an issuing warp each; at 64 filters the pipe (32 cycles) keeps up with both:
            // 56x56x64 -> 64, 23.7 us on two tiles per CTA against 26.5 on one)
            const double mma = (double)p.nCh * p.RS * (NT == 64 && MT == 2 ? per_mma : MT * per_mma);
            const double epi = (double)MT * NT * 16.;
            const double cost = (rounds * (mma + (q.nacc == 2 ? 0. : epi)) + epi + 6000.) * ((NT == 128 && MT == 1) ? 0.9 : 1.);
            if (!found || cost < best) { best = cost; p = q; found = true; }
        }
    }
    if (!found) return false;
    p.off_w = (uint32_t)p.SA * p.a_stage_bytes;
    p.off_tapu = p.off_w + (uint32_t)p.SB * p.w_bytes;
    p.off_bias = p.off_tapu + round_up((uint32_t)(d.K / p.GI) * p.nCh * 4u, 128);
    p.off_bar = p.off_bias + round_up((uint32_t)d.K * 4u, 128);
    p.smem_bytes = p.off_bar + sizeof(ConvD2Bars) + 1024;
    if (p.smem_bytes > kSmemLimit) return false;
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < p.nacc * p.dcols) p.tmem_cols *= 2;
    return true;
}

}  // namespace

bool conv_d2_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvD2Params p;
    return plan(d, bp, p, pairs_available());
}

// Whether the pair kernel is the better of the two dense-image kernels for this call (measured): always
// for the strided 3x3 geometry it computes by phases (a quarter of the MMAs); else as soon as there are
// 64 items of 128 positions x 128 filters (half a wave of pairs): 11.4 against 13.7 us on 32x14x14x256 -> 256,
// 17.5 against 22.0 on 64x28x28x128 -> 128, 26 against 36 on 64x7x7x512 -> 512.  Smaller problems stay on
// independent CTAs.
bool conv_d2_preferred(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvD2Params p;
    const int pairs = pairs_available();
    if (pairs < 1 || !plan(d, bp, p, pairs)) return false;
    if (p.nph == 4) return true;
    return (long long)p.n_tiles * ((d.K + 127) / 128) >= 64;
}

npas_status conv_d2_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st)
{
    ConvD2Params p;
    const int pairs = pairs_available();
    if (pairs < 1 || !plan(d, bp, p, pairs)) return NPAS_ERR_UNSUPPORTED;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return NPAS_ERR_CUDA;
    // X[N][H][W][C] bf16 as (C, W, H, N): a box of 64 channels x Wp columns x slab rows lands in shared
    // memory as one 128-byte-swizzled row per padded position; out-of-image positions are zero-filled
    CUtensorMap tmap;
    const cuuint64_t dims[4] = {(cuuint64_t)d.C, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N};
    const cuuint64_t strides[3] = {(cuuint64_t)d.C * 2, (cuuint64_t)d.W * d.C * 2, (cuuint64_t)d.H * d.W * d.C * 2};
    // (phase slabs: every other column and row, so the box spans twice as many pixels as it delivers)
    const cuuint32_t step = p.nph == 4 ? 2 : 1;
    const cuuint32_t box[4] = {64, (cuuint32_t)p.Wp * step, (cuuint32_t)p.slab_rows * step, (cuuint32_t)p.IT};
    const cuuint32_t estr[4] = {1, step, step, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return NPAS_ERR_CUDA;
    // The blob seen through a tensor map, so that the weight copies are tensor copies too (only those can complete
    // on the other CTA's barrier).  The blob's length depends on how many blocks were kept, which only its header
    // knows: the map is given the length of a blob that keeps everything, and the kernel asks for rows of the
    // operand image only, which every blob of this description holds in full.  A CTA holding 128 filters: rows of
    // 128 bytes, a stage is one run fetched in a few boxes.  A CTA holding 64 filters: (128 bytes, 8 lines of a
    // half row, 2 halves, rows of 2048 bytes), one box per stage (the image starts on a multiple of 2048 bytes).
    CUtensorMap tmap_w;
    const uint32_t all_pairs = (uint32_t)(bp.K / bp.Mb) * (uint32_t)(bp.C / bp.Nb) * (uint32_t)(bp.R * bp.S);
    const uint32_t blob_bytes = bp_layout(bp, all_pairs).total;
    if (p.GH == 128) {
        const uint32_t rows = p.w_bytes / 128u;
        p.w_box_rows = 256;
        while (rows % p.w_box_rows) --p.w_box_rows;
        const cuuint64_t wdims[2] = {128, (cuuint64_t)(blob_bytes / 128u)};
        const cuuint64_t wstrides[1] = {128};
        const cuuint32_t wbox[2] = {128, p.w_box_rows};
        const cuuint32_t westr[2] = {1, 1};
        if (enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(blob), wdims, wstrides, wbox, westr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return NPAS_ERR_CUDA;
    } else {
        // (a half row is GH filters x 16 bytes: 8 lines of 128 bytes at 64 filters, 4 at 32)
        const uint32_t half = (uint32_t)p.GH * 16u, lines = half / 128u;
        p.w_box_rows = lines;
        const cuuint64_t wdims[4] = {128, lines, 2, (cuuint64_t)(blob_bytes / (2u * half))};
        const cuuint64_t wstrides[3] = {128, half, 2u * half};
        const cuuint32_t wbox[4] = {128, lines, 1, (cuuint32_t)(2 * p.RS * p.CPW)};
        const cuuint32_t westr[4] = {1, 1, 1, 1};
        if (enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(blob), wdims, wstrides, wbox, westr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return NPAS_ERR_CUDA;
    }
    if (allow_dynamic_smem(reinterpret_cast<const void *>(conv_bp_d2_kernel), (int)kSmemLimit) != NPAS_OK) return NPAS_ERR_CUDA;
    const int n_pairs = p.n_items < pairs ? p.n_items : pairs;
    const cudaError_t e = launch_pdl(conv_bp_d2_kernel, dim3(2 * n_pairs), dim3(kThreads), p.smem_bytes, st, tmap, tmap_w, p,
                                     static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return e == cudaSuccess ? launch_status() : NPAS_ERR_CUDA;
}

}  // namespace npas
