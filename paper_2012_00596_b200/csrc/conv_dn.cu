// Block-punched convolution on the sm_100a tensor cores from the blob's dense operand image.
//
// The kept-only kernels issue one small MMA (N = Mb filters) per kept (block, tap) pair; at the
// block sizes of interest (4x4 ... 32x32) those MMAs and the activation copies into tensor memory
// that feed them cost more tensor-pipe time than the pruned taps save, and blocks narrower than 16
// filters cannot use the tensor core at all.  This kernel multiplies the masked dense weights
// instead, stored by the packer as ready-made operand tiles (section `image` of the blob): per
// 16-channel chunk and tap one MMA of M = 128 positions x N = GI filters (GI = 128 when K allows),
// both operands from shared memory, which runs at the tensor pipe's full rate and works for every
// block size.  A tap that no block of the (filter group, chunk) keeps is skipped through the
// blob's tap-union table, which is where structured masks still save time.
//
// Activations: as in the kept-only kernel, a haloed slab of the NHWC tensor is loaded by TMA
// through the 5-D view (8 channels, W, H, C/8, N) and lands as [octet][row][column][8], so that a
// tap shift is a change of the operand's start address; out-of-image positions are zero-filled.
// A CTA works on items = (MT position tiles of 128 padded positions) x (NG filter groups): every
// weight tile fetched is used by MT position tiles and every slab by NG groups.  Warp 0 produces
// (TMA slabs, bulk-copied weight tiles, ring of stages of one chunk each), one warp per accumulator
// issues its MMAs (so the summation order is fixed; an item of a single block splits its taps over
// two accumulators that the epilogue adds), eight warps run the epilogue (bias, residual, ReLU, one rounding; with a stride only the
// strided positions are stored) - overlapped with the next item when two accumulator sets fit in
// TMEM.  Every wait is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kEpiWarps = 8;
constexpr int kParts = kEpiWarps / 4;            // epilogue warps per TMEM lane quarter
constexpr int kMmaWarps = 4;                     // one per accumulator (position tile, filter group)
constexpr int kFirstEpiWarp = 1 + kMmaWarps;
constexpr int kThreads = (kFirstEpiWarp + kEpiWarps) * 32;
constexpr int kMaxStages = 6;
constexpr int kMaxTapsDn = 16;
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kDescHi = (128u >> 4) | (1u << 14);   // SBO = 128 bytes, descriptor version bit

struct ConvDnParams {
    int N, H, W, C, K, R, S, pad, stride, P, Q, Po, Qo;      // P, Q: positions at stride 1
    int Wp, TR, tiles_per_img, n_tiles, slab_rows;
    int CPS;                                                  // 16-channel chunks per stage (1 or 2)
    int RS, nCh, GI, MT, NG, TS, n_gsets, n_items, St, nacc, dcols;   // TS: accumulators per output block (taps split)
    int relu, y_bf16;
    uint32_t plane_bytes, act_stride, w_bytes, stage_bytes, off_tapu, off_bias, off_bar, smem_bytes, tmem_cols;
};

struct ConvDnBars {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t shift[kMaxTapsDn];      // operand start offset of every tap, in 16-byte units
};

__device__ __forceinline__ uint64_t desc64(uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; }
// barrier among all warps but the producer
__device__ __forceinline__ void consumers_sync() { asm volatile("bar.sync 3, %0;" ::"n"(kThreads - 32) : "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
conv_bp_dn_kernel(const __grid_constant__ CUtensorMap tmap_x, const ConvDnParams p, const uint8_t *__restrict__ x_bytes,
                  const uint8_t *__restrict__ blob, const float *__restrict__ bias,
                  const void *__restrict__ res, void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint32_t *tapu_s = reinterpret_cast<uint32_t *>(smem + p.off_tapu);     // [K / GI][nCh]
    float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);           // [K]
    ConvDnBars *bars = reinterpret_cast<ConvDnBars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);

    if (tid == 0) {
        const int nmma = p.MT * p.NG * p.TS;
        for (int s = 0; s < p.St; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], nmma); }
        for (int a = 0; a < 2; ++a) { mbar_init(&bars->acc_full[a], nmma); mbar_init(&bars->acc_empty[a], kEpiWarps); }
        for (int t = 0; t < p.RS; ++t) bars->shift[t] = (uint32_t)((t / p.S) * p.Wp + t % p.S);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
    }
    if (warp == 1) tmem_alloc(&bars->tmem_base, p.tmem_cols);          // warp 1 also frees it
    pdl_trigger();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_wait();                        // nothing above touches global memory
    const uint32_t tmem_base = bars->tmem_base;
    // Cold operands: the whole grid asks L2 for the operand image (one slice per CTA) and every CTA for the
    // input rows of its first item, so that DRAM latency is paid once, up front and in parallel, instead
    // of stage by stage inside the pipeline.
    if (warp == kFirstEpiWarp && lane == 0) {
        const uint32_t off_image = hdr[BP_OFF_IMAGE];
        if (off_image) {
            const uint32_t img_bytes = (uint32_t)p.K * p.RS * p.C * 2u;
            const uint32_t slice = round_up((img_bytes + gridDim.x - 1) / gridDim.x, 2048);
            const uint32_t b0 = blockIdx.x * slice;
            for (uint32_t o = b0; o < min(b0 + slice, img_bytes); o += 16384u)
                bulk_prefetch_l2(blob + off_image + o, min(16384u, min(b0 + slice, img_bytes) - o));
        }
        if ((int)blockIdx.x < p.n_items) {
            const int ts = blockIdx.x / p.n_gsets;
            for (int mt = 0; mt < p.MT && ts * p.MT + mt < p.n_tiles; ++mt) {
                const int tile = ts * p.MT + mt, n = tile / p.tiles_per_img, y0 = (tile - n * p.tiles_per_img) * p.TR;
                const int r0 = max(y0 - p.pad, 0), r1 = min(y0 - p.pad + p.slab_rows, p.H);
                const size_t row_b = (size_t)p.W * p.C * 2;
                const uint8_t *src = x_bytes + ((size_t)n * p.H + r0) * row_b;
                for (size_t o = 0; o < (size_t)(r1 - r0) * row_b; o += 16384)
                    bulk_prefetch_l2(src + o, (uint32_t)min((size_t)16384, (size_t)(r1 - r0) * row_b - o));
            }
        }
    }
    // the producer starts at once; the other warps first stage the biases and the tap unions
    if (warp != 0) {
        for (int i = tid - 32; i < p.K; i += kThreads - 32) bias_s[i] = bias ? bias[i] : 0.f;
        const uint32_t off_tapu = hdr[BP_OFF_TAPU];
        const uint32_t *tapu = reinterpret_cast<const uint32_t *>(blob + off_tapu);
        for (int i = tid - 32; i < (p.K / p.GI) * p.nCh; i += kThreads - 32) tapu_s[i] = off_tapu ? tapu[i] : 0xFFFFFFFFu;
        consumers_sync();
    }

    if (warp == 0) {
        // ---- producer ------------------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t off_image = hdr[BP_OFF_IMAGE];
            const uint8_t *image = blob + off_image;
            uint32_t s = 0, lap = 0;                                         // ring position and completed laps
            bool ok = true;
            // the blob must carry the operand image this kernel was planned for; if not, nothing is
            // requested and the other roles leave their first wait through the abort flag
            if (off_image == 0u || hdr[BP_GI] != (uint32_t)p.GI) {
                bars->abort_flag = 2;
                if (atomicCAS(ws, 0u, 6u /* NPAS_ERR_BLOB */) == 0u) ws[1] = 0x6001;
                ok = false;
            }
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const int ts = item / p.n_gsets, gs = item - ts * p.n_gsets;
                const int mtv = min(p.MT, p.n_tiles - ts * p.MT);            // position tiles that exist
                const uint32_t wst = (uint32_t)p.CPS * p.w_bytes;            // a stage's weights of one group
                for (int sc = 0; sc < p.nCh / p.CPS; ++sc) {
                    if (lap >= 1 && !mbar_wait(&bars->empty[s], (lap & 1u) ^ 1u, abort_flag, ws, 0x6100)) { ok = false; break; }
                    uint8_t *st = smem + (size_t)s * p.stage_bytes;
                    mbar_arrive_expect_tx(&bars->full[s], (uint32_t)mtv * 2u * p.CPS * p.plane_bytes + (uint32_t)p.NG * wst);
                    for (int mt = 0; mt < mtv; ++mt) {
                        const int tile = ts * p.MT + mt, n = tile / p.tiles_per_img, y0 = (tile - n * p.tiles_per_img) * p.TR;
                        tma_load_5d(st + (size_t)mt * p.act_stride, &tmap_x, &bars->full[s], 0, -p.pad, y0 - p.pad, sc * 2 * p.CPS, n);
                    }
                    for (int g = 0; g < p.NG; ++g) {
                        const uint8_t *src = image + ((size_t)(gs * p.NG + g) * p.nCh + sc * p.CPS) * p.w_bytes;
                        uint8_t *dst = st + (size_t)p.MT * p.act_stride + (size_t)g * wst;
                        for (uint32_t o = 0; o < wst; o += 16384u)
                            bulk_load_1d(dst + o, src + o, min(16384u, wst - o), &bars->full[s]);
                    }
                    if (++s == (uint32_t)p.St) { s = 0; ++lap; }
                }
            }
        }
    } else if (warp < kFirstEpiWarp) {
        // ---- MMA issue: warp w owns the accumulator of (position tile w / NG, filter group w % NG) ------
        // (one elected thread runs the whole role; the warp index through a shuffle, so that the compiler knows the
        // operands warp-uniform: about half the issue cost per MMA)
        const int w = __shfl_sync(0xFFFFFFFFu, warp, 0) - 1;
        if (w < p.MT * p.NG * p.TS && elect_one()) {
            const int blk = w / p.TS, half = w - blk * p.TS, mt = blk / p.NG, g = blk - mt * p.NG;
            // with two accumulators per output block this warp takes one half of the taps
            const int t0 = half ? (p.RS + 1) / 2 : 0, t1 = (p.TS == 2 && !half) ? (p.RS + 1) / 2 : p.RS;
            const int sx0 = t0 % p.S;
            const uint32_t idesc = idesc_bf16_f32(128, p.GI);
            const uint32_t base16 = smem_u32(smem) >> 4, stage16 = p.stage_bytes >> 4;
            const uint32_t a_off = (uint32_t)mt * (p.act_stride >> 4), a_hi = (p.plane_bytes >> 4) << 16;
            const uint32_t b_off = (uint32_t)p.MT * (p.act_stride >> 4) + (uint32_t)g * (uint32_t)p.CPS * (p.w_bytes >> 4), b_hi = (uint32_t)p.GI << 16;
            const uint32_t b_step = 2u * p.GI;
            uint32_t s = 0, ph = 0, it = 0;                 // ring position and its barrier parity
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++it) {
                const int ts = item / p.n_gsets, gs = item - ts * p.n_gsets;
                const bool live = ts * p.MT + mt < p.n_tiles;              // the last item may lack its second tile
                const uint32_t acc = p.nacc == 2 ? (it & 1u) : 0u, lap_acc = p.nacc == 2 ? (it >> 1) : it;
                if (lap_acc >= 1 && !mbar_wait(&bars->acc_empty[acc], (lap_acc & 1u) ^ 1u, abort_flag, ws, 0x6200)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * p.dcols + (uint32_t)w * p.GI;
                const uint32_t *tu = tapu_s + (gs * p.NG + g) * p.nCh;
                for (int sc = 0; sc < p.nCh / p.CPS; ++sc) {
                    if (!mbar_wait(&bars->full[s], ph, abort_flag, ws, 0x6300)) { ok = false; break; }
                    tc_fence_after_sync();
                    {
                      const uint32_t st16 = base16 + s * stage16;
                      for (int cc = 0; cc < p.CPS; ++cc) {
                        const int ch = sc * p.CPS + cc;
                        // a tap that no block of this (group, chunk) keeps multiplies zeros: skipped, except
                        // the very first MMA, which initialises the accumulator
                        const uint32_t mask = (tu[ch] | (ch == 0 ? 1u << t0 : 0u)) >> t0;
                        const uint32_t a0 = ((st16 + a_off) | a_hi) + (uint32_t)cc * 2u * (p.plane_bytes >> 4);
                        uint32_t b_lo = ((st16 + b_off) | b_hi) + (uint32_t)cc * (p.w_bytes >> 4) + (uint32_t)t0 * b_step;
                        if (live) {
                            // a plain loop (unrolled, the skipped slots cost as much as MMAs); the tap's
                            // operand offset r * Wp + s is carried along instead of being looked up
                            uint32_t a_lo = a0 + bars->shift[t0], m = mask;
                            int sx = sx0;
                            for (int t = t0; t < t1; ++t, b_lo += b_step, m >>= 1) {
                                if (m & 1u) mma_bf16_ss(d_tmem, desc64(a_lo), desc64(b_lo), idesc, (ch | (t - t0)) ? 1u : 0u);
                                ++a_lo;
                                if (++sx == p.S) { sx = 0; a_lo += (uint32_t)(p.Wp - p.S); }
                            }
                        }
                      }
                      mma_commit(&bars->empty[s]);
                      if (sc == p.nCh / p.CPS - 1) mma_commit(&bars->acc_full[acc]);
                    }
                    if (++s == (uint32_t)p.St) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else {
        // ---- epilogue: warp -> TMEM lane quarter (warp % 4) and every (kEpiWarps / 4)-th 16-column chunk ----------------
        const int quarter = warp & 3, part = (warp - kFirstEpiWarp) >> 2, m = quarter * 32 + lane;
        const int oy = m / p.Wp, ox = m - oy * p.Wp;
        const int cpg = p.GI / 16;                          // chunks per (position tile, group)
        const int sh = p.stride - 1;                        // stride 1 or 2: divide by shifting
        uint32_t it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++it) {
            const int ts = item / p.n_gsets, gs = item - ts * p.n_gsets;
            const int mtv = min(p.MT, p.n_tiles - ts * p.MT);
            const uint32_t acc = p.nacc == 2 ? (it & 1u) : 0u, lap_acc = p.nacc == 2 ? (it >> 1) : it;
            const int nch = mtv * p.NG * cpg;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * p.dcols;

            // where this thread's position of each tile goes (MT <= 2); with a stride the tile is computed
            // at every position and only the strided ones are stored (stride is 1 or 2)
            bool val[2];
            size_t obase[2];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const int tile = min(ts * p.MT + mt, p.n_tiles - 1), n = tile / p.tiles_per_img;
                const int yy = (tile - n * p.tiles_per_img) * p.TR + oy;
                val[mt] = mt < mtv && oy < p.TR && yy < p.P && ox < p.Q && ((yy | ox) & sh) == 0;
                obase[mt] = (((size_t)n * p.Po + (yy >> sh)) * p.Qo + (ox >> sh)) * p.K;
            }
            auto finish = [&](const uint32_t (&r)[16], int j) {
                const int per_mt = p.NG * cpg, mt = j >= per_mt ? 1 : 0, rem = j - mt * per_mt;
                const int g = rem >= cpg ? 1 : 0, c0 = (rem - g * cpg) * 16;
                // taps split over two accumulators (single-block items only): the other half's partial sums
                uint32_t r2[16];
                if (p.TS == 2) {
                    __syncwarp();
                    tmem_ld_x16(t_addr + p.GI + j * 16, r2);
                    tmem_ld_wait();
                }
                if (!(mt ? val[1] : val[0])) return;
                const int k0 = (gs * p.NG + g) * p.GI + c0;
                const size_t o0 = (mt ? obase[1] : obase[0]) + k0;
                float v[16];
                const float4 *b4 = reinterpret_cast<const float4 *>(bias_s + k0);
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float4 u = b4[h];
                    v[4 * h] = __uint_as_float(r[4 * h]) + u.x; v[4 * h + 1] = __uint_as_float(r[4 * h + 1]) + u.y;
                    v[4 * h + 2] = __uint_as_float(r[4 * h + 2]) + u.z; v[4 * h + 3] = __uint_as_float(r[4 * h + 3]) + u.w;
                }
                if (p.TS == 2) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] += __uint_as_float(r2[i]);
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

            if (!mbar_wait(&bars->acc_full[acc], lap_acc & 1u, abort_flag, ws, 0x6400)) { ok = false; break; }
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
            if (lane == 0) mbar_arrive(&bars->acc_empty[acc]);
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

bool plan(const npas_conv_desc &d, const npas_bp_desc &bp, ConvDnParams &p, int sms)
{
    if (d.x_dtype != NPAS_BF16 || bp.w_packed != NPAS_BF16) return false;
    if ((d.stride != 1 && d.stride != 2) || d.pad < 0 || d.C % 16 || d.K % 16) return false;
    p.RS = d.R * d.S;
    if (p.RS > kMaxTapsDn) return false;
    const BpLayout L = bp_layout(bp, 0);
    p.GI = (int)L.GI;
    if (p.GI < 16) return false;
    p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C; p.K = d.K; p.R = d.R; p.S = d.S; p.pad = d.pad; p.stride = d.stride;
    p.P = d.H + 2 * d.pad - d.R + 1; p.Q = d.W + 2 * d.pad - d.S + 1;
    if (p.P < 1 || p.Q < 1) return false;
    p.Po = (p.P - 1) / d.stride + 1; p.Qo = (p.Q - 1) / d.stride + 1;
    p.Wp = d.W + 2 * d.pad;
    if (p.Wp > 128) return false;
    p.TR = min(p.P, 128 / p.Wp);
    p.tiles_per_img = (p.P + p.TR - 1) / p.TR;
    p.n_tiles = d.N * p.tiles_per_img;
    p.slab_rows = p.TR + d.R - 1;
    if (p.slab_rows > 256) return false;
    p.nCh = d.C / 16;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    p.plane_bytes = (uint32_t)p.slab_rows * p.Wp * 16u;
    // a shifted operand reads up to 128 rows past its start: room behind the second plane
    const uint32_t reach = (128u + (uint32_t)(d.R - 1) * p.Wp + d.S) * 16u;
    const uint32_t slack = reach > p.plane_bytes ? reach - p.plane_bytes : 0u;
    p.w_bytes = (uint32_t)p.RS * 2u * p.GI * 16u;
    const int nGI = d.K / p.GI;
    const uint32_t fixed = round_up((uint32_t)nGI * p.nCh * 4u, 128) + round_up((uint32_t)d.K * 4u, 128) +
                           (uint32_t)sizeof(ConvDnBars) + 1024u + 256u;
    // position tiles x filter groups per item: prefer sharing the weight tiles (MT), then the slab (NG),
    // as long as there are items for every SM
    const int cand[4][2] = {{2, 1}, {1, 2}, {2, 2}, {1, 1}};   // the first two leave room for two accumulator sets
    bool found = false;
    for (int c = 0; c < 4 && !found; ++c) {
        const int MT = cand[c][0], NG = cand[c][1];
        if (NG > nGI || nGI % NG || MT * NG * p.GI > 512) continue;
        if (MT > 1 && p.n_tiles < 2) continue;
        const long long items = (long long)((p.n_tiles + MT - 1) / MT) * (nGI / NG);
        if (items > 0x7FFFFFFF) return false;
        if (c < 3 && items * 10 < (long long)sms * 9) continue;          // keep every SM busy
        // two chunks per stage halve the waits and commits per MMA; taken when two such stages fit
        p.CPS = p.nCh % 2 == 0 ? 2 : 1;
        uint32_t stage = 0;
        for (; p.CPS >= 1; --p.CPS) {
            p.act_stride = round_up(2u * p.CPS * p.plane_bytes + slack, 128);
            stage = round_up((uint32_t)MT * p.act_stride + (uint32_t)NG * p.CPS * p.w_bytes, 1024);
            if (fixed + 2 * stage <= kSmemLimit && 2u * p.CPS * p.plane_bytes < (1u << 18)) break;
        }
        if (p.CPS < 1) continue;
        p.MT = MT; p.NG = NG; p.n_gsets = nGI / NG; p.n_items = (int)items;
        // a single-block item would leave one warp issuing every MMA: split its taps over two accumulators
        p.TS = (MT * NG == 1 && p.RS >= 2 && 2 * p.GI <= 256) ? 2 : 1;
        p.stage_bytes = stage;
        p.St = (int)((kSmemLimit - fixed) / stage);
        if (p.St > kMaxStages) p.St = kMaxStages;
        found = true;
    }
    if (!found) return false;
    if ((uint32_t)p.St * p.stage_bytes >= (1u << 18)) return false;        // descriptor addresses are 14 bits of 16 bytes
    p.dcols = p.MT * p.NG * p.TS * p.GI;
    p.nacc = 2 * p.dcols <= 512 ? 2 : 1;
    p.off_tapu = (uint32_t)p.St * p.stage_bytes;
    p.off_bias = p.off_tapu + round_up((uint32_t)nGI * p.nCh * 4u, 128);
    p.off_bar = p.off_bias + round_up((uint32_t)d.K * 4u, 128);
    p.smem_bytes = p.off_bar + sizeof(ConvDnBars) + 1024;
    if (p.smem_bytes > kSmemLimit) return false;
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < p.nacc * p.dcols) p.tmem_cols *= 2;
    return true;
}

}  // namespace

bool conv_dn_supported(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    ConvDnParams p;
    return plan(d, bp, p, sm_count());
}

npas_status conv_dn_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st)
{
    ConvDnParams p;
    const int sms = sm_count();
    if (!plan(d, bp, p, sms)) return NPAS_ERR_UNSUPPORTED;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return NPAS_ERR_CUDA;
    // X[N][H][W][C] bf16 seen as (8 channels, W, H, C/8, N): a box lands in shared memory as
    // [octet][row][column][8 channels]
    CUtensorMap tmap;
    const cuuint64_t dims[5] = {8, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)(d.C / 8), (cuuint64_t)d.N};
    const cuuint64_t strides[4] = {(cuuint64_t)d.C * 2, (cuuint64_t)d.W * d.C * 2, 16, (cuuint64_t)d.H * d.W * d.C * 2};
    const cuuint32_t box[5] = {8, (cuuint32_t)p.Wp, (cuuint32_t)p.slab_rows, (cuuint32_t)(2 * p.CPS), 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return NPAS_ERR_CUDA;
    if (allow_dynamic_smem(reinterpret_cast<const void *>(conv_bp_dn_kernel), (int)kSmemLimit) != NPAS_OK) return NPAS_ERR_CUDA;
    const int grid = p.n_items < sms ? p.n_items : sms;
    const cudaError_t e = launch_pdl(conv_bp_dn_kernel, dim3(grid), dim3(kThreads), p.smem_bytes, st, tmap, p,
                                     static_cast<const uint8_t *>(x), static_cast<const uint8_t *>(blob), bias, res, y, ws);
    count_launch();
    return e == cudaSuccess ? launch_status() : NPAS_ERR_CUDA;
}

}  // namespace npas
