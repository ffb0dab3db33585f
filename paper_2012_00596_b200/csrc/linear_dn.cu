// Block-based pruned GEMM on the sm_100a tensor cores, both operands by TMA.
//
// Y[M x O] = act(X[M x I] * Wm[O x I]^T + bias (+ residual)) with Wm the masked weight matrix that
// the packer stores next to the compact form (section `dense` of the blob).  At the shapes this
// library meets, the layer is bound by moving X and Y, not by the multiply, and the tensor core
// reads operands in units of eight K elements, so skipping pruned columns inside a 64-wide block
// costs more shared-memory traffic (a gather of X) than the zeros cost tensor time.  This kernel
// therefore multiplies the zero-expanded matrix at the tensor pipe's full rate and spends its effort
// on streaming: a persistent CTA per SM walks output tiles of 128 rows x BN columns; warp 0 feeds
// a ring of stages (X tile 128 x 64 and W tile BN x 64, both 128-byte swizzled) with TMA, warp 1
// issues MMAs of M = 128, N = BN, K = 16 into one of two TMEM accumulators, and sixteen epilogue
// warps drain the other accumulator (fp32 bias, residual, ReLU, one rounding, 32 bytes per thread
// and chunk, the next chunk already on its way out of TMEM) while the next tile is being multiplied.
// With bf16 output and BN a multiple of 64 the epilogue goes through shared memory: the residual
// arrives by TMA in slabs of 128 rows x 64 columns (a ring of slots, requested a tile ahead by a
// warp of its own, so that enough bytes are in flight to hide DRAM latency), each thread finishes
// its 32 bytes in place in the slot (128-byte swizzled, conflict free) and its warp arrives on the
// slot's "done" barrier; a warp of its own waits for that barrier, sends the slot off with a TMA store
// and frees the slot before it once that store has read it.  No thread waits on a global load, the
// epilogue warps wait neither for the stores nor for each other, and the memory system sees whole
// lines instead of 32-byte pieces of 32 different lines per instruction.  Every wait is bounded.
#include <cstdlib>

#include "common.cuh"
#include "tc_common.cuh"

namespace npas {

using namespace tc;

namespace {

constexpr int kEpiWarps = 16;
constexpr int kFirstEpiWarp = 2;
constexpr int kResWarp = kFirstEpiWarp + kEpiWarps;         // requests the residual slabs
constexpr int kStoreWarp = kResWarp + 1;                    // stores the finished slabs
constexpr int kThreads = (kStoreWarp + 1) * 32;
constexpr int kRows = 128;
constexpr int kMaxStages = 6;
constexpr int kMaxSlots = 6;
constexpr uint32_t kSlotBytes = kRows * 128;              // 128 rows x 64 bf16, 128-byte swizzled
constexpr uint32_t kSmemLimit = 232448;
constexpr uint32_t kXBytes = kRows * 128;                 // 128 rows of 64 bf16
// shared-memory descriptor, high word: SBO = 1024 bytes (eight 128-byte rows), version bit, 128-byte swizzle
constexpr uint32_t kDescHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
constexpr uint32_t kDescLboOne = 1u << 16;                // LBO is not used by swizzled K-major layouts

struct LinDnParams {
    int M, I, O, BN, nK, nMT, nNT, n_tiles, S;
    int relu, y_bf16;
    int NS;                                               // epilogue slots (0: epilogue straight from registers)
    uint32_t stage_bytes, off_slots, off_bias, off_bar, smem_bytes, tmem_cols;
};

struct LinDnBars {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t res_full[kMaxSlots], res_empty[kMaxSlots];   // residual slab landed / slot free again
    uint64_t slot_done[kMaxSlots];                        // every epilogue warp has finished its part of the slab
    uint32_t tmem_base;
    uint32_t abort_flag;
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    return cvt_bf16x2(lo, hi);
}
__device__ __forceinline__ uint64_t desc64(uint32_t lo) { return ((uint64_t)kDescHiSw128 << 32) | lo; }

// barrier among the epilogue warps
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 2, %0;" ::"n"(kEpiWarps * 32) : "memory"); }
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *m, const void *src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
linear_bb_dn_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                    const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_r,
                    const LinDnParams p, const float *__restrict__ bias, const void *__restrict__ res,
                    void *__restrict__ y, uint32_t *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);      // [O]
    LinDnBars *bars = reinterpret_cast<LinDnBars *>(smem + p.off_bar);
    volatile uint32_t *abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < p.S; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&bars->acc_full[a], 1); mbar_init(&bars->acc_empty[a], kEpiWarps); }
        for (int s = 0; s < p.NS; ++s) {
            mbar_init(&bars->res_full[s], 1); mbar_init(&bars->res_empty[s], 1); mbar_init(&bars->slot_done[s], kEpiWarps);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
        if (p.NS) { prefetch_tensormap(&tmap_y); if (res) prefetch_tensormap(&tmap_r); }
    }
    if (warp == 1) tmem_alloc(&bars->tmem_base, p.tmem_cols);
    pdl_trigger();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_wait();                        // nothing above touches global memory
    // the biases: staged by the epilogue warps, which meet again before the first use
    if (warp >= kFirstEpiWarp && warp < kResWarp) {
        for (int i = tid - kFirstEpiWarp * 32; i < p.O; i += kEpiWarps * 32) bias_s[i] = bias ? bias[i] : 0.f;
        epi_sync();
    }
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ---- TMA producer: tiles in the order (row tile, column tile), K steps inside ---------------
        if (lane == 0) {
            // (ring slot and lap are carried along: a division per stage costs the issuing thread more
            // than the stage's copies)
            uint32_t s = 0, lap = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
                const int mt = tile / p.nNT, nt = tile - mt * p.nNT;
                for (int k = 0; k < p.nK; ++k) {
                    if (lap >= 1 && !mbar_wait(&bars->empty[s], (lap & 1u) ^ 1u, abort_flag, ws, 0x5100)) { ok = false; break; }
                    uint8_t *st = smem + (size_t)s * p.stage_bytes;
                    mbar_arrive_expect_tx(&bars->full[s], p.stage_bytes);
                    tma_load_2d(st, &tmap_x, &bars->full[s], k * 64, mt * kRows);
                    tma_load_2d(st + kXBytes, &tmap_w, &bars->full[s], k * 64, nt * p.BN);
                    if (++s == (uint32_t)p.S) { s = 0; ++lap; }
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue: one thread; its own instructions are on the critical path (four MMAs of a stage
        // execute in about 600 cycles), so the ring position is carried along and nothing else is computed
        if (elect_one()) {
            const uint32_t idesc = idesc_bf16_f32(128, p.BN);
            const uint32_t base16 = (smem_u32(smem) >> 4) | kDescLboOne, stage16 = p.stage_bytes >> 4;
            uint32_t s = 0, ph = 0, a_lo = base16, it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++it) {
                const uint32_t acc = it & 1u, lap_acc = it >> 1;
                if (lap_acc >= 1 && !mbar_wait(&bars->acc_empty[acc], (lap_acc & 1u) ^ 1u, abort_flag, ws, 0x5200)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * p.BN;
                for (int k = 0; k < p.nK; ++k) {
                    if (!mbar_wait(&bars->full[s], ph, abort_flag, ws, 0x5300)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t b_lo = a_lo + (kXBytes >> 4);
#pragma unroll
                    for (uint32_t j = 0; j < 4; ++j)          // 16 columns = 32 bytes inside the swizzled row
                        mma_bf16_ss(d_tmem, desc64(a_lo + 2 * j), desc64(b_lo + 2 * j), idesc, (k > 0 || j > 0) ? 1u : 0u);
                    mma_commit(&bars->empty[s]);
                    if (k == p.nK - 1) mma_commit(&bars->acc_full[acc]);
                    a_lo += stage16;
                    if (++s == (uint32_t)p.S) { s = 0; ph ^= 1u; a_lo = base16; }
                }
            }
        }
    } else if (warp == kResWarp) {
        // ---- residual producer: slab n of this CTA's sequence (tile, 64-column slab) goes to slot n % NS as
        // soon as the store that last used the slot has read it ----------------------------------------------
        if (lane == 0 && p.NS && res) {
            uint32_t n = 0;
            bool ok = true;
            const int nsl = p.BN / 64;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
                const int mt = tile / p.nNT, nt = tile - mt * p.nNT;
                for (int sl = 0; sl < nsl; ++sl, ++n) {
                    const uint32_t slot = n % (uint32_t)p.NS, lap = n / (uint32_t)p.NS;
                    if (lap >= 1 && !mbar_wait(&bars->res_empty[slot], (lap & 1u) ^ 1u, abort_flag, ws, 0x5500)) { ok = false; break; }
                    mbar_arrive_expect_tx(&bars->res_full[slot], kSlotBytes);
                    tma_load_2d(smem + p.off_slots + (size_t)slot * kSlotBytes, &tmap_r, &bars->res_full[slot], nt * p.BN + sl * 64, mt * kRows);
                }
            }
        }
    } else if (warp == kStoreWarp) {
        // ---- store role: slab n leaves by TMA as soon as every epilogue warp has finished its part; when the
        // store before it has read its slot, that slot is free again (for the next residual slab, or, without
        // a residual, for the epilogue itself).  The epilogue warps never wait for a store or for each other.
        if (lane == 0 && p.NS) {
            const int nsl = p.BN / 64;
            uint32_t slot = 0, ph = 0, prev = 0;
            bool ok = true, first = true;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
                const int mt = tile / p.nNT, nt = tile - mt * p.nNT;
                for (int sl = 0; sl < nsl; ++sl) {
                    if (!mbar_wait(&bars->slot_done[slot], ph, abort_flag, ws, 0x5600)) { ok = false; break; }
                    tma_store_2d(&tmap_y, smem + p.off_slots + (size_t)slot * kSlotBytes, nt * p.BN + sl * 64, mt * kRows);
                    bulk_commit();
                    if (!first) { bulk_wait_read<1>(); mbar_arrive(&bars->res_empty[prev]); }
                    first = false; prev = slot;
                    if (++slot == (uint32_t)p.NS) { slot = 0; ph ^= 1u; }
                }
            }
            bulk_wait_all();                            // the slots stay valid until the last store has read them
        }
    } else if (p.NS) {
        // ---- epilogue through shared memory: warp -> TMEM lane quarter (warp % 4) and the 16 columns
        // number (warp - first) / 4 of every 64-column slab ---------------------------------------------------
        const int quarter = warp & 3, part = (warp - kFirstEpiWarp) >> 2, m = quarter * 32 + lane;
        const int nsl = p.BN / 64;
        // this thread's two 16-byte pieces of its row of a slot (pieces XOR-ed with the row number)
        const uint32_t off0 = (uint32_t)m * 128u + (uint32_t)(((2 * part) ^ (m & 7)) * 16);
        const uint32_t off1 = (uint32_t)m * 128u + (uint32_t)(((2 * part + 1) ^ (m & 7)) * 16);
        uint32_t it = 0, n = 0, slot = 0, slot_ph = 0;      // slab count; its slot and the slot's lap parity
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++it) {
            const int mt = tile / p.nNT, nt = tile - mt * p.nNT;
            const uint32_t acc = it & 1u;
            const float *bs = bias_s + nt * p.BN + part * 16;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * p.BN + (uint32_t)part * 16u;
            if (!mbar_wait(&bars->acc_full[acc], (it >> 1) & 1u, abort_flag, ws, 0x5400)) { ok = false; break; }
            tc_fence_after_sync();
            uint32_t r[16];
            tmem_ld_x16(t_addr, r);
            for (int sl = 0; sl < nsl; ++sl, ++n) {
                uint8_t *sp = smem + p.off_slots + (size_t)slot * kSlotBytes;
                float v[16];
                tmem_ld_wait();
                {
                    const float4 *b4 = reinterpret_cast<const float4 *>(bs + sl * 64);
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const float4 u = b4[h];
                        v[4 * h] = __uint_as_float(r[4 * h]) + u.x; v[4 * h + 1] = __uint_as_float(r[4 * h + 1]) + u.y;
                        v[4 * h + 2] = __uint_as_float(r[4 * h + 2]) + u.z; v[4 * h + 3] = __uint_as_float(r[4 * h + 3]) + u.w;
                    }
                }
                if (sl + 1 < nsl) tmem_ld_x16(t_addr + (uint32_t)(sl + 1) * 64u, r);     // next slab's chunk on its way
                // the slot: with a residual it is free when the residual slab has landed in it; without, when the
                // store that last used it has read it (from its second use on)
                if (res) {
                    if (!mbar_wait(&bars->res_full[slot], slot_ph, abort_flag, ws, 0x5410)) { ok = false; break; }
                } else if (n >= (uint32_t)p.NS) {
                    if (!mbar_wait(&bars->res_empty[slot], slot_ph ^ 1u, abort_flag, ws, 0x5420)) { ok = false; break; }
                }
                if (res) {
                    const uint4 u0 = *reinterpret_cast<const uint4 *>(sp + off0), u1 = *reinterpret_cast<const uint4 *>(sp + off1);
                    const uint32_t wv[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        v[2 * i] += __uint_as_float(wv[i] << 16);
                        v[2 * i + 1] += __uint_as_float(wv[i] & 0xFFFF0000u);
                    }
                }
                // one rounding, then ReLU on the packed pairs (max with +0 is exact on the rounded values)
                uint32_t o[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) o[i] = pack2(v[2 * i], v[2 * i + 1]);
                if (p.relu) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) o[i] = relu_bf16x2(o[i]);
                }
                *reinterpret_cast<uint4 *>(sp + off0) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4 *>(sp + off1) = make_uint4(o[4], o[5], o[6], o[7]);
                fence_proxy_async_smem();               // the TMA store reads what this thread wrote
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->slot_done[slot]);
                if (++slot == (uint32_t)p.NS) { slot = 0; slot_ph ^= 1u; }
            }
            if (!ok) break;
            // this warp has read its part of the accumulator: the MMA warp may overwrite it
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc_empty[acc]);
        }
    } else {
        // ---- epilogue: warp -> TMEM lane quarter (warp % 4) and every fourth 16-column chunk ----------
        const int quarter = warp & 3, part = (warp - kFirstEpiWarp) >> 2, m = quarter * 32 + lane;
        const int nch = p.BN / 16;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++it) {
            const int mt = tile / p.nNT, nt = tile - mt * p.nNT;
            const uint32_t acc = it & 1u;
            const int row = mt * kRows + m;
            const bool valid = row < p.M;
            const size_t o0 = (size_t)row * p.O + (size_t)nt * p.BN;
            const float *bs = bias_s + nt * p.BN;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * p.BN;

            // one chunk: + bias (+ residual), ReLU, one rounding, 32 (bf16) or 64 (fp32) bytes per thread
            auto finish = [&](const uint32_t (&r)[16], int c0) {
                if (!valid) return;
                float v[16];
                const float4 *b4 = reinterpret_cast<const float4 *>(bs + c0);
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float4 u = b4[h];
                    v[4 * h] = __uint_as_float(r[4 * h]) + u.x; v[4 * h + 1] = __uint_as_float(r[4 * h + 1]) + u.y;
                    v[4 * h + 2] = __uint_as_float(r[4 * h + 2]) + u.z; v[4 * h + 3] = __uint_as_float(r[4 * h + 3]) + u.w;
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
                    yp[0] = make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
                    yp[1] = make_uint4(pack2(v[8], v[9]), pack2(v[10], v[11]), pack2(v[12], v[13]), pack2(v[14], v[15]));
                } else {
                    float4 *yp = reinterpret_cast<float4 *>(static_cast<float *>(y) + o0 + c0);
#pragma unroll
                    for (int h = 0; h < 4; ++h) yp[h] = make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]);
                }
            };

            if (!mbar_wait(&bars->acc_full[acc], (it >> 1) & 1u, abort_flag, ws, 0x5400)) { ok = false; break; }
            tc_fence_after_sync();
            // two register sets: the next chunk is on its way out of TMEM while this one is finished
            uint32_t ra[16], rb[16];
            int j = part;
            if (j < nch) tmem_ld_x16(t_addr + j * 16, ra);
            while (j < nch) {
                tmem_ld_wait();
                if (j + 4 < nch) tmem_ld_x16(t_addr + (j + 4) * 16, rb);
                finish(ra, j * 16);
                j += 4;
                if (j >= nch) break;
                tmem_ld_wait();
                if (j + 4 < nch) tmem_ld_x16(t_addr + (j + 4) * 16, ra);
                finish(rb, j * 16);
                j += 4;
            }
            // this warp has read its part of the accumulator: the MMA warp may overwrite it
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

bool plan(const npas_linear_desc &d, const npas_bb_desc &bb, LinDnParams &p)
{
    if (d.x_dtype != NPAS_BF16 || bb.w_packed != NPAS_BF16) return false;
    if (d.I % 64 || d.O % 16 || d.O > 16384) return false;
    p.M = d.M; p.I = d.I; p.O = d.O;
    p.nK = d.I / 64;
    p.nMT = (d.M + kRows - 1) / kRows;
    p.relu = d.relu; p.y_bf16 = d.y_dtype == NPAS_BF16;
    const uint32_t fixed = (uint32_t)d.O * 4 + 128 + (uint32_t)sizeof(LinDnBars) + 1024 + 256;
    // Column tile BN: the widest divisor of O that leaves room for enough stages (three once the K loop has
    // three or more steps), else the widest with two (measured: narrower tiles never won, the kernel is
    // bound by what the SMs take in from L2, and wide tiles take in the least per MAC).  Epilogue slots
    // (bf16 output, BN % 64 == 0, and the output side at least as large as the input side): three when
    // only stores pass through them, six when the residual is prefetched into them.
    // (the call descriptor's `variant` restricts the choice to one width)
    const int want = p.nK >= 3 ? 3 : 2;
    const int want_bn = d.variant;
    p.BN = 0;
    for (int pass = 0; pass < 2 && !p.BN; ++pass)
        for (int bn = 256; bn >= 16; bn /= 2) {
            if (d.O % bn || (want_bn && bn != want_bn)) continue;
            const int ns = (p.y_bf16 && bn % 64 == 0 && (d.has_residual || d.O >= d.I)) ? (d.has_residual ? kMaxSlots : 3) : 0;
            const uint32_t stage = round_up(kXBytes + (uint32_t)bn * 128u, 1024);   // multiples of 1024: swizzled tiles stay aligned
            const uint32_t need = fixed + (uint32_t)ns * kSlotBytes;
            if (need + 2 * stage > kSmemLimit) continue;
            const int st = (int)((kSmemLimit - need) / stage);
            if (pass == 0 && st < want) continue;
            p.BN = bn; p.NS = ns; p.stage_bytes = stage; p.S = st > kMaxStages ? kMaxStages : st;
            break;
        }
    if (p.BN == 0) return false;
    p.nNT = d.O / p.BN;
    const long long tiles = (long long)p.nMT * p.nNT;
    if (tiles > 0x7FFFFFFF) return false;
    p.n_tiles = (int)tiles;
    p.off_slots = (uint32_t)p.S * p.stage_bytes;
    p.off_bias = p.off_slots + (uint32_t)p.NS * kSlotBytes;
    p.off_bar = round_up(p.off_bias + (uint32_t)d.O * 4, 128);
    p.smem_bytes = p.off_bar + sizeof(LinDnBars) + 1024;
    if (p.smem_bytes > kSmemLimit) return false;
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < 2 * p.BN) p.tmem_cols *= 2;
    return true;
}

bool encode_2d(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint32_t box_outer)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {inner * 2};
    const cuuint32_t box[2] = {64, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool linear_dn_supported(const npas_linear_desc &d, const npas_bb_desc &bb)
{
    LinDnParams p;
    return plan(d, bb, p);
}

npas_status linear_dn_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                             const void *blob, const float *bias, const void *res, void *y, uint32_t *ws,
                             cudaStream_t st)
{
    LinDnParams p;
    if (!plan(d, bb, p)) return NPAS_ERR_UNSUPPORTED;
    const BbLayout L = bb_layout(bb);
    // X[M][I] and the masked weights [O][I]: boxes of 64 columns land as 128-byte rows, 16-byte
    // pieces XOR-ed with the row number; rows past the end read as zeros
    CUtensorMap tmx, tmw;
    if (!encode_2d(&tmx, x, (uint64_t)d.I, (uint64_t)d.M, kRows)) return NPAS_ERR_CUDA;
    if (!encode_2d(&tmw, static_cast<const uint8_t *>(blob) + L.off_dense, (uint64_t)d.I, (uint64_t)d.O, (uint32_t)p.BN))
        return NPAS_ERR_CUDA;
    // Y and the residual [M][O] in slabs of 128 rows x 64 columns (rows past M are clipped / read as zeros)
    CUtensorMap tmy = tmx, tmr = tmx;
    if (p.NS) {
        if (!encode_2d(&tmy, y, (uint64_t)d.O, (uint64_t)d.M, kRows)) return NPAS_ERR_CUDA;
        if (res && !encode_2d(&tmr, res, (uint64_t)d.O, (uint64_t)d.M, kRows)) return NPAS_ERR_CUDA;
    }
    if (allow_dynamic_smem(reinterpret_cast<const void *>(linear_bb_dn_kernel), (int)kSmemLimit) != NPAS_OK) return NPAS_ERR_CUDA;
    const int sms = sm_count();
    const int grid = p.n_tiles < sms ? p.n_tiles : sms;
    const cudaError_t e = launch_pdl(linear_bb_dn_kernel, dim3(grid), dim3(kThreads), p.smem_bytes, st, tmx, tmw, tmy, tmr,
                                     p, bias, res, y, ws);
    count_launch();
    return e == cudaSuccess ? launch_status() : NPAS_ERR_CUDA;
}

}  // namespace npas
