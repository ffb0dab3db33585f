// Packers and mask helpers: dense weights + block masks <-> the blobs described in npas.h.
// These run once per layer (offline with respect to inference), so they are plain, coalesced
// CUDA-core kernels; all index output is integer work and all value output is a bit copy or a
// single round-to-nearest-even conversion.
#include "common.cuh"

namespace npas {

// ------------------------------------------------------------------------------------------------
// Exclusive prefix sum of `count(i)` for i < n into out[0..n] by ONE block (n is a few thousand
// at most: one entry per weight block).  Every thread scans a contiguous chunk.
template <typename F>
__device__ void block_exclusive_scan(uint32_t n, F count, uint32_t *out, uint32_t *smem /*blockDim+1*/)
{
    const uint32_t T = blockDim.x, t = threadIdx.x;
    const uint32_t chunk = (n + T - 1) / T;
    const uint32_t lo = min(n, t * chunk), hi = min(n, lo + chunk);
    uint32_t sum = 0;
    for (uint32_t i = lo; i < hi; ++i) sum += count(i);
    smem[t] = sum;
    __syncthreads();
    if (t == 0) {
        uint32_t run = 0;
        for (uint32_t i = 0; i < T; ++i) { uint32_t v = smem[i]; smem[i] = run; run += v; }
        smem[T] = run;
    }
    __syncthreads();
    uint32_t run = smem[t];
    for (uint32_t i = lo; i < hi; ++i) { out[i] = run; run += count(i); }
    if (t == 0) out[n] = smem[T];
    __syncthreads();
}

// ---- block-punched ---------------------------------------------------------------------------

__global__ void bp_scan_kernel(npas_bp_desc d, const uint64_t *__restrict__ tap_mask, uint8_t *blob,
                               uint32_t blob_bytes)
{
    __shared__ uint32_t sm[1025];
    const uint32_t nFB = d.K / d.Mb, nCB = d.C / d.Nb, nBlk = nFB * nCB;
    const uint64_t live = d.R * d.S == 64 ? ~0ull : ((1ull << (d.R * d.S)) - 1);
    uint32_t *hdr = reinterpret_cast<uint32_t *>(blob);
    uint32_t *blk_off = reinterpret_cast<uint32_t *>(blob + 128);
    block_exclusive_scan(nBlk, [&](uint32_t i) { return (uint32_t)__popcll(tap_mask[i] & live); }, blk_off, sm);
    const uint32_t nPairs = blk_off[nBlk];
    const BpLayout L = bp_layout(d, nPairs);
    if (L.total > blob_bytes) {
        // A blob that does not fit keeps magic 0 and every section offset 0 (only the size that
        // would have been needed is recorded); the later kernels write nothing.
        if (threadIdx.x == 0) hdr[BP_TOTAL] = L.total;
        return;
    }
    if (threadIdx.x == 0) {
        hdr[BP_OFF_IMAGE] = L.off_image; hdr[BP_OFF_TAPU] = L.off_tapu; hdr[BP_GI] = L.GI;
        hdr[BP_OFF_KTOFF] = L.off_ktoff; hdr[BP_OFF_KT] = L.off_kt; hdr[BP_GS] = L.GS; hdr[BP_NKT] = L.nKt;
        hdr[BP_MAGIC] = kMagicBP;
        hdr[BP_VERSION] = kVersion; hdr[BP_DTYPE] = d.w_packed;
        hdr[BP_K] = d.K; hdr[BP_C] = d.C; hdr[BP_R] = d.R; hdr[BP_S] = d.S; hdr[BP_MB] = d.Mb; hdr[BP_NB] = d.Nb;
        hdr[BP_NFB] = nFB; hdr[BP_NCB] = nCB; hdr[BP_NPAIRS] = nPairs;
        hdr[BP_OFF_BLK] = 128; hdr[BP_OFF_PAIRS] = L.off_pairs; hdr[BP_OFF_VALUES] = L.off_values;
        hdr[BP_TOTAL] = L.total; hdr[BP_G] = L.G;
    }
    if (L.off_kt) {
        // tiles per (16-channel chunk, group of GS filter blocks), chunk major
        const uint32_t nCh = d.C / 16, cpb = d.Nb / 16;
        uint32_t *kt_off = reinterpret_cast<uint32_t *>(blob + L.off_ktoff);
        block_exclusive_scan(nCh * L.nGrp, [&](uint32_t i) {
            const uint32_t ch = i / L.nGrp, g = i % L.nGrp, cb = ch / cpb;
            uint32_t n = 0;
            for (uint32_t fb = g * L.GS; fb < (g + 1) * L.GS; ++fb) n += (uint32_t)__popcll(tap_mask[fb * nCB + cb] & live);
            return n; }, kt_off, sm);
    }
}

// One CTA per block (fb, cb): writes the block's pair words and gathers its kept weights.
template <typename TIn, typename TOut>
__global__ void bp_gather_kernel(npas_bp_desc d, const TIn *__restrict__ w, const uint64_t *__restrict__ tap_mask,
                                 uint8_t *blob)
{
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    if (hdr[BP_MAGIC] != kMagicBP) return;
    const uint32_t nCB = d.C / d.Nb, b = blockIdx.x, fb = b / nCB, cb = b % nCB;
    auto nFB_of = [](const npas_bp_desc &q) { return (uint32_t)(q.K / q.Mb); };
    const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + 128);
    uint32_t *pairs = reinterpret_cast<uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
    TOut *vals = reinterpret_cast<TOut *>(blob + hdr[BP_OFF_VALUES]);
    const uint32_t G = hdr[BP_G], Mb = d.Mb, Nb = d.Nb;
    const uint64_t live = d.R * d.S == 64 ? ~0ull : ((1ull << (d.R * d.S)) - 1);
    uint64_t bits = tap_mask[b] & live;
    uint32_t j = blk_off[b];
    // operand image (bf16 blobs with C % 16 == 0): element (k, tap, c) at
    // ((((k / GI) * nCh + c / 16) * RS + tap) * 2 + (c % 16) / 8) * GI + k % GI) * 8 + c % 8, zeros elsewhere;
    // and the union of kept taps per (filter group, 16-channel chunk)
    const uint32_t off_image = hdr[BP_OFF_IMAGE], GI = hdr[BP_GI], nCh = d.C / 16, RS = d.R * d.S;
    TOut *image = reinterpret_cast<TOut *>(blob + off_image);
    if (off_image && threadIdx.x == 0 && bits) {
        uint32_t *tapu = reinterpret_cast<uint32_t *>(blob + hdr[BP_OFF_TAPU]);
        const uint32_t lo32 = RS > 32 ? 0xFFFFFFFFu : (uint32_t)bits;
        for (uint32_t gi = fb * Mb / GI; gi <= ((fb + 1) * Mb - 1) / GI; ++gi)
            for (uint32_t ch = cb * Nb / 16; ch <= ((cb + 1) * Nb - 1) / 16; ++ch) atomicOr(&tapu[gi * nCh + ch], lo32);
    }
    // tile section: where this block's tile of (chunk, tap) goes inside its (chunk, group) run
    const uint32_t off_kt = hdr[BP_OFF_KT], GS = hdr[BP_GS];
    const uint32_t nGrp = GS ? nFB_of(d) / GS : 0u, grp = GS ? fb / GS : 0u, cpb = Nb / 16;
    const uint32_t *kt_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_KTOFF]);
    TOut *kt = reinterpret_cast<TOut *>(blob + off_kt);
    while (bits) {
        const uint32_t tap = __ffsll((long long)bits) - 1;
        bits &= bits - 1;
        if (threadIdx.x == 0) pairs[j] = cb | (tap << 16);
        uint32_t kt_idx = 0;
        if (off_kt) {
            // tiles of lower taps of the whole group, then the lower blocks of the group that keep this tap
            for (uint32_t f2 = grp * GS; f2 < (grp + 1) * GS; ++f2) {
                const uint64_t m2 = tap_mask[f2 * nCB + cb] & live;
                kt_idx += (uint32_t)__popcll(m2 & ((1ull << tap) - 1ull)) + (f2 < fb ? (uint32_t)((m2 >> tap) & 1ull) : 0u);
            }
        }
        for (uint32_t e = threadIdx.x; e < Mb * Nb; e += blockDim.x) {
            // e enumerates the destination order [c/G][f][c%G] so that stores are contiguous
            const uint32_t cg = e / (Mb * G), f = (e / G) % Mb, cl = e % G, c = cg * G + cl;
            const TIn v = w[((size_t)(fb * Mb + f) * (d.R * d.S) + tap) * d.C + cb * Nb + c];
            TOut o;
            if constexpr (sizeof(TIn) == sizeof(TOut)) o = v;
            else o = f32_bits_to_bf16(v);
            vals[(size_t)j * Mb * Nb + e] = o;
            if (off_image) {
                const uint32_t k = fb * Mb + f, cc = cb * Nb + c;
                image[((((size_t)(k / GI) * nCh + cc / 16) * RS + tap) * 2 + (cc % 16) / 8) * GI * 8 + (k % GI) * 8 + cc % 8] = o;
            }
            if (off_kt) {
                // tile = [Mb/8 filter octets][2 channel octets][8 filters][8 channels]
                const uint32_t ch = cb * cpb + c / 16, c16 = c % 16;
                const size_t tile = (size_t)kt_off[ch * nGrp + grp] + kt_idx;
                kt[tile * Mb * 16 + (((f / 8) * 2 + c16 / 8) * 8 + f % 8) * 8 + c16 % 8] = o;
            }
        }
        ++j;
    }
}

template <typename T>
__global__ void bp_scatter_kernel(npas_bp_desc d, const uint8_t *__restrict__ blob, T *w_out, uint64_t *tap_mask_out)
{
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    const uint32_t nCB = d.C / d.Nb, b = blockIdx.x, fb = b / nCB, cb = b % nCB;
    const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_BLK]);
    const uint32_t *pairs = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
    const T *vals = reinterpret_cast<const T *>(blob + hdr[BP_OFF_VALUES]);
    const uint32_t G = hdr[BP_G], Mb = d.Mb, Nb = d.Nb;
    uint64_t bits = 0;
    for (uint32_t j = blk_off[b]; j < blk_off[b + 1]; ++j) {
        const uint32_t tap = pairs[j] >> 16;
        bits |= 1ull << tap;
        if (!w_out) continue;
        for (uint32_t e = threadIdx.x; e < Mb * Nb; e += blockDim.x) {
            const uint32_t cg = e / (Mb * G), f = (e / G) % Mb, cl = e % G, c = cg * G + cl;
            w_out[((size_t)(fb * Mb + f) * (d.R * d.S) + tap) * d.C + cb * Nb + c] = vals[(size_t)j * Mb * Nb + e];
        }
    }
    if (tap_mask_out && threadIdx.x == 0) tap_mask_out[b] = bits;
}

// dense 0/1 mask [K][R][S][C] -> per-block tap bitsets; counts blocks that break the scheme.
__global__ void bp_mask_from_dense_kernel(npas_bp_desc d, const uint8_t *__restrict__ m, uint64_t *tap_mask,
                                          int32_t *violations)
{
    const uint32_t nCB = d.C / d.Nb, b = blockIdx.x, fb = b / nCB, cb = b % nCB, RS = d.R * d.S;
    auto kernel_bits = [&](uint32_t f, uint32_t c) {
        uint64_t bits = 0;
        for (uint32_t t = 0; t < RS; ++t)
            if (m[((size_t)(fb * d.Mb + f) * RS + t) * d.C + cb * d.Nb + c]) bits |= 1ull << t;
        return bits;
    };
    const uint64_t ref = kernel_bits(0, 0);
    int bad = 0;
    for (uint32_t e = threadIdx.x; e < (uint32_t)(d.Mb * d.Nb); e += blockDim.x)
        bad |= kernel_bits(e / d.Nb, e % d.Nb) != ref;
    bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        tap_mask[b] = ref;
        if (bad) atomicAdd(violations, 1);
    }
}

// ---- block-based -----------------------------------------------------------------------------

__global__ void bb_scan_kernel(npas_bb_desc d, const uint64_t *__restrict__ row_keep,
                               const uint64_t *__restrict__ col_keep, uint8_t *blob, uint32_t blob_bytes,
                               BbLayout L)
{
    __shared__ uint32_t sm[1025];
    const uint64_t rlive = d.Bo == 64 ? ~0ull : ((1ull << d.Bo) - 1), clive = d.Bi == 64 ? ~0ull : ((1ull << d.Bi) - 1);
    uint32_t *hdr = reinterpret_cast<uint32_t *>(blob);
    uint32_t *voff = reinterpret_cast<uint32_t *>(blob + L.off_voff);
    block_exclusive_scan(L.nBlk, [&](uint32_t i) {
        return round_up((uint32_t)(__popcll(row_keep[i] & rlive) * __popcll(col_keep[i] & clive)), 8u); }, voff, sm);
    // Kp = largest kept-column count, rounded up to 16 (at least 16)
    uint32_t mx = 0;
    for (uint32_t i = threadIdx.x; i < L.nBlk; i += blockDim.x) mx = max(mx, (uint32_t)__popcll(col_keep[i] & clive));
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < blockDim.x / 32; ++i) mx = max(mx, sm[i]);
        const uint32_t Kp = max(16u, round_up(mx, 16u));
        const uint32_t nVals = voff[L.nBlk];
        const uint32_t off_tiles = L.off_values + round_up(nVals * L.es, 128);
        const uint32_t total = off_tiles + round_up(L.nBlk * Kp * d.Bo * L.es, 128);
        if (total > blob_bytes) { hdr[BB_TOTAL] = total; return; }     // magic and offsets stay 0: nothing is written
        hdr[BB_MAGIC] = kMagicBB;
        hdr[BB_KP] = Kp; hdr[BB_OFF_TILES] = off_tiles; hdr[BB_OFF_DENSE] = L.off_dense;
        hdr[BB_VERSION] = kVersionBB; hdr[BB_DTYPE] = d.w_packed;
        hdr[BB_O] = d.O; hdr[BB_I] = d.I; hdr[BB_BO] = d.Bo; hdr[BB_BI] = d.Bi;
        hdr[BB_NBO] = L.nBo; hdr[BB_NBI] = L.nBi; hdr[BB_NVALS] = nVals;
        hdr[BB_OFF_CNT] = L.off_cnt; hdr[BB_OFF_ROWS] = L.off_rows; hdr[BB_OFF_COLS] = L.off_cols;
        hdr[BB_OFF_VOFF] = L.off_voff; hdr[BB_OFF_VALUES] = L.off_values; hdr[BB_TOTAL] = total;
    }
}

// One CTA per block: index lists (ascending) and the kept-rows x kept-cols values.
template <typename TIn, typename TOut>
__global__ void bb_gather_kernel(npas_bb_desc d, const TIn *__restrict__ w, const uint64_t *__restrict__ row_keep,
                                 const uint64_t *__restrict__ col_keep, uint8_t *blob, BbLayout L)
{
    __shared__ uint8_t rows[64], cols[64];
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    if (hdr[BB_MAGIC] != kMagicBB) return;
    const uint32_t b = blockIdx.x, bo = b / L.nBi, bi = b % L.nBi, t = threadIdx.x;
    const uint64_t rlive = d.Bo == 64 ? ~0ull : ((1ull << d.Bo) - 1), clive = d.Bi == 64 ? ~0ull : ((1ull << d.Bi) - 1);
    const uint64_t rk = row_keep[b] & rlive, ck = col_keep[b] & clive;
    const uint32_t nr = __popcll(rk), nc = __popcll(ck);
    if (t < 64) {
        // rank of bit t among the set bits = its slot in the ascending list
        const uint64_t below = t == 0 ? 0ull : (~0ull >> (64 - t));
        if (t < (uint32_t)d.Bo && (rk >> t) & 1) rows[__popcll(rk & below)] = (uint8_t)t;
        if (t < (uint32_t)d.Bi && (ck >> t) & 1) cols[__popcll(ck & below)] = (uint8_t)t;
    }
    __syncthreads();
    if (t < (uint32_t)d.Bo) blob[L.off_rows + b * d.Bo + t] = t < nr ? rows[t] : 0xFF;
    if (t < (uint32_t)d.Bi) blob[L.off_cols + b * d.Bi + t] = t < nc ? cols[t] : 0xFF;
    if (t == 0) { blob[L.off_cnt + 2 * b] = (uint8_t)nr; blob[L.off_cnt + 2 * b + 1] = (uint8_t)nc; }
    const uint32_t v0 = reinterpret_cast<const uint32_t *>(blob + L.off_voff)[b];
    TOut *vals = reinterpret_cast<TOut *>(blob + L.off_values) + v0;
    for (uint32_t e = t; e < nr * nc; e += blockDim.x) {
        const TIn v = w[(size_t)(bo * d.Bo + rows[e / nc]) * d.I + bi * d.Bi + cols[e % nc]];
        TOut o;
        if constexpr (sizeof(TIn) == sizeof(TOut)) o = v;
        else o = f32_bits_to_bf16(v);
        vals[e] = o;
        // the same weight in the block's [Kp/8][Bo][8] operand image (the blob was zeroed beforehand)
        const uint32_t Kp = hdr[BB_KP], r = rows[e / nc], c = e % nc;
        TOut *tile = reinterpret_cast<TOut *>(blob + hdr[BB_OFF_TILES]) + (size_t)b * Kp * d.Bo;
        tile[((size_t)(c >> 3) * d.Bo + r) * 8 + (c & 7)] = o;
        // and in the masked dense [O][I] image
        reinterpret_cast<TOut *>(blob + L.off_dense)[(size_t)(bo * d.Bo + r) * d.I + bi * d.Bi + cols[c]] = o;
    }
}

template <typename T>
__global__ void bb_scatter_kernel(npas_bb_desc d, const uint8_t *__restrict__ blob, T *w_out, uint64_t *rk_out,
                                  uint64_t *ck_out, BbLayout L)
{
    const uint32_t b = blockIdx.x, bo = b / L.nBi, bi = b % L.nBi, t = threadIdx.x;
    const uint32_t nr = blob[L.off_cnt + 2 * b], nc = blob[L.off_cnt + 2 * b + 1];
    const uint8_t *rows = blob + L.off_rows + b * d.Bo, *cols = blob + L.off_cols + b * d.Bi;
    if (t == 0) {
        uint64_t rk = 0, ck = 0;
        for (uint32_t i = 0; i < nr; ++i) rk |= 1ull << rows[i];
        for (uint32_t i = 0; i < nc; ++i) ck |= 1ull << cols[i];
        if (rk_out) rk_out[b] = rk;
        if (ck_out) ck_out[b] = ck;
    }
    if (!w_out) return;
    const uint32_t v0 = reinterpret_cast<const uint32_t *>(blob + L.off_voff)[b];
    const T *vals = reinterpret_cast<const T *>(blob + L.off_values) + v0;
    for (uint32_t e = t; e < nr * nc; e += blockDim.x)
        w_out[(size_t)(bo * d.Bo + rows[e / nc]) * d.I + bi * d.Bi + cols[e % nc]] = vals[e];
}

__global__ void bb_mask_from_dense_kernel(npas_bb_desc d, const uint8_t *__restrict__ m, uint64_t *row_keep,
                                          uint64_t *col_keep, int32_t *violations, uint32_t nBi)
{
    __shared__ uint64_t rowbits[64];
    const uint32_t b = blockIdx.x, bo = b / nBi, bi = b % nBi, t = threadIdx.x;
    uint64_t mine = 0;
    if (t < (uint32_t)d.Bo)
        for (uint32_t c = 0; c < (uint32_t)d.Bi; ++c)
            if (m[(size_t)(bo * d.Bo + t) * d.I + bi * d.Bi + c]) mine |= 1ull << c;
    rowbits[t] = mine;
    __syncthreads();
    uint64_t ck = 0, rk = 0;
    for (uint32_t r = 0; r < (uint32_t)d.Bo; ++r) { ck |= rowbits[r]; if (rowbits[r]) rk |= 1ull << r; }
    const int bad = __syncthreads_or(t < (uint32_t)d.Bo && mine != 0 && mine != ck);
    if (t == 0) {
        row_keep[b] = rk; col_keep[b] = ck;
        if (bad) atomicAdd(violations, 1);
    }
}

// The size a blob needs is known only on the device (it depends on the masks there).  The scan
// kernel leaves the magic word 0 when the caller's buffer is too small; read it back and say so.
static npas_status packed_fits(const void *blob, int magic_word, uint32_t magic, cudaStream_t st)
{
    uint32_t m = 0;
    if (cudaMemcpyAsync(&m, static_cast<const uint32_t *>(blob) + magic_word, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return NPAS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NPAS_ERR_CUDA;
    return m == magic ? NPAS_OK : NPAS_ERR_BUFFER_TOO_SMALL;
}

}  // namespace npas

using namespace npas;

// ================================================================================================
extern "C" {

npas_status npas_pack_bp_size(const npas_bp_desc *d, const uint64_t *tap_mask_host, size_t *blob_bytes)
{
    npas_status s = check_bp_desc(d);
    if (s != NPAS_OK) return s;
    if (!tap_mask_host || !blob_bytes) return NPAS_ERR_NULL;
    const uint64_t live = d->R * d->S == 64 ? ~0ull : ((1ull << (d->R * d->S)) - 1);
    uint64_t n = 0;
    for (int i = 0; i < (d->K / d->Mb) * (d->C / d->Nb); ++i) n += __builtin_popcountll(tap_mask_host[i] & live);
    if (n * d->Mb * d->Nb * 4 > 0x7FFFFFFFull) return NPAS_ERR_SHAPE;
    *blob_bytes = bp_layout(*d, (uint32_t)n).total;
    return NPAS_OK;
}

npas_status npas_pack_bp(const npas_bp_desc *d, const void *w, const uint64_t *tap_mask, void *blob,
                         size_t blob_bytes, void *stream)
{
    npas_status s = check_bp_desc(d);
    if (s != NPAS_OK) return s;
    if (!w || !tap_mask || !blob) return NPAS_ERR_NULL;
    if (!aligned16(w) || !aligned16(blob) || (reinterpret_cast<uintptr_t>(tap_mask) & 7)) return NPAS_ERR_ALIGNMENT;
    if (blob_bytes < bp_layout(*d, 0).total || blob_bytes > 0xFFFFFFFFull) return NPAS_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(blob, 0, blob_bytes, st) != cudaSuccess) return NPAS_ERR_CUDA;
    const uint32_t nBlk = (d->K / d->Mb) * (d->C / d->Nb);
    uint8_t *b8 = static_cast<uint8_t *>(blob);
    bp_scan_kernel<<<1, 1024, 0, st>>>(*d, tap_mask, b8, (uint32_t)blob_bytes);
    if (d->w_in == NPAS_F32 && d->w_packed == NPAS_F32)
        bp_gather_kernel<uint32_t, uint32_t><<<nBlk, 128, 0, st>>>(*d, static_cast<const uint32_t *>(w), tap_mask, b8);
    else if (d->w_in == NPAS_F32)
        bp_gather_kernel<uint32_t, uint16_t><<<nBlk, 128, 0, st>>>(*d, static_cast<const uint32_t *>(w), tap_mask, b8);
    else
        bp_gather_kernel<uint16_t, uint16_t><<<nBlk, 128, 0, st>>>(*d, static_cast<const uint16_t *>(w), tap_mask, b8);
    count_launch(2);
    if (launch_status() != NPAS_OK) return NPAS_ERR_CUDA;
    return packed_fits(blob, BP_MAGIC, kMagicBP, st);
}

npas_status npas_unpack_bp(const npas_bp_desc *d, const void *blob, size_t blob_bytes, void *w_out,
                           uint64_t *tap_mask_out, void *stream)
{
    npas_status s = check_bp_desc(d);
    if (s != NPAS_OK) return s;
    if (!blob) return NPAS_ERR_NULL;
    if (!aligned16(blob) || (w_out && !aligned16(w_out))) return NPAS_ERR_ALIGNMENT;
    if (blob_bytes < bp_layout(*d, 0).total) return NPAS_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t nW = (size_t)d->K * d->R * d->S * d->C;
    if (w_out && cudaMemsetAsync(w_out, 0, nW * dtype_size(d->w_packed), st) != cudaSuccess) return NPAS_ERR_CUDA;
    const uint32_t nBlk = (d->K / d->Mb) * (d->C / d->Nb);
    const uint8_t *b8 = static_cast<const uint8_t *>(blob);
    if (d->w_packed == NPAS_F32)
        bp_scatter_kernel<uint32_t><<<nBlk, 128, 0, st>>>(*d, b8, static_cast<uint32_t *>(w_out), tap_mask_out);
    else
        bp_scatter_kernel<uint16_t><<<nBlk, 128, 0, st>>>(*d, b8, static_cast<uint16_t *>(w_out), tap_mask_out);
    count_launch();
    return launch_status();
}

npas_status npas_mask_bp_from_dense(const npas_bp_desc *d, const uint8_t *m, uint64_t *tap_mask,
                                    int32_t *violations, void *stream)
{
    npas_status s = check_bp_desc(d);
    if (s != NPAS_OK) return s;
    if (!m || !tap_mask || !violations) return NPAS_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(violations, 0, 4, st) != cudaSuccess) return NPAS_ERR_CUDA;
    bp_mask_from_dense_kernel<<<(d->K / d->Mb) * (d->C / d->Nb), 128, 0, st>>>(*d, m, tap_mask, violations);
    count_launch();
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, violations, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NPAS_ERR_CUDA;
    return v ? NPAS_ERR_MASK_STRUCTURE : NPAS_OK;
}

npas_status npas_pack_bb_size(const npas_bb_desc *d, const uint64_t *rk, const uint64_t *ck, size_t *blob_bytes)
{
    npas_status s = check_bb_desc(d);
    if (s != NPAS_OK) return s;
    if (!rk || !ck || !blob_bytes) return NPAS_ERR_NULL;
    const BbLayout L = bb_layout(*d);
    const uint64_t rlive = d->Bo == 64 ? ~0ull : ((1ull << d->Bo) - 1), clive = d->Bi == 64 ? ~0ull : ((1ull << d->Bi) - 1);
    uint64_t n = 0;
    uint32_t mx = 0;
    for (uint32_t i = 0; i < L.nBlk; ++i) {
        n += round_up((uint32_t)(__builtin_popcountll(rk[i] & rlive) * __builtin_popcountll(ck[i] & clive)), 8u);
        mx = mx > (uint32_t)__builtin_popcountll(ck[i] & clive) ? mx : (uint32_t)__builtin_popcountll(ck[i] & clive);
    }
    const uint32_t Kp = round_up(mx, 16u) < 16u ? 16u : round_up(mx, 16u);
    const uint64_t tiles = (uint64_t)L.nBlk * Kp * d->Bo * L.es;
    if (n * 4 > 0x3FFFFFFFull || tiles > 0x3FFFFFFFull) return NPAS_ERR_SHAPE;
    *blob_bytes = (size_t)L.off_values + round_up((uint32_t)n * L.es, 128) + round_up((uint32_t)tiles, 128);
    return NPAS_OK;
}

npas_status npas_pack_bb(const npas_bb_desc *d, const void *w, const uint64_t *rk, const uint64_t *ck,
                         void *blob, size_t blob_bytes, void *stream)
{
    npas_status s = check_bb_desc(d);
    if (s != NPAS_OK) return s;
    if (!w || !rk || !ck || !blob) return NPAS_ERR_NULL;
    if (!aligned16(w) || !aligned16(blob)) return NPAS_ERR_ALIGNMENT;
    const BbLayout L = bb_layout(*d);
    if (blob_bytes < L.off_values || blob_bytes > 0xFFFFFFFFull) return NPAS_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(blob, 0, blob_bytes, st) != cudaSuccess) return NPAS_ERR_CUDA;
    uint8_t *b8 = static_cast<uint8_t *>(blob);
    bb_scan_kernel<<<1, 1024, 0, st>>>(*d, rk, ck, b8, (uint32_t)blob_bytes, L);
    if (d->w_in == NPAS_F32 && d->w_packed == NPAS_F32)
        bb_gather_kernel<uint32_t, uint32_t><<<L.nBlk, 128, 0, st>>>(*d, static_cast<const uint32_t *>(w), rk, ck, b8, L);
    else if (d->w_in == NPAS_F32)
        bb_gather_kernel<uint32_t, uint16_t><<<L.nBlk, 128, 0, st>>>(*d, static_cast<const uint32_t *>(w), rk, ck, b8, L);
    else
        bb_gather_kernel<uint16_t, uint16_t><<<L.nBlk, 128, 0, st>>>(*d, static_cast<const uint16_t *>(w), rk, ck, b8, L);
    count_launch(2);
    if (launch_status() != NPAS_OK) return NPAS_ERR_CUDA;
    return packed_fits(blob, BB_MAGIC, kMagicBB, st);
}

npas_status npas_unpack_bb(const npas_bb_desc *d, const void *blob, size_t blob_bytes, void *w_out,
                           uint64_t *rk_out, uint64_t *ck_out, void *stream)
{
    npas_status s = check_bb_desc(d);
    if (s != NPAS_OK) return s;
    if (!blob) return NPAS_ERR_NULL;
    if (!aligned16(blob) || (w_out && !aligned16(w_out))) return NPAS_ERR_ALIGNMENT;
    const BbLayout L = bb_layout(*d);
    if (blob_bytes < L.off_values) return NPAS_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (w_out && cudaMemsetAsync(w_out, 0, (size_t)d->O * d->I * L.es, st) != cudaSuccess) return NPAS_ERR_CUDA;
    const uint8_t *b8 = static_cast<const uint8_t *>(blob);
    if (d->w_packed == NPAS_F32)
        bb_scatter_kernel<uint32_t><<<L.nBlk, 128, 0, st>>>(*d, b8, static_cast<uint32_t *>(w_out), rk_out, ck_out, L);
    else
        bb_scatter_kernel<uint16_t><<<L.nBlk, 128, 0, st>>>(*d, b8, static_cast<uint16_t *>(w_out), rk_out, ck_out, L);
    count_launch();
    return launch_status();
}

npas_status npas_mask_bb_from_dense(const npas_bb_desc *d, const uint8_t *m, uint64_t *rk, uint64_t *ck,
                                    int32_t *violations, void *stream)
{
    npas_status s = check_bb_desc(d);
    if (s != NPAS_OK) return s;
    if (!m || !rk || !ck || !violations) return NPAS_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(violations, 0, 4, st) != cudaSuccess) return NPAS_ERR_CUDA;
    const BbLayout L = bb_layout(*d);
    bb_mask_from_dense_kernel<<<L.nBlk, 64, 0, st>>>(*d, m, rk, ck, violations, L.nBi);
    count_launch();
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, violations, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NPAS_ERR_CUDA;
    return v ? NPAS_ERR_MASK_STRUCTURE : NPAS_OK;
}

}  // extern "C"
