// One-shot magnitude pruning of a layer under the two schemes (paper Sec. 5.2): turns dense
// weights into the block masks the packers take.  The score of a prunable group (a tap of a block;
// a row or a column of a block) is the sum of the squares of its weights, accumulated in fp64 in a
// fixed order (filters / rows outer, channels / columns inner; a square of a float is exact in
// fp64, so fused or separate multiply-add give the same bits); a block keeps its `keep`
// highest-scoring groups, ties go to the lower index.  Offline step: one CTA per block.
#include "common.cuh"

namespace npas {

template <typename T> __device__ inline double prune_load(const T *p);
template <> __device__ inline double prune_load<float>(const float *p) { return (double)*p; }
template <> __device__ inline double prune_load<uint16_t>(const uint16_t *p) { return (double)bf16_bits_to_f32(*p); }

// the `keep` largest of n <= 64 scores as a bitset; ties to the lower index
__device__ inline uint64_t top_k_bits(const double *score, int n, int keep)
{
    uint64_t bits = 0;
    for (int k = 0; k < keep; ++k) {
        int best = -1;
        for (int t = 0; t < n; ++t)
            if (!((bits >> t) & 1ull) && (best < 0 || score[t] > score[best])) best = t;
        bits |= 1ull << best;
    }
    return bits;
}

template <typename T>
__global__ void prune_bp_kernel(npas_bp_desc d, const T *__restrict__ w, int keep, uint64_t *tap_mask)
{
    __shared__ double score[64];
    const int RS = d.R * d.S, nCB = d.C / d.Nb, b = blockIdx.x, fb = b / nCB, cb = b - fb * nCB;
    const int t = threadIdx.x;
    if (t < RS) {
        double s = 0.0;
        for (int f = 0; f < d.Mb; ++f)
            for (int c = 0; c < d.Nb; ++c) {
                const double v = prune_load(w + ((size_t)(fb * d.Mb + f) * RS + t) * d.C + cb * d.Nb + c);
                s = fma(v, v, s);
            }
        score[t] = s;
    }
    __syncthreads();
    if (t == 0) tap_mask[b] = top_k_bits(score, RS, keep);
}

template <typename T>
__global__ void prune_bb_kernel(npas_bb_desc d, const T *__restrict__ w, int keep_rows, int keep_cols,
                                uint64_t *row_keep, uint64_t *col_keep)
{
    __shared__ double rs[64], cs[64];
    const int nBi = d.I / d.Bi, b = blockIdx.x, bo = b / nBi, bi = b - bo * nBi, t = threadIdx.x;
    const T *blk = w + (size_t)bo * d.Bo * d.I + (size_t)bi * d.Bi;
    if (t < d.Bo) {
        double s = 0.0;
        for (int c = 0; c < d.Bi; ++c) { const double v = prune_load(blk + (size_t)t * d.I + c); s = fma(v, v, s); }
        rs[t] = s;
    } else if (t >= 64 && t - 64 < d.Bi) {
        const int c = t - 64;
        double s = 0.0;
        for (int r = 0; r < d.Bo; ++r) { const double v = prune_load(blk + (size_t)r * d.I + c); s = fma(v, v, s); }
        cs[c] = s;
    }
    __syncthreads();
    if (t == 0) row_keep[b] = top_k_bits(rs, d.Bo, keep_rows);
    if (t == 64) col_keep[b] = top_k_bits(cs, d.Bi, keep_cols);
}

// ---- layer-wide budget -------------------------------------------------------------------------
// Scores of all (block, tap) groups, in group order (block major, tap minor), as fp64.
template <typename T>
__global__ void prune_bp_scores_kernel(npas_bp_desc d, const T *__restrict__ w, double *scores)
{
    const int RS = d.R * d.S, nCB = d.C / d.Nb, b = blockIdx.x, fb = b / nCB, cb = b - fb * nCB;
    const int t = threadIdx.x;
    if (t >= RS) return;
    double s = 0.0;
    for (int f = 0; f < d.Mb; ++f)
        for (int c = 0; c < d.Nb; ++c) {
            const double v = prune_load(w + ((size_t)(fb * d.Mb + f) * RS + t) * d.C + cb * d.Nb + c);
            s = fma(v, v, s);
        }
    scores[(size_t)b * RS + t] = s;
}

// Keeps the n_keep largest of G scores, ties to the lower index.  One CTA.  A sum of squares is never
// negative, so the order of the fp64 values is the order of their bit patterns as unsigned integers:
// the n_keep-th largest pattern is found by a radix select, eight bits at a time from the top (count the
// candidates per digit, walk the digits downwards until the remaining budget falls inside one, narrow
// the candidates to that digit).  Groups above the threshold are kept; of the groups equal to it, the
// first `need` in index order.
__global__ void prune_select_kernel(const unsigned long long *__restrict__ keys, long long G, long long n_keep, int RS,
                                    unsigned long long *tap_mask, long long n_blocks)
{
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ long long s_need;
    __shared__ unsigned int warp_sums[32];
    __shared__ long long s_seen;
    const int t = threadIdx.x, T = blockDim.x;
    for (long long b = t; b < n_blocks; b += T) tap_mask[b] = 0ull;
    if (n_keep <= 0) return;
    if (t == 0) { s_prefix = 0ull; s_need = n_keep; }
    __syncthreads();
    for (int shift = 56; shift >= 0; shift -= 8) {
        for (int i = t; i < 256; i += T) hist[i] = 0u;
        __syncthreads();
        const unsigned long long prefix = s_prefix;
        const unsigned long long high_mask = shift == 56 ? 0ull : ~0ull << (shift + 8);
        for (long long i = t; i < G; i += T) {
            const unsigned long long k = keys[i];
            if ((k & high_mask) == prefix) atomicAdd(&hist[(unsigned)(k >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (t == 0) {
            long long need = s_need;
            int digit = 255;
            for (; digit > 0; --digit) {                       // from the largest digit down
                if ((long long)hist[digit] >= need) break;
                need -= hist[digit];
            }
            s_need = need;                                      // still to take among the keys with this digit
            s_prefix = prefix | ((unsigned long long)digit << shift);
        }
        __syncthreads();
    }
    const unsigned long long thr = s_prefix;                    // the n_keep-th largest key
    const long long need = s_need;                              // how many keys equal to it are kept
    if (t == 0) s_seen = 0;
    __syncthreads();
    // in index order: every key above the threshold, and the first `need` equal to it
    for (long long base = 0; base < G; base += T) {
        const long long i = base + t;
        const unsigned long long k = i < G ? keys[i] : 0ull;
        const bool eq = i < G && k == thr;
        // rank of this thread among the equal keys of the chunk
        const unsigned int ballot = __ballot_sync(0xFFFFFFFFu, eq);
        const int lane = t & 31, wid = t >> 5;
        if (lane == 0) warp_sums[wid] = __popc(ballot);
        __syncthreads();
        long long before = s_seen;
        for (int wv = 0; wv < wid; ++wv) before += warp_sums[wv];
        before += __popc(ballot & ((1u << lane) - 1u));
        if (i < G && (k > thr || (eq && before < need)))
            atomicOr(&tap_mask[i / RS], 1ull << (unsigned)(i % RS));
        __syncthreads();
        if (t == 0) {
            long long tot = 0;
            for (int wv = 0; wv < T / 32; ++wv) tot += warp_sums[wv];
            s_seen += tot;
        }
        __syncthreads();
    }
}

extern "C" {

npas_status npas_prune_bp_magnitude(const npas_bp_desc *d, const void *w, int32_t keep_taps, uint64_t *tap_mask,
                                    void *stream)
{
    npas_status s = check_bp_desc(d);
    if (s != NPAS_OK) return s;
    if (!w || !tap_mask) return NPAS_ERR_NULL;
    if (keep_taps < 0 || keep_taps > d->R * d->S) return NPAS_ERR_SHAPE;
    if (!aligned16(w) || (reinterpret_cast<uintptr_t>(tap_mask) & 7)) return NPAS_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int nBlk = (d->K / d->Mb) * (d->C / d->Nb);
    if (d->w_in == NPAS_F32) prune_bp_kernel<float><<<nBlk, 64, 0, st>>>(*d, static_cast<const float *>(w), keep_taps, tap_mask);
    else prune_bp_kernel<uint16_t><<<nBlk, 64, 0, st>>>(*d, static_cast<const uint16_t *>(w), keep_taps, tap_mask);
    count_launch();
    return launch_status();
}

npas_status npas_prune_bp_global_workspace(const npas_bp_desc *d, size_t *ws_bytes)
{
    npas_status s = check_bp_desc(d);
    if (s != NPAS_OK) return s;
    if (!ws_bytes) return NPAS_ERR_NULL;
    *ws_bytes = round_up((uint32_t)((d->K / d->Mb) * (d->C / d->Nb) * d->R * d->S) * 8u, 256);
    return NPAS_OK;
}

npas_status npas_prune_bp_magnitude_global(const npas_bp_desc *d, const void *w, int64_t n_keep, uint64_t *tap_mask,
                                           void *ws, size_t ws_bytes, void *stream)
{
    npas_status s = check_bp_desc(d);
    if (s != NPAS_OK) return s;
    if (!w || !tap_mask || !ws) return NPAS_ERR_NULL;
    const long long nBlk = (long long)(d->K / d->Mb) * (d->C / d->Nb), G = nBlk * d->R * d->S;
    if (n_keep < 0 || n_keep > G) return NPAS_ERR_SHAPE;
    if (!aligned16(w) || !aligned16(ws) || (reinterpret_cast<uintptr_t>(tap_mask) & 7)) return NPAS_ERR_ALIGNMENT;
    size_t need = 0;
    npas_prune_bp_global_workspace(d, &need);
    if (ws_bytes < need) return NPAS_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double *scores = static_cast<double *>(ws);
    if (d->w_in == NPAS_F32) prune_bp_scores_kernel<float><<<(unsigned)nBlk, 64, 0, st>>>(*d, static_cast<const float *>(w), scores);
    else prune_bp_scores_kernel<uint16_t><<<(unsigned)nBlk, 64, 0, st>>>(*d, static_cast<const uint16_t *>(w), scores);
    prune_select_kernel<<<1, 1024, 0, st>>>(reinterpret_cast<const unsigned long long *>(scores), G, (long long)n_keep, d->R * d->S,
                                            reinterpret_cast<unsigned long long *>(tap_mask), nBlk);
    count_launch(2);
    return launch_status();
}

npas_status npas_prune_bb_magnitude(const npas_bb_desc *d, const void *w, int32_t keep_rows, int32_t keep_cols,
                                    uint64_t *row_keep, uint64_t *col_keep, void *stream)
{
    npas_status s = check_bb_desc(d);
    if (s != NPAS_OK) return s;
    if (!w || !row_keep || !col_keep) return NPAS_ERR_NULL;
    if (keep_rows < 0 || keep_rows > d->Bo || keep_cols < 0 || keep_cols > d->Bi) return NPAS_ERR_SHAPE;
    if (!aligned16(w) || (reinterpret_cast<uintptr_t>(row_keep) & 7) || (reinterpret_cast<uintptr_t>(col_keep) & 7))
        return NPAS_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int nBlk = (d->O / d->Bo) * (d->I / d->Bi);
    if (d->w_in == NPAS_F32)
        prune_bb_kernel<float><<<nBlk, 128, 0, st>>>(*d, static_cast<const float *>(w), keep_rows, keep_cols, row_keep, col_keep);
    else
        prune_bb_kernel<uint16_t><<<nBlk, 128, 0, st>>>(*d, static_cast<const uint16_t *>(w), keep_rows, keep_cols, row_keep, col_keep);
    count_launch();
    return launch_status();
}

}  // extern "C"

}  // namespace npas
