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
