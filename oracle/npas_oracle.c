/*
 * CPU oracle for block-punched convolution and block-based pruned GEMM.
 *
 * TEST INFRASTRUCTURE ONLY: a plain, slow, fp64 restatement of the definitions.  It shares no
 * code with the CUDA library and is never on a product path; only the tests, the smoke check
 * and the benchmark's CPU-baseline leg call it.
 *
 * What it computes (paper Sec. 3):
 *   - "Block-punched Pruning": the weight tensor is cut into blocks of Mb filters x Nb input
 *     channels; inside a block the same kernel positions (taps) are pruned in every filter and
 *     every channel.  A pruned weight is absent, i.e. zero, so the layer output is the ordinary
 *     convolution (cross-correlation, zero padding) over the masked dense weights.
 *   - "Block-based Pruning": the weight matrix is cut into equal blocks; inside each block whole
 *     rows and/or columns are pruned.  A weight survives iff its row and its column both survive
 *     in its own block; the output is the ordinary matrix product over the masked weights.
 *
 * Nothing here knows about packed formats, tap lists or tiles: the loops run over the dense
 * tensors and evaluate the mask predicate term by term.
 */
#include <stdint.h>
#include <stdlib.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* mask predicate of block-punched pruning: is tap (r,s) of kernel (k,c) kept? */
static inline int bp_kept(const uint64_t *tap_mask, int C, int S, int Mb, int Nb,
                          int k, int r, int s, int c)
{
    int n_cb = C / Nb;
    uint64_t bits = tap_mask[(size_t)(k / Mb) * n_cb + (c / Nb)];
    return (int)((bits >> (r * S + s)) & 1u);
}

/* one output element of the block-punched convolution, fp64 */
static double conv_point(int H, int W, int C, int R, int S, int stride, int pad, int Mb, int Nb,
                         const double *x, const double *w, const uint64_t *tap_mask,
                         const double *bias, const double *res, int relu,
                         int P, int Q, int K, int n, int p, int q, int k)
{
    double acc = bias ? bias[k] : 0.0;
    for (int r = 0; r < R; ++r) {
        for (int s = 0; s < S; ++s) {
            int h = p * stride + r - pad;
            int v = q * stride + s - pad;
            if (h < 0 || h >= H || v < 0 || v >= W) continue;   /* zero padding */
            for (int c = 0; c < C; ++c) {
                if (!bp_kept(tap_mask, C, S, Mb, Nb, k, r, s, c)) continue;  /* pruned = absent */
                double xv = x[(((size_t)n * H + h) * W + v) * C + c];
                double wv = w[(((size_t)k * R + r) * S + s) * C + c];
                acc += xv * wv;
            }
        }
    }
    if (res) acc += res[(((size_t)n * P + p) * Q + q) * K + k];
    if (relu && acc < 0.0) acc = 0.0;
    return acc;
}

/* Y[n,p,q,k] = act(b[k] + sum_{r,s,c} m[k,r,s,c] W[k,r,s,c] Xpad[n, p*stride+r-pad, q*stride+s-pad, c] (+Res))
 * x: [N,H,W,C]  w: [K,R,S,C]  tap_mask: [K/Mb][C/Nb]  y,res: [N,P,Q,K]; bias/res may be NULL. */
int oracle_conv2d_bp(int N, int H, int W, int C, int K, int R, int S, int stride, int pad,
                     int Mb, int Nb, const double *x, const double *w, const uint64_t *tap_mask,
                     const double *bias, const double *res, int relu, double *y)
{
    if (Mb <= 0 || Nb <= 0 || K % Mb || C % Nb || R * S > 64 || stride <= 0) return 1;
    int P = (H + 2 * pad - R) / stride + 1;
    int Q = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int k = 0; k < K; ++k)
                    y[(((size_t)n * P + p) * Q + q) * K + k] =
                        conv_point(H, W, C, R, S, stride, pad, Mb, Nb, x, w, tap_mask, bias, res,
                                   relu, P, Q, K, n, p, q, k);
    return 0;
}

/* Same definition, evaluated only at the listed output coordinates idx[i] = {n,p,q,k}. */
int oracle_conv2d_bp_points(int N, int H, int W, int C, int K, int R, int S, int stride, int pad,
                            int Mb, int Nb, const double *x, const double *w,
                            const uint64_t *tap_mask, const double *bias, const double *res,
                            int relu, const int32_t *idx, int64_t n_points, double *out)
{
    if (Mb <= 0 || Nb <= 0 || K % Mb || C % Nb || R * S > 64 || stride <= 0) return 1;
    int P = (H + 2 * pad - R) / stride + 1;
    int Q = (W + 2 * pad - S) / stride + 1;
    (void)N;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_points; ++i)
        out[i] = conv_point(H, W, C, R, S, stride, pad, Mb, Nb, x, w, tap_mask, bias, res, relu,
                            P, Q, K, idx[4 * i], idx[4 * i + 1], idx[4 * i + 2], idx[4 * i + 3]);
    return 0;
}

/* mask predicate of block-based pruning: weight (o,i) survives iff its row and its column are
 * both kept inside its own block */
static inline int bb_kept(const uint64_t *row_keep, const uint64_t *col_keep, int I, int Bo,
                          int Bi, int o, int i)
{
    size_t blk = (size_t)(o / Bo) * (I / Bi) + (i / Bi);
    return (int)(((row_keep[blk] >> (o % Bo)) & 1u) & ((col_keep[blk] >> (i % Bi)) & 1u));
}

static double linear_point(int I, int Bo, int Bi, const double *x, const double *w,
                           const uint64_t *row_keep, const uint64_t *col_keep, const double *bias,
                           const double *res, int O, int relu, int m, int o)
{
    double acc = bias ? bias[o] : 0.0;
    for (int i = 0; i < I; ++i) {
        if (!bb_kept(row_keep, col_keep, I, Bo, Bi, o, i)) continue;
        acc += x[(size_t)m * I + i] * w[(size_t)o * I + i];
    }
    if (res) acc += res[(size_t)m * O + o];      /* shortcut branch, added before the activation */
    if (relu && acc < 0.0) acc = 0.0;
    return acc;
}

/* Y[m,o] = act(b[o] + sum_i X[m,i] m[o,i] W[o,i] (+ res[m,o]));  x: [M,I]  w: [O,I]  y, res: [M,O] */
int oracle_linear_bb(int M, int I, int O, int Bo, int Bi, const double *x, const double *w,
                     const uint64_t *row_keep, const uint64_t *col_keep, const double *bias,
                     const double *res, int relu, double *y)
{
    if (Bo <= 0 || Bi <= 0 || Bo > 64 || Bi > 64 || O % Bo || I % Bi) return 1;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int o = 0; o < O; ++o)
            y[(size_t)m * O + o] = linear_point(I, Bo, Bi, x, w, row_keep, col_keep, bias, res, O, relu, m, o);
    return 0;
}

int oracle_linear_bb_points(int M, int I, int O, int Bo, int Bi, const double *x, const double *w,
                            const uint64_t *row_keep, const uint64_t *col_keep,
                            const double *bias, const double *res, int relu, const int32_t *idx,
                            int64_t n_points, double *out)
{
    if (Bo <= 0 || Bi <= 0 || Bo > 64 || Bi > 64 || O % Bo || I % Bi) return 1;
    (void)M;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_points; ++i)
        out[i] = linear_point(I, Bo, Bi, x, w, row_keep, col_keep, bias, res, O, relu, idx[2 * i], idx[2 * i + 1]);
    return 0;
}

/* 3x3 stride-2 pad-1 style max pooling on NHWC (used only by the layer-stack checks). */
int oracle_maxpool2d(int N, int H, int W, int C, int R, int stride, int pad, const double *x,
                     double *y)
{
    int P = (H + 2 * pad - R) / stride + 1;
    int Q = (W + 2 * pad - R) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int c = 0; c < C; ++c) {
                    double best = 0.0;
                    int seen = 0;
                    for (int r = 0; r < R; ++r)
                        for (int s = 0; s < R; ++s) {
                            int h = p * stride + r - pad, v = q * stride + s - pad;
                            if (h < 0 || h >= H || v < 0 || v >= W) continue;
                            double xv = x[(((size_t)n * H + h) * W + v) * C + c];
                            if (!seen || xv > best) { best = xv; seen = 1; }
                        }
                    y[(((size_t)n * P + p) * Q + q) * C + c] = best;
                }
    return 0;
}

/*
 * One-shot magnitude pruning of a layer under the two schemes (paper Sec. 5.2, "One-shot Pruning
 * and Early Stopping for Fast Accuracy Evaluation": the layer is pruned once, by weight magnitude,
 * following the scheme and rate of the candidate).  The paper does not say how magnitudes are
 * grouped; the reading taken: the score of a prunable group is the sum of the squares of its
 * weights (the squared L2 norm), a block keeps its `keep` highest-scoring groups, ties go to the
 * lower index.  Sums are fp64, taken in the order filter-major / channel-minor (rows: columns
 * ascending; columns: rows ascending) so that the selection is reproducible bit for bit.
 *
 * Block-punched: group = one tap of one block (all Mb x Nb weights at that kernel position).
 */
int oracle_prune_bp(int K, int C, int R, int S, int Mb, int Nb, const double *w, int keep,
                    uint64_t *tap_mask)
{
    int RS = R * S, n_fb = K / Mb, n_cb = C / Nb;
    if (K % Mb || C % Nb || RS > 64 || keep < 0 || keep > RS) return 1;
    for (int fb = 0; fb < n_fb; ++fb)
        for (int cb = 0; cb < n_cb; ++cb) {
            double score[64];
            for (int t = 0; t < RS; ++t) {
                double s = 0.0;
                for (int f = 0; f < Mb; ++f)
                    for (int c = 0; c < Nb; ++c) {
                        double v = w[((size_t)(fb * Mb + f) * RS + t) * C + cb * Nb + c];
                        s += v * v;
                    }
                score[t] = s;
            }
            uint64_t bits = 0;
            for (int n = 0; n < keep; ++n) {            /* repeatedly take the best tap not yet taken */
                int best = -1;
                for (int t = 0; t < RS; ++t)
                    if (!((bits >> t) & 1) && (best < 0 || score[t] > score[best])) best = t;
                bits |= (uint64_t)1 << best;
            }
            tap_mask[(size_t)fb * n_cb + cb] = bits;
        }
    return 0;
}

/*
 * One-shot magnitude pruning to a layer-wide budget (paper Sec. 5.2 with the pruning rates of Table 1,
 * e.g. 2.5x or 7x, which no uniform per-block count can express): of all G = (K/Mb)(C/Nb)(R*S)
 * prunable groups of the layer (one tap of one block, scored as above) the n_keep with the largest
 * scores are kept, ties going to the lower group index (blocks filter-block major, taps ascending).
 * Plain definition: sort all groups by (score descending, index ascending), keep the first n_keep.
 */
typedef struct { double score; int64_t index; } oracle_group;

static int oracle_group_cmp(const void *a, const void *b)
{
    const oracle_group *x = (const oracle_group *)a, *y = (const oracle_group *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return x->index < y->index ? -1 : (x->index > y->index ? 1 : 0);
}

int oracle_prune_bp_global(int K, int C, int R, int S, int Mb, int Nb, const double *w, int64_t n_keep,
                           uint64_t *tap_mask)
{
    int RS = R * S, n_fb = K / Mb, n_cb = C / Nb;
    int64_t G = (int64_t)n_fb * n_cb * RS;
    if (K % Mb || C % Nb || RS > 64 || n_keep < 0 || n_keep > G) return 1;
    oracle_group *g = (oracle_group *)malloc((size_t)(G ? G : 1) * sizeof(oracle_group));
    if (!g) return 2;
    for (int fb = 0; fb < n_fb; ++fb)
        for (int cb = 0; cb < n_cb; ++cb)
            for (int t = 0; t < RS; ++t) {
                double s = 0.0;
                for (int f = 0; f < Mb; ++f)
                    for (int c = 0; c < Nb; ++c) {
                        double v = w[((size_t)(fb * Mb + f) * RS + t) * C + cb * Nb + c];
                        s += v * v;
                    }
                int64_t i = ((int64_t)fb * n_cb + cb) * RS + t;
                g[i].score = s;
                g[i].index = i;
            }
    qsort(g, (size_t)G, sizeof(oracle_group), oracle_group_cmp);
    for (int64_t b = 0; b < (int64_t)n_fb * n_cb; ++b) tap_mask[b] = 0;
    for (int64_t j = 0; j < n_keep; ++j) tap_mask[g[j].index / RS] |= (uint64_t)1 << (g[j].index % RS);
    free(g);
    return 0;
}

/* Block-based: groups = the rows and the columns of a block, scored over the whole block. */
int oracle_prune_bb(int O, int I, int Bo, int Bi, const double *w, int keep_rows, int keep_cols,
                    uint64_t *row_keep, uint64_t *col_keep)
{
    int n_bo = O / Bo, n_bi = I / Bi;
    if (O % Bo || I % Bi || Bo > 64 || Bi > 64 || keep_rows < 0 || keep_rows > Bo || keep_cols < 0 || keep_cols > Bi)
        return 1;
    for (int bo = 0; bo < n_bo; ++bo)
        for (int bi = 0; bi < n_bi; ++bi) {
            double rs[64], cs[64];
            for (int r = 0; r < Bo; ++r) {
                double s = 0.0;
                for (int c = 0; c < Bi; ++c) { double v = w[(size_t)(bo * Bo + r) * I + bi * Bi + c]; s += v * v; }
                rs[r] = s;
            }
            for (int c = 0; c < Bi; ++c) {
                double s = 0.0;
                for (int r = 0; r < Bo; ++r) { double v = w[(size_t)(bo * Bo + r) * I + bi * Bi + c]; s += v * v; }
                cs[c] = s;
            }
            uint64_t rb = 0, cbits = 0;
            for (int n = 0; n < keep_rows; ++n) {
                int best = -1;
                for (int r = 0; r < Bo; ++r)
                    if (!((rb >> r) & 1) && (best < 0 || rs[r] > rs[best])) best = r;
                rb |= (uint64_t)1 << best;
            }
            for (int n = 0; n < keep_cols; ++n) {
                int best = -1;
                for (int c = 0; c < Bi; ++c)
                    if (!((cbits >> c) & 1) && (best < 0 || cs[c] > cs[best])) best = c;
                cbits |= (uint64_t)1 << best;
            }
            row_keep[(size_t)bo * n_bi + bi] = rb;
            col_keep[(size_t)bo * n_bi + bi] = cbits;
        }
    return 0;
}
