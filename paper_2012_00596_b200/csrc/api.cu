// C-ABI entry points that validate arguments and pick a kernel; see npas.h for the contract.
#include "common.cuh"

namespace npas {

std::atomic<uint64_t> &launch_counter()
{
    static std::atomic<uint64_t> c{0};
    return c;
}

// Y[n,p,q,:] = X[n, p*stride, q*stride, :]; one thread per 16 bytes of output
__global__ void subsample_kernel(int H, int W, int P, int Q, int stride, int row16, long long total,
                                 const uint4 *__restrict__ x, uint4 *__restrict__ y)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int c = (int)(idx % row16);
    long long pix = idx / row16;
    const int q = (int)(pix % Q); pix /= Q;
    const int p = (int)(pix % P);
    const long long n = pix / P;
    y[idx] = x[((n * H + (long long)p * stride) * W + (long long)q * stride) * row16 + c];
}

__global__ void maxpool_kernel(int N, int H, int W, int C, int R, int stride, int pad, int P, int Q,
                               const uint16_t *__restrict__ x, uint16_t *__restrict__ y)
{
    // one thread per (pixel, group of 8 channels): 16-byte loads and stores
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int c8n = C / 8;
    const long long total = (long long)N * P * Q * c8n;
    if (idx >= total) return;
    const int c8 = (int)(idx % c8n);
    long long pix = idx / c8n;
    const int q = (int)(pix % Q); pix /= Q;
    const int p = (int)(pix % P);
    const int n = (int)(pix / P);
    float best[8];
    bool seen = false;
    for (int r = 0; r < R; ++r)
        for (int s = 0; s < R; ++s) {
            const int h = p * stride + r - pad, v = q * stride + s - pad;
            if (h < 0 || h >= H || v < 0 || v >= W) continue;
            const uint4 u = *reinterpret_cast<const uint4 *>(x + (((size_t)n * H + h) * W + v) * C + c8 * 8);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
                best[2 * i] = seen ? fmaxf(best[2 * i], lo) : lo;
                best[2 * i + 1] = seen ? fmaxf(best[2 * i + 1], hi) : hi;
            }
            seen = true;
        }
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t lo = seen ? __float_as_uint(best[2 * i]) >> 16 : 0u;
        const uint32_t hi = seen ? __float_as_uint(best[2 * i + 1]) & 0xFFFF0000u : 0u;
        o[i] = lo | hi;
    }
    *reinterpret_cast<uint4 *>(y + (((size_t)n * P + p) * Q + q) * C + c8 * 8) = make_uint4(o[0], o[1], o[2], o[3]);
}

}  // namespace npas

using namespace npas;

extern "C" {

const char *npas_status_string(npas_status s)
{
    switch (s) {
        case NPAS_OK: return "ok";
        case NPAS_ERR_NULL: return "null pointer argument";
        case NPAS_ERR_SHAPE: return "shape or block size not accepted";
        case NPAS_ERR_DTYPE: return "dtype combination not accepted";
        case NPAS_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case NPAS_ERR_MASK_STRUCTURE: return "mask is not of the pruning scheme's block structure";
        case NPAS_ERR_BLOB: return "packed blob header does not match the descriptor";
        case NPAS_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case NPAS_ERR_UNSUPPORTED: return "geometry not supported by the requested kernel";
        case NPAS_ERR_CUDA: return "CUDA runtime error";
        case NPAS_ERR_TIMEOUT: return "a bounded device-side wait expired";
    }
    return "unknown status";
}

uint32_t npas_abi_version(void) { return kAbiVersion; }
uint64_t npas_launch_count(void) { return launch_counter().load(); }

npas_status npas_conv2d_bp_workspace(const npas_conv_desc *d, const npas_bp_desc *bp, size_t *ws_bytes)
{
    if (!d || !ws_bytes) return NPAS_ERR_NULL;
    npas_status s = check_bp_desc(bp);
    if (s != NPAS_OK) return s;
    *ws_bytes = NPAS_WORKSPACE_BYTES;      // status words only: no kernel of this build needs more
    return NPAS_OK;
}

npas_status npas_linear_bb_workspace(const npas_linear_desc *d, const npas_bb_desc *bb, size_t *ws_bytes)
{
    if (!d || !ws_bytes) return NPAS_ERR_NULL;
    npas_status s = check_bb_desc(bb);
    if (s != NPAS_OK) return s;
    *ws_bytes = NPAS_WORKSPACE_BYTES;
    return NPAS_OK;
}

// Kernel ids (the values `path` takes to force one): 1 CUDA cores, 3 tcgen05 with both operands in
// shared memory, 5 three-channel first layer, 6 dense operand image, 7 the same on CTA pairs, 8 kept
// pairs only.  Returns 0 when the requested path does not take the geometry.
static int conv_kernel_for(const npas_conv_desc &d, const npas_bp_desc &bp)
{
    switch (d.path) {
        case 1: return 1;
        case 3: return conv_tc_supported(d, bp) ? 3 : 0;
        case 5: return conv_stem_supported(d, bp) ? 5 : 0;
        case 6: return conv_dn_supported(d, bp) ? 6 : 0;
        case 7: return conv_d2_supported(d, bp) ? 7 : 0;
        case 8: return conv_kr_supported(d, bp) ? 8 : 0;
        case 0: case 2: break;
        default: return 0;
    }
    // automatic: the first-layer kernel; kept pairs only where that was measured faster (few taps kept,
    // blocks of 16 channels or more); else the dense-image kernels; else shared-memory operands; else CUDA cores
    if (conv_stem_supported(d, bp)) return 5;
    if (conv_kr_preferred(d, bp)) return 8;
    if (conv_d2_preferred(d, bp)) return 7;
    if (conv_dn_supported(d, bp)) return 6;
    if (conv_tc_supported(d, bp)) return 3;
    return d.path == 2 ? 0 : 1;
}

// 1 CUDA cores, 3 gathered X (kept columns only), 5 masked dense image by TMA, 6 the same on CTA pairs.
static int linear_kernel_for(const npas_linear_desc &d, const npas_bb_desc &bb)
{
    switch (d.path) {
        case 1: return 1;
        case 3: return linear_tc_supported(d, bb) ? 3 : 0;
        case 5: return linear_dn_supported(d, bb) ? 5 : 0;
        case 6: return linear_d2_supported(d, bb) ? 6 : 0;
        case 0: case 2: break;
        default: return 0;
    }
    // automatic: both operands by TMA (on CTA pairs where measured faster: few rows, 256 or more input
    // features), then the gather kernel, then CUDA cores
    if (d.I >= 256 && d.M <= 16384 && linear_d2_supported(d, bb)) return 6;
    if (linear_dn_supported(d, bb)) return 5;
    if (linear_tc_supported(d, bb)) return 3;
    return d.path == 2 ? 0 : 1;
}

static npas_status check_conv_args(const npas_conv_desc *d, const npas_bp_desc *bp)
{
    if (!d) return NPAS_ERR_NULL;
    npas_status s = check_bp_desc(bp);
    if (s != NPAS_OK) return s;
    if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->stride <= 0 || d->pad < 0) return NPAS_ERR_SHAPE;
    if (d->C != bp->C || d->K != bp->K || d->R != bp->R || d->S != bp->S) return NPAS_ERR_SHAPE;
    if (d->H + 2 * d->pad < d->R || d->W + 2 * d->pad < d->S) return NPAS_ERR_SHAPE;
    if (d->x_dtype != bp->w_packed) return NPAS_ERR_DTYPE;
    if (d->y_dtype != NPAS_F32 && d->y_dtype != NPAS_BF16) return NPAS_ERR_DTYPE;
    if (d->x_dtype == NPAS_F32 && d->y_dtype != NPAS_F32) return NPAS_ERR_DTYPE;
    return NPAS_OK;
}

static npas_status check_linear_args(const npas_linear_desc *d, const npas_bb_desc *bb)
{
    if (!d) return NPAS_ERR_NULL;
    npas_status s = check_bb_desc(bb);
    if (s != NPAS_OK) return s;
    if (d->M <= 0 || d->I != bb->I || d->O != bb->O) return NPAS_ERR_SHAPE;
    if (d->x_dtype != bb->w_packed) return NPAS_ERR_DTYPE;
    if (d->y_dtype != NPAS_F32 && d->y_dtype != NPAS_BF16) return NPAS_ERR_DTYPE;
    if (d->x_dtype == NPAS_F32 && d->y_dtype != NPAS_F32) return NPAS_ERR_DTYPE;
    return NPAS_OK;
}

npas_status npas_conv2d_bp_kernel(const npas_conv_desc *d, const npas_bp_desc *bp, int32_t *kernel_id)
{
    if (!kernel_id) return NPAS_ERR_NULL;
    npas_status s = check_conv_args(d, bp);
    if (s != NPAS_OK) return s;
    *kernel_id = conv_kernel_for(*d, *bp);
    return *kernel_id ? NPAS_OK : NPAS_ERR_UNSUPPORTED;
}

npas_status npas_linear_bb_kernel(const npas_linear_desc *d, const npas_bb_desc *bb, int32_t *kernel_id)
{
    if (!kernel_id) return NPAS_ERR_NULL;
    npas_status s = check_linear_args(d, bb);
    if (s != NPAS_OK) return s;
    *kernel_id = linear_kernel_for(*d, *bb);
    return *kernel_id ? NPAS_OK : NPAS_ERR_UNSUPPORTED;
}

npas_status npas_conv2d_bp(const npas_conv_desc *d, const npas_bp_desc *bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y, void *ws,
                           size_t ws_bytes, void *stream)
{
    npas_status s = check_conv_args(d, bp);
    if (s != NPAS_OK) return s;
    if (!x || !blob || !y || !ws) return NPAS_ERR_NULL;
    if (d->has_bias && !bias) return NPAS_ERR_NULL;
    if (d->has_residual && !res) return NPAS_ERR_NULL;
    if (!aligned16(x) || !aligned16(blob) || !aligned16(y) || !aligned16(ws) || (bias && !aligned16(bias)) ||
        (res && !aligned16(res)))
        return NPAS_ERR_ALIGNMENT;
    if (ws_bytes < NPAS_WORKSPACE_BYTES) return NPAS_ERR_BUFFER_TOO_SMALL;
    if (x == y) return NPAS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float *b = d->has_bias ? bias : nullptr;
    const void *r = d->has_residual ? res : nullptr;
    uint32_t *w = static_cast<uint32_t *>(ws);
    switch (conv_kernel_for(*d, *bp)) {
        case 1: return conv_simt_launch(*d, *bp, x, blob, b, r, y, st);
        case 3: return conv_tc_launch(*d, *bp, x, blob, b, r, y, w, st);
        case 5: return conv_stem_launch(*d, *bp, x, blob, b, y, w, st);
        case 6: return conv_dn_launch(*d, *bp, x, blob, b, r, y, w, st);
        case 7: return conv_d2_launch(*d, *bp, x, blob, b, r, y, w, st);
        case 8: return conv_kr_launch(*d, *bp, x, blob, b, r, y, w, st);
    }
    return NPAS_ERR_UNSUPPORTED;
}

npas_status npas_conv2d_bp_maxpool(const npas_conv_desc *d, const npas_bp_desc *bp, int32_t pool_r, int32_t pool_stride,
                                   int32_t pool_pad, const void *x, const void *blob, const float *bias, void *y_pooled,
                                   void *ws, size_t ws_bytes, void *stream)
{
    npas_status s = check_conv_args(d, bp);
    if (s != NPAS_OK) return s;
    if (!x || !blob || !y_pooled || !ws) return NPAS_ERR_NULL;
    if (d->has_bias && !bias) return NPAS_ERR_NULL;
    if (pool_r <= 0 || pool_stride <= 0 || pool_pad < 0 || pool_pad >= pool_r) return NPAS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(blob) || !aligned16(y_pooled) || !aligned16(ws) || (bias && !aligned16(bias)))
        return NPAS_ERR_ALIGNMENT;
    if (ws_bytes < NPAS_WORKSPACE_BYTES) return NPAS_ERR_BUFFER_TOO_SMALL;
    if (x == y_pooled) return NPAS_ERR_UNSUPPORTED;
    // fused where a kernel has the pooled epilogue: the three-channel first layer with ReLU, bf16 output and
    // the 3x3 / stride-2 / pad-1 window; everything else is left to the two separate calls
    if (d->has_residual || pool_r != 3 || pool_stride != 2 || pool_pad != 1 || (d->path != 0 && d->path != 2 && d->path != 5) ||
        !conv_stem_pool_supported(*d, *bp))
        return NPAS_ERR_UNSUPPORTED;
    return conv_stem_launch(*d, *bp, x, blob, d->has_bias ? bias : nullptr, y_pooled, static_cast<uint32_t *>(ws),
                            static_cast<cudaStream_t>(stream), true);
}

npas_status npas_linear_bb(const npas_linear_desc *d, const npas_bb_desc *bb, const void *x,
                           const void *blob, const float *bias, const void *residual, void *y, void *ws,
                           size_t ws_bytes, void *stream)
{
    npas_status s = check_linear_args(d, bb);
    if (s != NPAS_OK) return s;
    if (!x || !blob || !y || !ws) return NPAS_ERR_NULL;
    if (d->has_bias && !bias) return NPAS_ERR_NULL;
    if (d->has_residual && !residual) return NPAS_ERR_NULL;
    if (!aligned16(x) || !aligned16(blob) || !aligned16(y) || !aligned16(ws) || (bias && !aligned16(bias)))
        return NPAS_ERR_ALIGNMENT;
    if (ws_bytes < NPAS_WORKSPACE_BYTES) return NPAS_ERR_BUFFER_TOO_SMALL;
    if (x == y) return NPAS_ERR_UNSUPPORTED;
    const void *r = d->has_residual ? residual : nullptr;
    if (r && (!aligned16(r) || r == y)) return r == y ? NPAS_ERR_UNSUPPORTED : NPAS_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float *b = d->has_bias ? bias : nullptr;
    uint32_t *w = static_cast<uint32_t *>(ws);
    switch (linear_kernel_for(*d, *bb)) {
        case 1: return linear_simt_launch(*d, *bb, x, blob, b, r, y, st);
        case 3: return linear_tc_launch(*d, *bb, x, blob, b, r, y, w, st);
        case 5: return linear_dn_launch(*d, *bb, x, blob, b, r, y, w, st);
        case 6: return linear_d2_launch(*d, *bb, x, blob, b, r, y, w, st);
    }
    return NPAS_ERR_UNSUPPORTED;
}

}  // extern "C"

// ---- auto-tuning: measure every kernel / tile shape that takes the layer, keep the fastest --------
namespace {

struct Timer {
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    bool ok = false;
    Timer() { ok = cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess; }
    ~Timer() { if (e0) cudaEventDestroy(e0); if (e1) cudaEventDestroy(e1); }
};

// Times `reps` launches of one candidate after a warm-up launch; < 0 when it declined or failed.
template <typename F>
float time_candidate(F launch, int reps, void *ws, cudaStream_t st, Timer &t)
{
    if (launch() != NPAS_OK) return -1.f;
    int32_t detail = 0;
    if (npas_check_device_status(ws, st, &detail) != NPAS_OK) return -1.f;
    cudaEventRecord(t.e0, st);
    for (int i = 0; i < reps; ++i)
        if (launch() != NPAS_OK) return -1.f;
    cudaEventRecord(t.e1, st);
    if (cudaEventSynchronize(t.e1) != cudaSuccess) return -1.f;
    if (npas_check_device_status(ws, st, &detail) != NPAS_OK) return -1.f;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, t.e0, t.e1) != cudaSuccess) return -1.f;
    return ms * 1000.f / reps;
}

}  // namespace

extern "C" {

npas_status npas_tune_conv2d_bp(const npas_conv_desc *d, const npas_bp_desc *bp, const void *x, const void *blob,
                                const float *bias, const void *res, void *y, void *ws, size_t ws_bytes,
                                int32_t reps, int32_t *path_out, int32_t *variant_out, float *us_out, void *stream)
{
    if (!path_out || !variant_out) return NPAS_ERR_NULL;
    npas_status s = check_conv_args(d, bp);
    if (s != NPAS_OK) return s;
    if (reps < 1 || reps > 10000) return NPAS_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Timer t;
    if (!t.ok) return NPAS_ERR_CUDA;
    struct Cand { int path, variant; };
    // (every item shape of the pair kernel: filters per item 64, 128 or 256, position tiles per CTA 1 or 2)
    const Cand cands[] = {{5, 0}, {8, 0}, {7, 64 | (1 << 16)}, {7, 64 | (2 << 16)}, {7, 128 | (1 << 16)}, {7, 128 | (2 << 16)},
                          {7, 256 | (1 << 16)}, {7, 256 | (2 << 16)}, {6, 0}, {3, 0}, {1, 0}};
    float best = -1.f;
    bool tensor_core_found = false;
    for (const Cand &c : cands) {
        if (c.path == 1 && tensor_core_found) continue;          // CUDA cores only when nothing else takes the layer
        npas_conv_desc q = *d;
        q.path = c.path; q.variant = c.variant;
        if (!conv_kernel_for(q, *bp)) continue;
        const float us = time_candidate([&] { return npas_conv2d_bp(&q, bp, x, blob, bias, res, y, ws, ws_bytes, stream); },
                                        reps, ws, st, t);
        if (us < 0.f) continue;
        tensor_core_found = tensor_core_found || c.path != 1;
        if (best < 0.f || us < best) { best = us; *path_out = c.path; *variant_out = c.variant; }
    }
    if (best < 0.f) return NPAS_ERR_UNSUPPORTED;
    if (us_out) *us_out = best;
    return NPAS_OK;
}

npas_status npas_tune_linear_bb(const npas_linear_desc *d, const npas_bb_desc *bb, const void *x, const void *blob,
                                const float *bias, const void *res, void *y, void *ws, size_t ws_bytes,
                                int32_t reps, int32_t *path_out, int32_t *variant_out, float *us_out, void *stream)
{
    if (!path_out || !variant_out) return NPAS_ERR_NULL;
    npas_status s = check_linear_args(d, bb);
    if (s != NPAS_OK) return s;
    if (reps < 1 || reps > 10000) return NPAS_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Timer t;
    if (!t.ok) return NPAS_ERR_CUDA;
    struct Cand { int path, variant; };
    const Cand cands[] = {{6, 256}, {6, 128}, {5, 256}, {5, 128}, {5, 64}, {5, 32}, {5, 16}, {3, 0}, {1, 0}};
    float best = -1.f;
    bool tensor_core_found = false;
    for (const Cand &c : cands) {
        if (c.path == 1 && tensor_core_found) continue;
        npas_linear_desc q = *d;
        q.path = c.path; q.variant = c.variant;
        if (!linear_kernel_for(q, *bb)) continue;
        const float us = time_candidate([&] { return npas_linear_bb(&q, bb, x, blob, bias, res, y, ws, ws_bytes, stream); },
                                        reps, ws, st, t);
        if (us < 0.f) continue;
        tensor_core_found = tensor_core_found || c.path != 1;
        if (best < 0.f || us < best) { best = us; *path_out = c.path; *variant_out = c.variant; }
    }
    if (best < 0.f) return NPAS_ERR_UNSUPPORTED;
    if (us_out) *us_out = best;
    return NPAS_OK;
}

npas_status npas_blob_check(const npas_bp_desc *bp, const npas_bb_desc *bb, const void *blob,
                            size_t blob_bytes, void *stream)
{
    if (!blob || (!bp && !bb) || (bp && bb)) return NPAS_ERR_NULL;
    if (blob_bytes < 128) return NPAS_ERR_BUFFER_TOO_SMALL;
    uint32_t h[32];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(h, blob, 128, cudaMemcpyDeviceToHost, st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (bp) {
        npas_status s = check_bp_desc(bp);
        if (s != NPAS_OK) return s;
        if (h[BP_MAGIC] != kMagicBP || h[BP_VERSION] != kVersion) return NPAS_ERR_BLOB;
        const BpLayout L = bp_layout(*bp, h[BP_NPAIRS]);
        const uint32_t want[] = {(uint32_t)bp->w_packed, (uint32_t)bp->K, (uint32_t)bp->C, (uint32_t)bp->R,
                                 (uint32_t)bp->S, (uint32_t)bp->Mb, (uint32_t)bp->Nb, L.nFB, L.nCB, h[BP_NPAIRS],
                                 L.off_blk, L.off_pairs, L.off_values, L.total, L.G, L.off_image, L.off_tapu, L.GI,
                                 L.off_ktoff, L.off_kt, L.GS, L.nKt};
        for (int i = 0; i < 22; ++i)
            if (h[BP_DTYPE + i] != want[i]) return NPAS_ERR_BLOB;
        if (h[BP_NPAIRS] > L.nFB * L.nCB * (uint32_t)(bp->R * bp->S)) return NPAS_ERR_BLOB;
        return L.total <= blob_bytes ? NPAS_OK : NPAS_ERR_BUFFER_TOO_SMALL;
    }
    npas_status s = check_bb_desc(bb);
    if (s != NPAS_OK) return s;
    if (h[BB_MAGIC] != kMagicBB || h[BB_VERSION] != kVersionBB) return NPAS_ERR_BLOB;
    const BbLayout L = bb_layout(*bb);
    const uint32_t off_tiles = L.off_values + round_up(h[BB_NVALS] * L.es, 128);
    if (h[BB_KP] < 16 || h[BB_KP] % 16 || h[BB_KP] > 64 || h[BB_OFF_TILES] != off_tiles) return NPAS_ERR_BLOB;
    const uint32_t total = off_tiles + round_up(L.nBlk * h[BB_KP] * (uint32_t)bb->Bo * L.es, 128);
    const uint32_t want[] = {(uint32_t)bb->w_packed, (uint32_t)bb->O, (uint32_t)bb->I, (uint32_t)bb->Bo,
                             (uint32_t)bb->Bi, L.nBo, L.nBi, h[BB_NVALS], L.off_cnt, L.off_rows, L.off_cols,
                             L.off_voff, L.off_values, total};
    for (int i = 0; i < 14; ++i)
        if (h[BB_DTYPE + i] != want[i]) return NPAS_ERR_BLOB;
    if (h[BB_OFF_DENSE] != L.off_dense) return NPAS_ERR_BLOB;
    return total <= blob_bytes ? NPAS_OK : NPAS_ERR_BUFFER_TOO_SMALL;
}

npas_status npas_check_device_status(void *ws, void *stream, int32_t *detail)
{
    if (!ws) return NPAS_ERR_NULL;
    uint32_t w[2] = {0, 0};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(w, ws, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (detail) *detail = (int32_t)w[WS_DETAIL];
    if (w[WS_STATUS] == 0) return NPAS_OK;
    if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NPAS_ERR_CUDA;
    return w[WS_STATUS] == (uint32_t)NPAS_ERR_BLOB ? NPAS_ERR_BLOB : NPAS_ERR_TIMEOUT;
}

npas_status npas_maxpool2d(int32_t N, int32_t H, int32_t W, int32_t C, int32_t R, int32_t stride,
                           int32_t pad, const void *x, void *y, void *stream)
{
    if (!x || !y) return NPAS_ERR_NULL;
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || C % 8 || R <= 0 || stride <= 0 || pad < 0 || pad >= R)
        return NPAS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return NPAS_ERR_ALIGNMENT;
    const int P = (H + 2 * pad - R) / stride + 1, Q = (W + 2 * pad - R) / stride + 1;
    const long long total = (long long)N * P * Q * (C / 8);
    maxpool_kernel<<<(unsigned)((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        N, H, W, C, R, stride, pad, P, Q, static_cast<const uint16_t *>(x), static_cast<uint16_t *>(y));
    count_launch();
    return launch_status();
}

npas_status npas_subsample2d(int32_t N, int32_t H, int32_t W, int32_t C, int32_t stride,
                             int32_t elem_bytes, const void *x, void *y, void *stream)
{
    if (!x || !y) return NPAS_ERR_NULL;
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || stride <= 0) return NPAS_ERR_SHAPE;
    if (elem_bytes != 2 && elem_bytes != 4) return NPAS_ERR_DTYPE;
    if (((long long)C * elem_bytes) % 16) return NPAS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return NPAS_ERR_ALIGNMENT;
    if (x == y) return NPAS_ERR_UNSUPPORTED;
    const int P = (H - 1) / stride + 1, Q = (W - 1) / stride + 1, row16 = C * elem_bytes / 16;
    const long long total = (long long)N * P * Q * row16;
    subsample_kernel<<<(unsigned)((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        H, W, P, Q, stride, row16, total, static_cast<const uint4 *>(x), static_cast<uint4 *>(y));
    count_launch();
    return launch_status();
}

}  // extern "C"
