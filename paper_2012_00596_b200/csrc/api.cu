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

npas_status npas_conv2d_bp(const npas_conv_desc *d, const npas_bp_desc *bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y, void *ws,
                           size_t ws_bytes, void *stream)
{
    if (!d) return NPAS_ERR_NULL;
    npas_status s = check_bp_desc(bp);
    if (s != NPAS_OK) return s;
    if (!x || !blob || !y || !ws) return NPAS_ERR_NULL;
    if (d->has_bias && !bias) return NPAS_ERR_NULL;
    if (d->has_residual && !res) return NPAS_ERR_NULL;
    if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->stride <= 0 || d->pad < 0) return NPAS_ERR_SHAPE;
    if (d->C != bp->C || d->K != bp->K || d->R != bp->R || d->S != bp->S) return NPAS_ERR_SHAPE;
    if (d->H + 2 * d->pad < d->R || d->W + 2 * d->pad < d->S) return NPAS_ERR_SHAPE;
    if (d->x_dtype != bp->w_packed) return NPAS_ERR_DTYPE;
    if (d->y_dtype != NPAS_F32 && d->y_dtype != NPAS_BF16) return NPAS_ERR_DTYPE;
    if (d->x_dtype == NPAS_F32 && d->y_dtype != NPAS_F32) return NPAS_ERR_DTYPE;
    if (!aligned16(x) || !aligned16(blob) || !aligned16(y) || !aligned16(ws) || (bias && !aligned16(bias)) ||
        (res && !aligned16(res)))
        return NPAS_ERR_ALIGNMENT;
    if (ws_bytes < NPAS_WORKSPACE_BYTES) return NPAS_ERR_BUFFER_TOO_SMALL;
    if (x == y) return NPAS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float *b = d->has_bias ? bias : nullptr;
    const void *r = d->has_residual ? res : nullptr;
    if (d->path < 0 || d->path > 8) return NPAS_ERR_UNSUPPORTED;
    if (d->path == 8)
        return conv_kr_supported(*d, *bp) ? conv_kr_launch(*d, *bp, x, blob, b, r, y, static_cast<uint32_t *>(ws), st)
                                          : NPAS_ERR_UNSUPPORTED;
    if ((d->path == 0 || d->path == 2 || d->path == 5) && conv_stem_supported(*d, *bp))
        return conv_stem_launch(*d, *bp, x, blob, b, y, static_cast<uint32_t *>(ws), st);
    if (d->path == 5) return NPAS_ERR_UNSUPPORTED;
    if (d->path == 7)
        return conv_d2_supported(*d, *bp) ? conv_d2_launch(*d, *bp, x, blob, b, r, y, static_cast<uint32_t *>(ws), st)
                                          : NPAS_ERR_UNSUPPORTED;
    // automatic choice between the two dense-image kernels
    if ((d->path == 0 || d->path == 2) && conv_d2_preferred(*d, *bp))
        return conv_d2_launch(*d, *bp, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if ((d->path == 0 || d->path == 2 || d->path == 6) && conv_dn_supported(*d, *bp))
        return conv_dn_launch(*d, *bp, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if (d->path == 6) return NPAS_ERR_UNSUPPORTED;
    const bool ts_ok = d->path != 1 && d->path != 3 && conv_ts_supported(*d, *bp);
    const bool ss_ok = d->path != 1 && d->path != 4 && conv_tc_supported(*d, *bp);
    if (ts_ok) return conv_ts_launch(*d, *bp, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if (ss_ok) return conv_tc_launch(*d, *bp, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if (d->path >= 2) return NPAS_ERR_UNSUPPORTED;
    return conv_simt_launch(*d, *bp, x, blob, b, r, y, st);
}

npas_status npas_linear_bb(const npas_linear_desc *d, const npas_bb_desc *bb, const void *x,
                           const void *blob, const float *bias, const void *residual, void *y, void *ws,
                           size_t ws_bytes, void *stream)
{
    if (!d) return NPAS_ERR_NULL;
    npas_status s = check_bb_desc(bb);
    if (s != NPAS_OK) return s;
    if (!x || !blob || !y || !ws) return NPAS_ERR_NULL;
    if (d->has_bias && !bias) return NPAS_ERR_NULL;
    if (d->has_residual && !residual) return NPAS_ERR_NULL;
    if (d->M <= 0 || d->I != bb->I || d->O != bb->O) return NPAS_ERR_SHAPE;
    if (d->x_dtype != bb->w_packed) return NPAS_ERR_DTYPE;
    if (d->y_dtype != NPAS_F32 && d->y_dtype != NPAS_BF16) return NPAS_ERR_DTYPE;
    if (d->x_dtype == NPAS_F32 && d->y_dtype != NPAS_F32) return NPAS_ERR_DTYPE;
    if (!aligned16(x) || !aligned16(blob) || !aligned16(y) || !aligned16(ws) || (bias && !aligned16(bias)))
        return NPAS_ERR_ALIGNMENT;
    if (ws_bytes < NPAS_WORKSPACE_BYTES) return NPAS_ERR_BUFFER_TOO_SMALL;
    if (x == y) return NPAS_ERR_UNSUPPORTED;
    const void *r = d->has_residual ? residual : nullptr;
    if (r && (!aligned16(r) || r == y)) return r == y ? NPAS_ERR_UNSUPPORTED : NPAS_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float *b = d->has_bias ? bias : nullptr;
    if (d->path < 0 || d->path > 6) return NPAS_ERR_UNSUPPORTED;
    if (d->path == 6)
        return linear_d2_supported(*d, *bb) ? linear_d2_launch(*d, *bb, x, blob, b, r, y, static_cast<uint32_t *>(ws), st)
                                            : NPAS_ERR_UNSUPPORTED;
    if (d->path == 1) return linear_simt_launch(*d, *bb, x, blob, b, r, y, st);
    // automatic choice: the kernels that stream both operands by TMA (on CTA pairs where measured faster:
    // few rows, 256 or more input features), then the gather kernel
    if ((d->path == 0 || d->path == 2) && d->I >= 256 && d->M <= 16384 && linear_d2_supported(*d, *bb))
        return linear_d2_launch(*d, *bb, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if ((d->path == 0 || d->path == 2 || d->path == 5) && linear_dn_supported(*d, *bb))
        return linear_dn_launch(*d, *bb, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if (d->path == 5) return NPAS_ERR_UNSUPPORTED;
    const bool tc_ok = d->path != 4 && linear_tc_supported(*d, *bb);
    const bool dx_ok = d->path != 3 && linear_dx_supported(*d, *bb);
    if (tc_ok) return linear_tc_launch(*d, *bb, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if (dx_ok) return linear_dx_launch(*d, *bb, x, blob, b, r, y, static_cast<uint32_t *>(ws), st);
    if (d->path >= 2) return NPAS_ERR_UNSUPPORTED;
    return linear_simt_launch(*d, *bb, x, blob, b, r, y, st);
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
