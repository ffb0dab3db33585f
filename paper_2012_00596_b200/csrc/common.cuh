// Shared host/device helpers of the library: blob header views, bf16 conversion, launch
// accounting and argument checks.  Nothing here is visible through the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <atomic>

#include "npas.h"

namespace npas {

constexpr uint32_t kMagicBP = 0x5042504Eu;  // 'NPBP'
constexpr uint32_t kMagicBB = 0x4242504Eu;  // 'NPBB'
constexpr uint32_t kVersion = 4;
constexpr uint32_t kAbiVersion = 1;

// Field indices of the 32-word blob headers (layout documented in npas.h).
enum BpHdr { BP_MAGIC, BP_VERSION, BP_DTYPE, BP_K, BP_C, BP_R, BP_S, BP_MB, BP_NB, BP_NFB, BP_NCB,
             BP_NPAIRS, BP_OFF_BLK, BP_OFF_PAIRS, BP_OFF_VALUES, BP_TOTAL, BP_G, BP_OFF_IMAGE, BP_OFF_TAPU, BP_GI,
             BP_OFF_KTOFF, BP_OFF_KT, BP_GS, BP_NKT };
enum BbHdr { BB_MAGIC, BB_VERSION, BB_DTYPE, BB_O, BB_I, BB_BO, BB_BI, BB_NBO, BB_NBI, BB_NVALS,
             BB_OFF_CNT, BB_OFF_ROWS, BB_OFF_COLS, BB_OFF_VOFF, BB_OFF_VALUES, BB_TOTAL, BB_KP, BB_OFF_TILES,
             BB_OFF_DENSE };
constexpr uint32_t kVersionBB = 3;

// Section offsets of a block-punched blob, computed on the host from the descriptor and nPairs.
struct BpLayout {
    uint32_t nFB, nCB, nPairs, G, es;
    uint32_t off_blk, off_pairs, off_values, total;
    uint32_t off_image, off_tapu, GI;          // dense operand image (bf16, C % 16 == 0 only; else 0)
    uint32_t off_ktoff, off_kt, GS, nKt, nGrp;  // kept 16-channel tiles by (chunk, filter group, tap); else 0
};
struct BbLayout {
    uint32_t nBo, nBi, nBlk, es;
    uint32_t off_cnt, off_rows, off_cols, off_voff, off_dense, off_values;  // total needs nVals
};

__host__ __device__ inline uint32_t round_up(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }
__host__ __device__ inline uint32_t dtype_size(int dt) { return dt == NPAS_F32 ? 4u : 2u; }

__host__ __device__ inline BpLayout bp_layout(const npas_bp_desc &d, uint32_t nPairs)
{
    BpLayout L;
    L.nFB = d.K / d.Mb; L.nCB = d.C / d.Nb; L.nPairs = nPairs;
    L.G = (d.Nb % 8 == 0) ? 8 : d.Nb;
    L.es = dtype_size(d.w_packed);
    L.off_blk = 128;
    L.off_pairs = round_up(L.off_blk + 4 * (L.nFB * L.nCB + 1), 128);
    L.off_values = round_up(L.off_pairs + 4 * nPairs, 128);
    L.total = L.off_values + round_up(nPairs * d.Mb * d.Nb * L.es, 128);
    // filters per group of the operand image: the largest power of two <= 128 that divides K
    L.GI = 128;
    while (d.K % L.GI) L.GI >>= 1;
    L.off_image = 0; L.off_tapu = 0;
    if (d.w_packed == NPAS_BF16 && d.C % 16 == 0) {
        L.off_image = round_up(L.total, 2048);     // on a multiple of a 128-filter row, so that tensor maps over the blob can count in rows
        L.off_tapu = L.off_image + round_up((uint32_t)d.K * d.R * d.S * d.C * 2u, 128);
        L.total = L.off_tapu + round_up((uint32_t)(d.K / L.GI) * (d.C / 16) * 4u, 128);
    }
    // kept weights as tiles of Mb filters x 16 channels, grouped for the kept-only tensor-core kernel
    uint32_t fgw = 256;
    while (d.K % fgw) fgw >>= 1;
    L.off_ktoff = 0; L.off_kt = 0; L.GS = 0; L.nKt = 0; L.nGrp = 0;
    if (d.w_packed == NPAS_BF16 && d.Mb % 16 == 0 && d.Nb % 16 == 0 && d.R * d.S <= 16 && fgw % d.Mb == 0) {
        L.GS = fgw / d.Mb;
        L.nGrp = d.K / fgw;
        L.nKt = nPairs * (d.Nb / 16);
        L.off_ktoff = L.total;
        L.off_kt = L.off_ktoff + round_up(4u * ((uint32_t)(d.C / 16) * L.nGrp + 1u), 128);
        L.total = L.off_kt + round_up(L.nKt * (uint32_t)d.Mb * 32u, 128);
    }
    return L;
}

inline BbLayout bb_layout(const npas_bb_desc &d)
{
    BbLayout L;
    L.nBo = d.O / d.Bo; L.nBi = d.I / d.Bi; L.nBlk = L.nBo * L.nBi;
    L.es = dtype_size(d.w_packed);
    L.off_cnt = 128;
    L.off_rows = round_up(L.off_cnt + 2 * L.nBlk, 128);
    L.off_cols = round_up(L.off_rows + d.Bo * L.nBlk, 128);
    L.off_voff = round_up(L.off_cols + d.Bi * L.nBlk, 128);
    L.off_dense = round_up(L.off_voff + 4 * (L.nBlk + 1), 128);
    L.off_values = L.off_dense + round_up((uint32_t)d.O * d.I * L.es, 128);
    return L;
}

// float32 -> bf16 bits, round to nearest even on the bit pattern; NaN keeps sign / upper payload.
__host__ __device__ inline uint16_t f32_bits_to_bf16(uint32_t b)
{
    if ((b & 0x7F800000u) == 0x7F800000u && (b & 0x007FFFFFu) != 0u)
        return (uint16_t)((b >> 16) | 0x0040u);
    return (uint16_t)((b + 0x7FFFu + ((b >> 16) & 1u)) >> 16);
}
__device__ inline float bf16_bits_to_f32(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline npas_status check_bp_desc(const npas_bp_desc *d)
{
    if (!d) return NPAS_ERR_NULL;
    if (d->K <= 0 || d->C <= 0 || d->R <= 0 || d->S <= 0 || d->Mb <= 0 || d->Nb <= 0) return NPAS_ERR_SHAPE;
    if (d->K % d->Mb || d->C % d->Nb || d->R * d->S > 64) return NPAS_ERR_SHAPE;
    if (d->C >= 65536 || d->Mb > 4096 || d->Nb > 4096 || d->max_taps < 0) return NPAS_ERR_SHAPE;
    if ((uint64_t)d->K * d->R * d->S * (uint64_t)d->C > (1ull << 28)) return NPAS_ERR_SHAPE;   // blob offsets are 32-bit
    if ((d->w_in != NPAS_F32 && d->w_in != NPAS_BF16) || (d->w_packed != NPAS_F32 && d->w_packed != NPAS_BF16))
        return NPAS_ERR_DTYPE;
    if (d->w_in == NPAS_BF16 && d->w_packed == NPAS_F32) return NPAS_ERR_DTYPE;
    return NPAS_OK;
}

inline npas_status check_bb_desc(const npas_bb_desc *d)
{
    if (!d) return NPAS_ERR_NULL;
    if (d->O <= 0 || d->I <= 0 || d->Bo <= 0 || d->Bi <= 0) return NPAS_ERR_SHAPE;
    if (d->Bo > 64 || d->Bi > 64 || d->O % d->Bo || d->I % d->Bi || d->max_cols < 0) return NPAS_ERR_SHAPE;
    if ((uint64_t)d->O * (uint64_t)d->I > (1ull << 27)) return NPAS_ERR_SHAPE;      // blob offsets are 32-bit
    if ((d->w_in != NPAS_F32 && d->w_in != NPAS_BF16) || (d->w_packed != NPAS_F32 && d->w_packed != NPAS_BF16))
        return NPAS_ERR_DTYPE;
    if (d->w_in == NPAS_BF16 && d->w_packed == NPAS_F32) return NPAS_ERR_DTYPE;
    return NPAS_OK;
}

// Process-wide count of kernels launched by this library.
std::atomic<uint64_t> &launch_counter();
inline void count_launch(uint64_t n = 1) { launch_counter().fetch_add(n, std::memory_order_relaxed); }

inline npas_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? NPAS_OK : NPAS_ERR_CUDA;
}

// Multiprocessors of the current device.
int sm_count();
npas_status allow_dynamic_smem(const void *kernel, int bytes);     // once per (kernel, device)

// Words of the caller's workspace.
enum WsWord { WS_STATUS = 0, WS_DETAIL = 1 };

// ---- kernels implemented in the other translation units (host launchers) ------------------------
npas_status conv_simt_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                             const void *blob, const float *bias, const void *res, void *y,
                             cudaStream_t st);
bool conv_tc_supported(const npas_conv_desc &d, const npas_bp_desc &bp);
npas_status conv_tc_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st);
bool conv_stem_supported(const npas_conv_desc &d, const npas_bp_desc &bp);
bool conv_stem_pool_supported(const npas_conv_desc &d, const npas_bp_desc &bp);
npas_status conv_stem_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                             const void *blob, const float *bias, void *y, uint32_t *ws, cudaStream_t st,
                             bool pool = false);
bool conv_dn_supported(const npas_conv_desc &d, const npas_bp_desc &bp);
npas_status conv_dn_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st);
bool conv_d2_supported(const npas_conv_desc &d, const npas_bp_desc &bp);
bool conv_d2_preferred(const npas_conv_desc &d, const npas_bp_desc &bp);
npas_status conv_d2_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st);
bool conv_kr_supported(const npas_conv_desc &d, const npas_bp_desc &bp);
bool conv_kr_preferred(const npas_conv_desc &d, const npas_bp_desc &bp);
npas_status conv_kr_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                           const void *blob, const float *bias, const void *res, void *y,
                           uint32_t *ws, cudaStream_t st);
npas_status linear_simt_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                               const void *blob, const float *bias, const void *res, void *y, cudaStream_t st);
bool linear_dn_supported(const npas_linear_desc &d, const npas_bb_desc &bb);
npas_status linear_dn_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                             const void *blob, const float *bias, const void *res, void *y, uint32_t *ws,
                             cudaStream_t st);
bool linear_d2_supported(const npas_linear_desc &d, const npas_bb_desc &bb);
npas_status linear_d2_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                             const void *blob, const float *bias, const void *res, void *y, uint32_t *ws,
                             cudaStream_t st);
bool linear_tc_supported(const npas_linear_desc &d, const npas_bb_desc &bb);
npas_status linear_tc_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                             const void *blob, const float *bias, const void *res, void *y, uint32_t *ws,
                             cudaStream_t st);

}  // namespace npas
