// Block-based pruned GEMM on CUDA cores: the float32 path (float64 accumulation, one rounding at
// the store) and the fall-back for geometries the tcgen05 kernel does not take (bf16 inputs,
// float32 accumulation).  One CTA owns 128 rows of X and one row of weight
// blocks; per column block it stages the X tile in shared memory, then every thread (one row of
// X) walks the block's kept columns and kept rows, accumulating into a transposed shared tile so
// that the warp's accesses fall on distinct banks.
#include "common.cuh"

namespace npas {

constexpr int kLinRows = 128;

template <typename T> __device__ inline float lin_load(const T *p);
template <> __device__ inline float lin_load<float>(const float *p) { return *p; }
template <> __device__ inline float lin_load<uint16_t>(const uint16_t *p) { return bf16_bits_to_f32(*p); }
template <typename T> __device__ inline void lin_store(T *p, float v);
template <> __device__ inline void lin_store<float>(float *p, float v) { *p = v; }
template <> __device__ inline void lin_store<uint16_t>(uint16_t *p, float v) { *p = f32_bits_to_bf16(__float_as_uint(v)); }

template <typename T> struct LinAcc { typedef float type; };
template <> struct LinAcc<float> { typedef double type; };

template <typename TX, typename TY>
__global__ void __launch_bounds__(kLinRows)
linear_bb_simt_kernel(npas_linear_desc d, int Bo, int Bi, BbLayout L, const TX *__restrict__ x,
                      const uint8_t *__restrict__ blob, const float *__restrict__ bias, const TY *__restrict__ res,
                      TY *__restrict__ y)
{
    typedef typename LinAcc<TX>::type TA;
    extern __shared__ double sm_raw[];
    TA *acc_s = reinterpret_cast<TA *>(sm_raw);                        // [Bo][128]
    float *x_s = reinterpret_cast<float *>(acc_s + Bo * kLinRows);    // [128][Bi + 1]
    const int t = threadIdx.x, bo = blockIdx.y;
    const int m0 = blockIdx.x * kLinRows, m = m0 + t;
    const int rows_here = min(kLinRows, d.M - m0);
    const uint32_t *voff = reinterpret_cast<const uint32_t *>(blob + L.off_voff);
    const TX *vals = reinterpret_cast<const TX *>(blob + L.off_values);

    for (int r = 0; r < Bo; ++r) acc_s[r * kLinRows + t] = 0;
    for (uint32_t bi = 0; bi < L.nBi; ++bi) {
        const uint32_t b = bo * L.nBi + bi;
        const int nr = blob[L.off_cnt + 2 * b], nc = blob[L.off_cnt + 2 * b + 1];
        __syncthreads();
        for (int e = t; e < rows_here * Bi; e += kLinRows) {
            const int rr = e / Bi, cc = e % Bi;
            x_s[rr * (Bi + 1) + cc] = lin_load(x + (size_t)(m0 + rr) * d.I + bi * Bi + cc);
        }
        __syncthreads();
        if (m >= d.M || nr == 0 || nc == 0) continue;
        const uint8_t *rows = blob + L.off_rows + (size_t)b * Bo, *cols = blob + L.off_cols + (size_t)b * Bi;
        const TX *v = vals + voff[b];
        for (int r = 0; r < nr; ++r) {
            TA a = 0;
            for (int c = 0; c < nc; ++c) a = fma((TA)x_s[t * (Bi + 1) + cols[c]], (TA)lin_load(v + r * nc + c), a);
            acc_s[rows[r] * kLinRows + t] += a;
        }
    }
    if (m >= d.M) return;
    for (int r = 0; r < Bo; ++r) {
        TA v = acc_s[r * kLinRows + t];
        if (bias) v += (TA)bias[bo * Bo + r];
        if (res) v += (TA)lin_load(res + (size_t)m * d.O + bo * Bo + r);
        if (d.relu) v = v > 0 ? v : 0;
        lin_store(y + (size_t)m * d.O + bo * Bo + r, (float)v);
    }
}

npas_status linear_simt_launch(const npas_linear_desc &d, const npas_bb_desc &bb, const void *x,
                               const void *blob, const float *bias, const void *res, void *y, cudaStream_t st)
{
    const BbLayout L = bb_layout(bb);
    const dim3 grid((d.M + kLinRows - 1) / kLinRows, L.nBo);
    if (grid.y > 65535) return NPAS_ERR_UNSUPPORTED;
    const size_t smem = (d.x_dtype == NPAS_F32 ? sizeof(double) : sizeof(float)) * bb.Bo * kLinRows + sizeof(float) * kLinRows * (bb.Bi + 1);
    const uint8_t *b8 = static_cast<const uint8_t *>(blob);
    cudaError_t e = cudaSuccess;
    if (d.x_dtype == NPAS_F32 && d.y_dtype == NPAS_F32) {
        auto k = linear_bb_simt_kernel<float, float>;
        e = allow_dynamic_smem(reinterpret_cast<const void *>(k), (int)smem) == NPAS_OK ? cudaSuccess : cudaErrorUnknown;
        k<<<grid, kLinRows, smem, st>>>(d, bb.Bo, bb.Bi, L, static_cast<const float *>(x), b8, bias, static_cast<const float *>(res), static_cast<float *>(y));
    } else if (d.x_dtype == NPAS_BF16 && d.y_dtype == NPAS_BF16) {
        auto k = linear_bb_simt_kernel<uint16_t, uint16_t>;
        e = allow_dynamic_smem(reinterpret_cast<const void *>(k), (int)smem) == NPAS_OK ? cudaSuccess : cudaErrorUnknown;
        k<<<grid, kLinRows, smem, st>>>(d, bb.Bo, bb.Bi, L, static_cast<const uint16_t *>(x), b8, bias, static_cast<const uint16_t *>(res), static_cast<uint16_t *>(y));
    } else if (d.x_dtype == NPAS_BF16 && d.y_dtype == NPAS_F32) {
        auto k = linear_bb_simt_kernel<uint16_t, float>;
        e = allow_dynamic_smem(reinterpret_cast<const void *>(k), (int)smem) == NPAS_OK ? cudaSuccess : cudaErrorUnknown;
        k<<<grid, kLinRows, smem, st>>>(d, bb.Bo, bb.Bi, L, static_cast<const uint16_t *>(x), b8, bias, static_cast<const float *>(res), static_cast<float *>(y));
    } else {
        return NPAS_ERR_DTYPE;
    }
    if (e != cudaSuccess) return NPAS_ERR_CUDA;
    count_launch();
    return launch_status();
}

}  // namespace npas
