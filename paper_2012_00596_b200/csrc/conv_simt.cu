// Block-punched convolution on CUDA cores.  This is the kernel for the float32 path (TF32
// tensor-core products are too coarse for a 1e-5 tolerance) and for geometries outside the
// tcgen05 kernel's envelope (tiny blocks, strides, wide images).  float32 inputs accumulate in
// float64 (products of two float32 are exact there), so the only rounding is the final store;
// bf16 inputs accumulate in float32 like the tensor-core path.  One CTA owns 128 consecutive
// output pixels and up to 8 filters of one filter block; it walks that block's kept (channel
// block, tap) pairs, staging the packed weights of a run of pairs in shared memory as fp32 so
// that every thread reads them as broadcast 16-byte words.
#include "common.cuh"

namespace npas {

constexpr int kSimtPixels = 128;   // threads per CTA = output pixels per CTA
constexpr int kSimtFilters = 8;    // filters per thread
constexpr int kSimtWFloats = 4096; // fp32 weights staged per round (16 KB)

template <typename T> __device__ inline float load_as_f32(const T *p);
template <> __device__ inline float load_as_f32<float>(const float *p) { return *p; }
template <> __device__ inline float load_as_f32<uint16_t>(const uint16_t *p) { return bf16_bits_to_f32(*p); }

template <typename T> __device__ inline void store_from_f32(T *p, float v);
template <> __device__ inline void store_from_f32<float>(float *p, float v) { *p = v; }
template <> __device__ inline void store_from_f32<uint16_t>(uint16_t *p, float v) { *p = f32_bits_to_bf16(__float_as_uint(v)); }

// 4 consecutive channels as fp32 (pointer is 4-element aligned)
__device__ inline float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ inline float4 load4(const uint16_t *p)
{
    const uint2 u = *reinterpret_cast<const uint2 *>(p);
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u),
                       __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u));
}

template <typename T> struct AccOf { typedef float type; };
template <> struct AccOf<float> { typedef double type; };

template <typename TX, typename TY>
__global__ void __launch_bounds__(kSimtPixels)
conv_bp_simt_kernel(npas_conv_desc d, int Mb, int Nb, int P, int Q, const TX *__restrict__ x,
                    const uint8_t *__restrict__ blob, const float *__restrict__ bias,
                    const TY *__restrict__ res, TY *__restrict__ y)
{
    __shared__ __align__(16) float w_s[kSimtWFloats];
    __shared__ uint32_t pair_s[kSimtWFloats / kSimtFilters];

    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(blob);
    const uint32_t nCB = d.C / Nb, G = (Nb % 8 == 0) ? 8 : Nb;
    const uint32_t *blk_off = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_BLK]);
    const uint32_t *pairs = reinterpret_cast<const uint32_t *>(blob + hdr[BP_OFF_PAIRS]);
    const TX *vals = reinterpret_cast<const TX *>(blob + hdr[BP_OFF_VALUES]);

    const int fb = blockIdx.y, f0 = blockIdx.z * kSimtFilters;
    const int nf = min(kSimtFilters, Mb - f0);
    const long long npix = (long long)d.N * P * Q;
    const long long pix = (long long)blockIdx.x * kSimtPixels + threadIdx.x;
    const bool live = pix < npix;
    int n = 0, p = 0, q = 0;
    if (live) { n = (int)(pix / (P * Q)); const int rem = (int)(pix % (P * Q)); p = rem / Q; q = rem % Q; }

    typedef typename AccOf<TX>::type TA;
    TA acc[kSimtFilters];
#pragma unroll
    for (int f = 0; f < kSimtFilters; ++f) acc[f] = 0;

    const uint32_t j_begin = blk_off[(size_t)fb * nCB], j_end = blk_off[(size_t)(fb + 1) * nCB];
    const uint32_t pairs_per_round = max(1u, (uint32_t)kSimtWFloats / (kSimtFilters * Nb));
    const bool vec4 = (Nb % 4 == 0) && (d.C % 4 == 0);

    for (uint32_t j0 = j_begin; j0 < j_end; j0 += pairs_per_round) {
        const uint32_t nj = min(pairs_per_round, j_end - j0);
        __syncthreads();
        // stage weights of pairs j0..j0+nj as fp32 in [pair][f][c] order
        for (uint32_t e = threadIdx.x; e < nj * kSimtFilters * Nb; e += blockDim.x) {
            const uint32_t pj = e / (kSimtFilters * Nb), f = (e / Nb) % kSimtFilters, c = e % Nb;
            float v = 0.f;
            if ((int)f < nf)
                v = load_as_f32(vals + ((size_t)((j0 + pj) * (Nb / G) + c / G) * Mb + f0 + f) * G + c % G);
            w_s[e] = v;
        }
        for (uint32_t e = threadIdx.x; e < nj; e += blockDim.x) pair_s[e] = pairs[j0 + e];
        __syncthreads();
        if (!live) continue;
        for (uint32_t pj = 0; pj < nj; ++pj) {
            const uint32_t pw = pair_s[pj], cb = pw & 0xFFFFu, tap = pw >> 16;
            const int r = tap / d.S, s = tap % d.S;
            const int h = p * d.stride + r - d.pad, v = q * d.stride + s - d.pad;
            if (h < 0 || h >= d.H || v < 0 || v >= d.W) continue;     // zero padding
            const TX *xp = x + (((size_t)n * d.H + h) * d.W + v) * d.C + cb * Nb;
            const float *wp = w_s + pj * kSimtFilters * Nb;
            if (vec4) {
                for (int c = 0; c < Nb; c += 4) {
                    const float4 xv = load4(xp + c);
#pragma unroll
                    for (int f = 0; f < kSimtFilters; ++f) {
                        const float4 wv = *reinterpret_cast<const float4 *>(wp + f * Nb + c);
                        acc[f] = fma((TA)xv.x, (TA)wv.x, acc[f]); acc[f] = fma((TA)xv.y, (TA)wv.y, acc[f]);
                        acc[f] = fma((TA)xv.z, (TA)wv.z, acc[f]); acc[f] = fma((TA)xv.w, (TA)wv.w, acc[f]);
                    }
                }
            } else {
                for (int c = 0; c < Nb; ++c) {
                    const float xv = load_as_f32(xp + c);
#pragma unroll
                    for (int f = 0; f < kSimtFilters; ++f) acc[f] = fma((TA)xv, (TA)wp[f * Nb + c], acc[f]);
                }
            }
        }
    }
    if (!live) return;
    // fused epilogue: bias, residual, ReLU, one rounding at the store
    const size_t o0 = (size_t)pix * d.K + fb * Mb + f0;
#pragma unroll
    for (int f = 0; f < kSimtFilters; ++f) {
        if (f >= nf) break;
        TA v = acc[f];
        if (bias) v += (TA)bias[fb * Mb + f0 + f];
        if (res) v += (TA)load_as_f32(res + o0 + f);
        if (d.relu) v = v > 0 ? v : 0;
        store_from_f32(y + o0 + f, (float)v);
    }
}

npas_status conv_simt_launch(const npas_conv_desc &d, const npas_bp_desc &bp, const void *x,
                             const void *blob, const float *bias, const void *res, void *y,
                             cudaStream_t st)
{
    const int P = (d.H + 2 * d.pad - d.R) / d.stride + 1, Q = (d.W + 2 * d.pad - d.S) / d.stride + 1;
    const long long npix = (long long)d.N * P * Q;
    if (kSimtFilters * bp.Nb > kSimtWFloats) return NPAS_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)((npix + kSimtPixels - 1) / kSimtPixels), bp.K / bp.Mb,
                    (bp.Mb + kSimtFilters - 1) / kSimtFilters);
    if (grid.y > 65535 || grid.z > 65535) return NPAS_ERR_UNSUPPORTED;
    const uint8_t *b8 = static_cast<const uint8_t *>(blob);
    if (d.x_dtype == NPAS_F32 && d.y_dtype == NPAS_F32)
        conv_bp_simt_kernel<float, float><<<grid, kSimtPixels, 0, st>>>(
            d, bp.Mb, bp.Nb, P, Q, static_cast<const float *>(x), b8, bias, static_cast<const float *>(res),
            static_cast<float *>(y));
    else if (d.x_dtype == NPAS_BF16 && d.y_dtype == NPAS_BF16)
        conv_bp_simt_kernel<uint16_t, uint16_t><<<grid, kSimtPixels, 0, st>>>(
            d, bp.Mb, bp.Nb, P, Q, static_cast<const uint16_t *>(x), b8, bias, static_cast<const uint16_t *>(res),
            static_cast<uint16_t *>(y));
    else if (d.x_dtype == NPAS_BF16 && d.y_dtype == NPAS_F32)
        conv_bp_simt_kernel<uint16_t, float><<<grid, kSimtPixels, 0, st>>>(
            d, bp.Mb, bp.Nb, P, Q, static_cast<const uint16_t *>(x), b8, bias, static_cast<const float *>(res),
            static_cast<float *>(y));
    else
        return NPAS_ERR_DTYPE;
    count_launch();
    return launch_status();
}

}  // namespace npas
