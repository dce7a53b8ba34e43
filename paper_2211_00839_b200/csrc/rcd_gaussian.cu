// Gaussian-kernel similarity (Section 4, item 2: "a Gaussian kernel with L2 distance" whose
// bandwidth is sigma = sum_{v,v'} ||v - v'||_2 / n^2).  Reading taken (the paper gives neither the
// exponent nor what n counts): n = |V_l|, all ordered pairs of the class, and
//     sim(v, v') = exp(-||v - v'||^2 / (2 sigma^2)).
//
// Built on the dot-product matrix the similarity kernels have already written:
//     ||v - v'||^2 = ||v||^2 + ||v'||^2 - 2 <v, v'>,
// exact in integers for int8 features.  Four small kernels: row norms, per-row-block sums of the
// distances (fp64, fixed order), sigma per class, and the in-place transform of S to fp32 kernel
// values.  The sums are reduced in a fixed order so that sigma, and with it every similarity, is
// reproducible from run to run.
#include "rcd_internal.h"

namespace rcd {

constexpr int kGaussRows = 64;       // rows of S per CTA
constexpr int kGaussWarps = 8;

__device__ __forceinline__ float bf16_bits_as_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

// ||x_r||^2 of every class-sorted row: int32 for int8 features (exact), fp32 for bf16.
template <bool kInt8>
__global__ void __launch_bounds__(256, 4) row_norms_kernel(const void *__restrict__ Xs, int64_t N, int64_t d, void *__restrict__ norms)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= N) return;
    if constexpr (kInt8) {
        const int8_t *x = reinterpret_cast<const int8_t *>(Xs) + row * d;
        int acc = 0;
        for (int64_t k = lane; k < d; k += 32) acc += (int)x[k] * (int)x[k];
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) reinterpret_cast<int32_t *>(norms)[row] = acc;
    } else {
        const uint16_t *x = reinterpret_cast<const uint16_t *>(Xs) + row * d;
        float acc = 0.f;
        for (int64_t k = lane; k < d; k += 32) { const float v = bf16_bits_as_float(x[k]); acc = fmaf(v, v, acc); }
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) reinterpret_cast<float *>(norms)[row] = acc;
    }
}

// Squared distance of samples i and j of a class from their norms and dot product.
template <bool kInt8>
__device__ __forceinline__ float squared_distance(const void *norms, int64_t gi, int64_t gj, uint32_t dotBits, bool same)
{
    if (same) return 0.f;
    if constexpr (kInt8) {
        const int32_t *n = reinterpret_cast<const int32_t *>(norms);
        const long long v = (long long)n[gi] + (long long)n[gj] - 2ll * (long long)(int32_t)dotBits;
        return (float)v;                                   // exact integer, one rounding
    } else {
        const float *n = reinterpret_cast<const float *>(norms);
        return fmaxf(n[gi] + n[gj] - 2.f * __uint_as_float(dotBits), 0.f);
    }
}

template <bool kInt8>
__global__ void __launch_bounds__(kGaussWarps * 32, 4) gauss_dist_sum_kernel(DescSource src, const uint32_t *__restrict__ S,
                                                                            const void *__restrict__ norms, int32_t maxBlocks,
                                                                            double *__restrict__ partial)
{
    __shared__ double shWarp[kGaussWarps];
    const int l = blockIdx.y;
    const ClassDesc c = src.get(l);
    const int first = blockIdx.x * kGaussRows;
    if (first >= c.M) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double mine = 0.0;
    for (int r = warp; r < kGaussRows; r += kGaussWarps) {
        const int i = first + r;
        if (i >= c.M) break;
        const uint32_t *row = S + c.sOff + (int64_t)i * c.ld;
        double acc = 0.0;
        for (int j = lane; j < c.M; j += 32)
            acc += sqrt((double)squared_distance<kInt8>(norms, c.row0 + i, c.row0 + j, row[j], i == j));
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        mine += acc;                                       // rows of this warp, in row order
    }
    if (lane == 0) shWarp[warp] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < kGaussWarps; ++w) s += shWarp[w];
        partial[(int64_t)l * maxBlocks + blockIdx.x] = s;
    }
}

// sigma_l = (sum of all pairwise distances) / M^2 ; scale_l = 1 / (2 sigma^2)  (0 when sigma = 0)
__global__ void gauss_sigma_kernel(DescSource src, int32_t L, const double *__restrict__ partial, int32_t maxBlocks,
                                   float *__restrict__ sigma, float *__restrict__ scale)
{
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= L) return;
    const ClassDesc c = src.get(l);
    const int nb = (c.M + kGaussRows - 1) / kGaussRows;
    double s = 0.0;
    for (int b = 0; b < nb; ++b) s += partial[(int64_t)l * maxBlocks + b];
    const double sg = c.M > 0 ? s / ((double)c.M * (double)c.M) : 0.0;
    sigma[l] = (float)sg;
    scale[l] = sg > 0.0 ? (float)(1.0 / (2.0 * sg * sg)) : 0.f;
}

template <bool kInt8>
__global__ void __launch_bounds__(kGaussWarps * 32, 4) gauss_apply_kernel(DescSource src, uint32_t *__restrict__ S,
                                                                         const void *__restrict__ norms,
                                                                         const float *__restrict__ scale)
{
    const int l = blockIdx.y;
    const ClassDesc c = src.get(l);
    const int first = blockIdx.x * kGaussRows;
    if (first >= c.M) return;
    const float k = scale[l];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int r = warp; r < kGaussRows; r += kGaussWarps) {
        const int i = first + r;
        if (i >= c.M) break;
        uint32_t *row = S + c.sOff + (int64_t)i * c.ld;
        for (int j = lane; j < c.M; j += 32) {
            const float d2 = squared_distance<kInt8>(norms, c.row0 + i, c.row0 + j, row[j], i == j);
            row[j] = __float_as_uint(k > 0.f ? expf(-d2 * k) : 1.0f);       // sigma = 0: all points coincide
        }
    }
}

rcd_status launch_gaussian(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t N, int64_t d, const SimClasses &cls,
                           void *S, void *norms, double *partial, float *sigma, float *scale, cudaStream_t st)
{
    if (N == 0 || cls.L == 0 || cls.maxM == 0) return RCD_OK;
    if (cls.L > 65535) return fail(ctx, RCD_ERR_UNSUPPORTED, "Gaussian similarity: more than 65535 classes");
    const int maxBlocks = (int)((cls.maxM + kGaussRows - 1) / kGaussRows);
    const unsigned normBlocks = (unsigned)((N + 7) / 8);
    dim3 grid(maxBlocks, cls.L);
    if (dtype == RCD_FEAT_I8) {
        row_norms_kernel<true><<<normBlocks, 256, 0, st>>>(Xs, N, d, norms);
        gauss_dist_sum_kernel<true><<<grid, kGaussWarps * 32, 0, st>>>(cls.src, (const uint32_t *)S, norms, maxBlocks, partial);
    } else {
        row_norms_kernel<false><<<normBlocks, 256, 0, st>>>(Xs, N, d, norms);
        gauss_dist_sum_kernel<false><<<grid, kGaussWarps * 32, 0, st>>>(cls.src, (const uint32_t *)S, norms, maxBlocks, partial);
    }
    gauss_sigma_kernel<<<(cls.L + 127) / 128, 128, 0, st>>>(cls.src, cls.L, partial, maxBlocks, sigma, scale);
    if (dtype == RCD_FEAT_I8) gauss_apply_kernel<true><<<grid, kGaussWarps * 32, 0, st>>>(cls.src, (uint32_t *)S, norms, scale);
    else gauss_apply_kernel<false><<<grid, kGaussWarps * 32, 0, st>>>(cls.src, (uint32_t *)S, norms, scale);
    ctx->kernelLaunches += 4;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

size_t gaussian_scratch_bytes(int64_t N, int32_t L, int64_t maxM)
{
    const size_t maxBlocks = (size_t)((maxM + kGaussRows - 1) / kGaussRows);
    return align_up((size_t)(N > 0 ? N : 1) * 4) + align_up((size_t)L * (maxBlocks ? maxBlocks : 1) * 8) + 2 * align_up((size_t)L * 4);
}

}  // namespace rcd
