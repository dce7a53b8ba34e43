// Similarity matrices S_l = X_l X_l^T (Section 3.1: similarities are computed from the feature
// vectors; dot product for int8 features, cosine for L2-normalised bf16 features).
//
// This file holds the dispatcher and the generic CUDA-core kernel, which takes any d and any
// alignment (dp4a for int8, fp32 FMA for bf16).  The tensor-core kernel (tcgen05 + TMEM, fed
// by TMA) lives in rcd_similarity_tc.cu and is used whenever the rows are 16-byte multiples.
#include "rcd_internal.h"

namespace rcd {

constexpr int kTile = 64;     // output tile per CTA (kTile x kTile), 16x16 threads, 4x4 per thread

// int8: k-slab of 64 bytes per row = 16 packed words (+1 pad word against bank conflicts)
__global__ void __launch_bounds__(256, 2) sim_generic_i8_kernel(const int8_t *__restrict__ Xs, int64_t d,
                                                            DescSource src, int32_t L,
                                                            int32_t *__restrict__ S)
{
    __shared__ int32_t As[kTile][17];
    __shared__ int32_t Bs[kTile][17];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const bool words = (d % 4 == 0) && (((uintptr_t)Xs) % 4 == 0);
    for (int l = blockIdx.z; l < L; l += gridDim.z) {
        const ClassDesc c = src.get(l);
        const int tilesN = (c.ld + kTile - 1) / kTile;
        const int tilesM = (c.M + kTile - 1) / kTile;
        if ((int)blockIdx.x >= tilesN || (int)blockIdx.y >= tilesM) continue;
        const int rowA0 = blockIdx.y * kTile, rowB0 = blockIdx.x * kTile;
        const int8_t *X = Xs + (int64_t)c.row0 * d;
        int32_t acc[4][4] = {};
        for (int64_t k0 = 0; k0 < d; k0 += 64) {
            // each thread loads 4 words of A and 4 of B: word w of row r, idx = r*16 + w
            for (int q = 0; q < 4; ++q) {
                int idx = threadIdx.x + q * 256;
                int r = idx >> 4, w = idx & 15;
                int64_t k = k0 + 4 * w;
                int32_t va = 0, vb = 0;
                int ra = rowA0 + r, rb = rowB0 + r;
                if (words) {
                    if (k < d) {
                        if (ra < c.M) va = *(const int32_t *)(X + (int64_t)ra * d + k);
                        if (rb < c.M) vb = *(const int32_t *)(X + (int64_t)rb * d + k);
                    }
                } else {
                    for (int b = 0; b < 4; ++b) {
                        if (k + b < d) {
                            if (ra < c.M) va |= (int32_t)(uint8_t)X[(int64_t)ra * d + k + b] << (8 * b);
                            if (rb < c.M) vb |= (int32_t)(uint8_t)X[(int64_t)rb * d + k + b] << (8 * b);
                        }
                    }
                }
                As[r][w] = va;
                Bs[r][w] = vb;
            }
            __syncthreads();
#pragma unroll
            for (int w = 0; w < 16; ++w) {
                int32_t a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { a[i] = As[ty * 4 + i][w]; b[i] = Bs[tx * 4 + i][w]; }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(a[i], b[j], acc[i][j]);
            }
            __syncthreads();
        }
        int32_t *Sl = S + c.sOff;
        for (int i = 0; i < 4; ++i) {
            int r = rowA0 + ty * 4 + i;
            if (r >= c.M) continue;
            for (int j = 0; j < 4; ++j) {
                int col = rowB0 + tx * 4 + j;
                if (col < c.ld) Sl[(int64_t)r * c.ld + col] = (col < c.M) ? acc[i][j] : 0;
            }
        }
    }
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

// bf16: k-slab of 32 elements per row, widened to fp32 in shared memory
__global__ void __launch_bounds__(256, 2) sim_generic_bf16_kernel(const uint16_t *__restrict__ Xs, int64_t d,
                                                              DescSource src, int32_t L,
                                                              float *__restrict__ S)
{
    __shared__ float As[kTile][33];
    __shared__ float Bs[kTile][33];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    for (int l = blockIdx.z; l < L; l += gridDim.z) {
        const ClassDesc c = src.get(l);
        const int tilesN = (c.ld + kTile - 1) / kTile;
        const int tilesM = (c.M + kTile - 1) / kTile;
        if ((int)blockIdx.x >= tilesN || (int)blockIdx.y >= tilesM) continue;
        const int rowA0 = blockIdx.y * kTile, rowB0 = blockIdx.x * kTile;
        const uint16_t *X = Xs + (int64_t)c.row0 * d;
        float acc[4][4] = {};
        for (int64_t k0 = 0; k0 < d; k0 += 32) {
            for (int q = 0; q < 8; ++q) {
                int idx = threadIdx.x + q * 256;
                int r = idx >> 5, w = idx & 31;
                int64_t k = k0 + w;
                float va = 0.f, vb = 0.f;
                int ra = rowA0 + r, rb = rowB0 + r;
                if (k < d) {
                    if (ra < c.M) va = bf16_bits_to_float(X[(int64_t)ra * d + k]);
                    if (rb < c.M) vb = bf16_bits_to_float(X[(int64_t)rb * d + k]);
                }
                As[r][w] = va;
                Bs[r][w] = vb;
            }
            __syncthreads();
#pragma unroll 8
            for (int w = 0; w < 32; ++w) {
                float a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { a[i] = As[ty * 4 + i][w]; b[i] = Bs[tx * 4 + i][w]; }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
            __syncthreads();
        }
        float *Sl = S + c.sOff;
        for (int i = 0; i < 4; ++i) {
            int r = rowA0 + ty * 4 + i;
            if (r >= c.M) continue;
            for (int j = 0; j < 4; ++j) {
                int col = rowB0 + tx * 4 + j;
                if (col < c.ld) Sl[(int64_t)r * c.ld + col] = (col < c.M) ? acc[i][j] : 0.f;
            }
        }
    }
}

static rcd_status launch_similarity_generic(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t d,
                                            const SimClasses &cls, void *S, cudaStream_t st)
{
    const int32_t L = cls.L;
    const int maxLd = pad_row(cls.maxM), maxM = (int)cls.maxM;     // covers either row pitch (pad4 <= pad_row)
    const DescSource src = cls.src;
    if (L == 0 || maxM == 0) return RCD_OK;
    dim3 grid((maxLd + kTile - 1) / kTile, (maxM + kTile - 1) / kTile, L > 65535 ? 65535 : L);
    if (dtype == RCD_FEAT_I8)
        sim_generic_i8_kernel<<<grid, 256, 0, st>>>((const int8_t *)Xs, d, src, L, (int32_t *)S);
    else
        sim_generic_bf16_kernel<<<grid, 256, 0, st>>>((const uint16_t *)Xs, d, src, L, (float *)S);
    ctx->kernelLaunches++;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

rcd_status launch_similarity_tc(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t Ntot, int64_t d,
                                const SimClasses &cls, void *S, cudaStream_t st, bool *handled);

rcd_status launch_similarity(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t Ntot, int64_t d,
                             const SimClasses &cls, void *S, cudaStream_t st)
{
    if (ctx->cfg.similarity_path != 2) {
        bool handled = false;
        rcd_status rs = launch_similarity_tc(ctx, Xs, dtype, Ntot, d, cls, S, st, &handled);
        if (rs != RCD_OK) return rs;
        if (handled) return RCD_OK;
    }
    return launch_similarity_generic(ctx, Xs, dtype, d, cls, S, st);
}

}  // namespace rcd
