// Class split (Algorithm 1: "Split the ground set V into L sets according to class labels"):
// label histogram, stable ranking of every sample inside its class, and the gather of the
// feature rows into class-sorted order.  Stable = inside a class the samples keep their
// dataset order, which is what fixes the lowest-index tie-breaks downstream.
#include "rcd_internal.h"

namespace rcd {

// ---- label histogram ------------------------------------------------------------------------
__global__ void count_labels_kernel(const int32_t *__restrict__ labels, int64_t N, int32_t L,
                                    int32_t *__restrict__ counts, int32_t *__restrict__ status)
{
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += stride) {
        int32_t lab = labels[i];
        if (lab < 0 || lab >= L) { bad = true; continue; }
        atomicAdd(&counts[lab], 1);
    }
    if (bad) atomicOr(status, kDevBadLabel);
}

rcd_status launch_count_labels(rcd_ctx *ctx, const int32_t *labels, int64_t N, int32_t L, int32_t *counts,
                               int32_t *status, cudaStream_t st)
{
    if (N == 0) return RCD_OK;
    int threads = 256;
    int64_t blocks = (N + threads - 1) / threads;
    if (blocks > 4LL * ctx->smCount) blocks = 4LL * ctx->smCount;
    count_labels_kernel<<<(unsigned)blocks, threads, 0, st>>>(labels, N, L, counts, status);
    ctx->kernelLaunches++;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

// ---- stable split ---------------------------------------------------------------------------
// Chunks of kGroupChunk consecutive samples.  Pass A: per chunk and label, how many samples of
// that label the chunk holds (written by the chunk's last sample of the label).  Pass B: per
// label, exclusive running sum over chunks, started at the class offset.  Pass C: position =
// chunk base + rank inside the chunk.

__device__ __forceinline__ void chunk_rank(const int32_t *sh, int n, int t, int lab, int &rank, bool &last)
{
    rank = 0;
    last = true;
    for (int i = 0; i < n; ++i) {
        int other = sh[i];
        if (other == lab) {
            if (i < t) ++rank;
            if (i > t) last = false;
        }
    }
}

__global__ void __launch_bounds__(kGroupChunk, 1) chunk_hist_kernel(const int32_t *__restrict__ labels, int64_t N,
                                                                int32_t L, int32_t *__restrict__ chunkHist)
{
    __shared__ int32_t sh[kGroupChunk];
    int64_t base = (int64_t)blockIdx.x * kGroupChunk;
    int n = (int)min((int64_t)kGroupChunk, N - base);
    int t = threadIdx.x;
    int lab = -1;
    if (t < n) lab = labels[base + t];
    sh[t] = lab;
    __syncthreads();
    if (t < n && lab >= 0 && lab < L) {
        int rank; bool last;
        chunk_rank(sh, n, t, lab, rank, last);
        if (last) chunkHist[(int64_t)blockIdx.x * L + lab] = rank + 1;
    }
}

__global__ void chunk_scan_kernel(int32_t *__restrict__ chunkHist, int32_t nChunks, int32_t L,
                                  const ClassDesc *__restrict__ desc)
{
    int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= L) return;
    int32_t run = desc[l].row0;
    for (int c = 0; c < nChunks; ++c) {
        int64_t at = (int64_t)c * L + l;
        int32_t h = chunkHist[at];
        chunkHist[at] = run;
        run += h;
    }
}

__global__ void __launch_bounds__(kGroupChunk, 1) chunk_place_kernel(const int32_t *__restrict__ labels, int64_t N,
                                                                 int32_t L, const int32_t *__restrict__ chunkBase,
                                                                 int32_t *__restrict__ perm)
{
    __shared__ int32_t sh[kGroupChunk];
    int64_t base = (int64_t)blockIdx.x * kGroupChunk;
    int n = (int)min((int64_t)kGroupChunk, N - base);
    int t = threadIdx.x;
    int lab = -1;
    if (t < n) lab = labels[base + t];
    sh[t] = lab;
    __syncthreads();
    if (t < n && lab >= 0 && lab < L) {
        int rank; bool last;
        chunk_rank(sh, n, t, lab, rank, last);
        perm[chunkBase[(int64_t)blockIdx.x * L + lab] + rank] = (int32_t)(base + t);
    }
}

rcd_status launch_stable_split(rcd_ctx *ctx, const int32_t *labels, int64_t N, int32_t L, int32_t nChunks,
                               int32_t *chunkHist, const ClassDesc *descDev, int32_t *perm, cudaStream_t st)
{
    if (N == 0) return RCD_OK;
    RCD_CUDA(ctx, cudaMemsetAsync(chunkHist, 0, (size_t)nChunks * L * sizeof(int32_t), st));
    chunk_hist_kernel<<<nChunks, kGroupChunk, 0, st>>>(labels, N, L, chunkHist);
    chunk_scan_kernel<<<(L + 127) / 128, 128, 0, st>>>(chunkHist, nChunks, L, descDev);
    chunk_place_kernel<<<nChunks, kGroupChunk, 0, st>>>(labels, N, L, chunkHist, perm);
    ctx->kernelLaunches += 3;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

// ---- feature gather -------------------------------------------------------------------------
__global__ void gather_rows16_kernel(const int4 *__restrict__ X, const int32_t *__restrict__ perm, int64_t N,
                                     int64_t row16, int4 *__restrict__ Xs)
{
    int64_t total = N * row16;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int64_t r = i / row16, c = i - r * row16;
        Xs[i] = X[(int64_t)perm[r] * row16 + c];
    }
}

__global__ void gather_rows1_kernel(const uint8_t *__restrict__ X, const int32_t *__restrict__ perm, int64_t N,
                                    int64_t rowBytes, uint8_t *__restrict__ Xs)
{
    int64_t total = N * rowBytes;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int64_t r = i / rowBytes, c = i - r * rowBytes;
        Xs[i] = X[(int64_t)perm[r] * rowBytes + c];
    }
}

rcd_status launch_gather_rows(rcd_ctx *ctx, const void *X, const int32_t *perm, int64_t N, int64_t rowBytes,
                              void *Xs, cudaStream_t st)
{
    if (N == 0 || rowBytes == 0) return RCD_OK;
    int threads = 256;
    bool vec = (rowBytes % 16 == 0) && (((uintptr_t)X) % 16 == 0) && (((uintptr_t)Xs) % 16 == 0);
    int64_t total = vec ? N * (rowBytes / 16) : N * rowBytes;
    int64_t blocks = (total + threads - 1) / threads;
    int64_t cap = 32LL * ctx->smCount;
    if (blocks > cap) blocks = cap;
    if (vec)
        gather_rows16_kernel<<<(unsigned)blocks, threads, 0, st>>>((const int4 *)X, perm, N, rowBytes / 16, (int4 *)Xs);
    else
        gather_rows1_kernel<<<(unsigned)blocks, threads, 0, st>>>((const uint8_t *)X, perm, N, rowBytes, (uint8_t *)Xs);
    ctx->kernelLaunches++;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

}  // namespace rcd
