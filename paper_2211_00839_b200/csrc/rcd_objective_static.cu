// rcd_objective_class_static: the facility-location value of every block of ONE class, from a
// similarity matrix the caller already holds, for callers that cannot allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- inside a region that must not
// touch the allocator (a latency-critical serving loop, a callback running under another
// framework's memory pool with a fixed budget, a process whose memory was carved up front) -- and
// that therefore cannot provide the workspace rcd_objective asks for.  The per-row-block partial
// sums that the objective kernels need live in a fixed array inside the library image instead.
//
// Consequences of that choice, all of them the caller's to respect:
//   - the array is part of the loaded library: every GPU that loads it holds kStaticScratchBytes
//     (1 MiB) until the process exits;
//   - sizes are bounded: ceil(M/64) * W * 8 bytes must fit in the array;
//   - all calls on a device share the one array, so two calls whose kernels overlap on the GPU
//     (different streams) race on it; the array keeps the previous call's partial sums, but
//     nothing in it has to start at zero: every slot a call reads it has written first;
//   - the first call on each device looks the array's device address up (cudaGetSymbolAddress);
//     make that first call outside any stream capture.
#include "rcd_internal.h"

#include <mutex>
#include <type_traits>

namespace rcd {

constexpr size_t kStaticScratchBytes = 1u << 20;
constexpr int kStaticRowsPerCta = 64;
constexpr int kStaticWarps = 8;
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the runtime's symbol table, not an address a
// kernel could use; the address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_objectiveScratch[kStaticScratchBytes];

// One address per device, looked up once; the table is shared by every context of the process, so the
// lookup is serialised (two contexts on two host threads may make their first call at the same time).
static void *g_scratchAddr[kMaxDevices] = {};
static std::mutex g_scratchLock;

static rcd_status static_scratch(rcd_ctx *ctx, void **out)
{
    if (ctx->device < 0 || ctx->device >= kMaxDevices)
        return fail(ctx, RCD_ERR_UNSUPPORTED, "device index %d beyond the %d devices this entry point tracks", ctx->device, kMaxDevices);
    std::lock_guard<std::mutex> guard(g_scratchLock);
    if (!g_scratchAddr[ctx->device]) {
        void *p = nullptr;
        RCD_CUDA(ctx, cudaSetDevice(ctx->device));
        RCD_CUDA(ctx, cudaGetSymbolAddress(&p, g_objectiveScratch));
        g_scratchAddr[ctx->device] = p;
    }
    *out = g_scratchAddr[ctx->device];
    return RCD_OK;
}

// Row block b of the class: per block p the sum over the block's rows i of
// max(0, max_{v: assignment[v] == p} S[i][v]), written to partial[b][p].
template <typename SV, typename FV>
__global__ void __launch_bounds__(kStaticWarps * 32, 4) objective_class_rows_kernel(const SV *__restrict__ S, int M, int ld,
                                                                                   const int32_t *__restrict__ assignment,
                                                                                   int W, FV *__restrict__ partial)
{
    extern __shared__ unsigned char shraw[];
    FV *shSum = reinterpret_cast<FV *>(shraw);                                        // [warps][W]
    int32_t *shTop = reinterpret_cast<int32_t *>(shSum + (size_t)kStaticWarps * W);   // [warps][W]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int first = blockIdx.x * kStaticRowsPerCta;
    FV *sum = shSum + (size_t)warp * W;
    int32_t *top = shTop + (size_t)warp * W;
    for (int p = lane; p < W; p += 32) sum[p] = (FV)0;
    for (int r = warp; r < kStaticRowsPerCta; r += kStaticWarps) {
        const int i = first + r;
        if (i >= M) break;
        for (int p = lane; p < W; p += 32) top[p] = 0;
        __syncwarp();
        const SV *row = S + (int64_t)i * ld;
        for (int v = lane; v < M; v += 32) {
            const int a = assignment[v];
            if (a < 0 || a >= W) continue;
            const SV s = row[v];
            if (s > (SV)0) {
                // positive int32 and positive fp32 values both compare like their bit patterns
                int32_t bits;
                if constexpr (std::is_integral<SV>::value) bits = (int32_t)s;
                else bits = __float_as_int((float)s);
                atomicMax(&top[a], bits);
            }
        }
        __syncwarp();
        for (int p = lane; p < W; p += 32) {
            if constexpr (std::is_integral<SV>::value) sum[p] += (FV)top[p];
            else sum[p] += (FV)__int_as_float(top[p]);
        }
        __syncwarp();
    }
    __syncthreads();
    FV *out = partial + (int64_t)blockIdx.x * W;
    for (int p = threadIdx.x; p < W; p += blockDim.x) {
        FV s = (FV)0;
        for (int w = 0; w < kStaticWarps; ++w) s += shSum[(size_t)w * W + p];
        out[p] = s;
    }
}

// One CTA: block values in row-block order, then their total by a fixed tree (reproducible).
template <typename FV>
__global__ void __launch_bounds__(256, 1) objective_class_finish_kernel(const FV *__restrict__ partial, int nBlocks, int W,
                                                                       FV *__restrict__ partValues, FV *__restrict__ total)
{
    __shared__ FV sh[256];
    FV mine = (FV)0;
    for (int p = threadIdx.x; p < W; p += 256) {
        FV s = (FV)0;
        for (int b = 0; b < nBlocks; ++b) s += partial[(int64_t)b * W + p];
        partValues[p] = s;
        mine += s;
    }
    sh[threadIdx.x] = mine;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if ((int)threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) *total = sh[0];
}

template <typename SV, typename FV>
static rcd_status run_static(rcd_ctx *ctx, const void *S, int M, int ld, const int32_t *assignment, int W,
                             void *partValues, void *total, void *scratch, cudaStream_t st)
{
    const int nBlocks = (M + kStaticRowsPerCta - 1) / kStaticRowsPerCta;
    const size_t smem = (size_t)kStaticWarps * W * (sizeof(FV) + sizeof(int32_t));
    if ((int64_t)smem > ctx->maxSmemOptin - 1024)
        return fail(ctx, RCD_ERR_UNSUPPORTED, "W=%d needs %zu bytes of shared memory", W, smem);
    RCD_CUDA(ctx, cudaFuncSetAttribute(objective_class_rows_kernel<SV, FV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (nBlocks > 0)
        objective_class_rows_kernel<SV, FV><<<nBlocks, kStaticWarps * 32, smem, st>>>((const SV *)S, M, ld, assignment, W, (FV *)scratch);
    objective_class_finish_kernel<FV><<<1, 256, 0, st>>>((const FV *)scratch, nBlocks, W, (FV *)partValues, (FV *)total);
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

}  // namespace rcd

using namespace rcd;

extern "C" rcd_status rcd_objective_class_static(rcd_ctx *ctx, const void *S_dev, rcd_feat_dtype dtype, int64_t M,
                                                 int64_t ldS, const int32_t *assignment_dev, int32_t W,
                                                 void *part_values_dev, void *total_dev, void *cuda_stream)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    if (dtype != RCD_FEAT_I8 && dtype != RCD_FEAT_BF16) return fail(ctx, RCD_ERR_INVALID_ARG, "unknown dtype %d", (int)dtype);
    if (ctx->cfg.objective != RCD_OBJ_FACILITY)
        return fail(ctx, RCD_ERR_UNSUPPORTED, "rcd_objective_class_static evaluates facility location only; this context is set to another objective");
    if (M < 0 || W <= 0 || ldS < M) return fail(ctx, RCD_ERR_INVALID_ARG, "need M >= 0, W > 0, ldS >= M");
    if (!part_values_dev || !total_dev || (M > 0 && (!S_dev || !assignment_dev)))
        return fail(ctx, RCD_ERR_INVALID_ARG, "null device pointer");
    const int64_t nBlocks = (M + kStaticRowsPerCta - 1) / kStaticRowsPerCta;
    if (M > 0x7fffffffLL || W > 1024 || (uint64_t)nBlocks * (uint64_t)W * 8u > kStaticScratchBytes)
        return fail(ctx, RCD_ERR_UNSUPPORTED,
                    "M=%lld, W=%d: ceil(M/64)*W*8 = %lld bytes exceeds the %zu-byte built-in scratch array (and W <= 1024)",
                    (long long)M, W, (long long)(nBlocks * W * 8), kStaticScratchBytes);
    void *scratch = nullptr;
    rcd_status rs = static_scratch(ctx, &scratch);
    if (rs != RCD_OK) return rs;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    if (dtype == RCD_FEAT_I8)
        return run_static<int32_t, long long>(ctx, S_dev, (int)M, (int)ldS, assignment_dev, W, part_values_dev, total_dev, scratch, st);
    return run_static<float, double>(ctx, S_dev, (int)M, (int)ldS, assignment_dev, W, part_values_dev, total_dev, scratch, st);
}
