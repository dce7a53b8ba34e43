// f(A_j^l) = sum_{i in V_l} max(0, max_{v' in A_j^l} S[i][v'])  for every class l and block j,
// straight from the definition (Section 4, item 2), given an assignment vector.  Independent of
// the greedy state: one pass over S; per row i a per-block running maximum, then fixed-order sums
// so that the fp64 result is reproducible.
#include "rcd_internal.h"

#include <type_traits>

namespace rcd {

constexpr int kObjWarps = 8;
constexpr int kObjRowsPerCta = 64;

template <typename SV, typename FV>
__global__ void __launch_bounds__(kObjWarps * 32, 4) objective_rows_kernel(const ClassDesc *__restrict__ desc,
                                                                       const SV *__restrict__ S,
                                                                       const int32_t *__restrict__ perm,
                                                                       const int32_t *__restrict__ assignment,
                                                                       int32_t W, int32_t maxBlocks,
                                                                       FV *__restrict__ partial)
{
    extern __shared__ unsigned char shraw[];
    // per warp: running maxima of the current row [W] (int bits) and accumulated sums [W]
    FV *shAcc = reinterpret_cast<FV *>(shraw);                        // [kObjWarps][W]
    int32_t *shMax = reinterpret_cast<int32_t *>(shAcc + (size_t)kObjWarps * W);   // [kObjWarps][W]
    const int l = blockIdx.y;
    const ClassDesc c = desc[l];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row0 = blockIdx.x * kObjRowsPerCta;
    if (row0 >= c.M) return;
    FV *acc = shAcc + (size_t)warp * W;
    int32_t *mx = shMax + (size_t)warp * W;
    for (int p = lane; p < W; p += 32) acc[p] = (FV)0;
    const SV *Sl = S + c.sOff;
    const int32_t *pl = perm + c.row0;
    for (int r = warp; r < kObjRowsPerCta; r += kObjWarps) {
        const int i = row0 + r;
        if (i >= c.M) break;
        for (int p = lane; p < W; p += 32) mx[p] = 0;
        __syncwarp();
        const SV *row = Sl + (int64_t)i * c.ld;
        for (int v = lane; v < c.M; v += 32) {
            const int a = assignment[pl[v]];
            if (a < 0 || a >= W) continue;
            const SV s = row[v];
            if (s > (SV)0) {
                // positive int32 and positive fp32 both order like their bit patterns
                int32_t bits;
                if constexpr (sizeof(SV) == 4 && !std::is_integral<SV>::value) bits = __float_as_int((float)s);
                else bits = (int32_t)s;
                atomicMax(&mx[a], bits);
            }
        }
        __syncwarp();
        for (int p = lane; p < W; p += 32) {
            int32_t bits = mx[p];
            FV val;
            if constexpr (!std::is_integral<SV>::value) val = (FV)__int_as_float(bits);
            else val = (FV)bits;
            acc[p] += val;
        }
        __syncwarp();
    }
    __syncthreads();
    FV *out = partial + ((int64_t)l * maxBlocks + blockIdx.x) * W;
    for (int p = threadIdx.x; p < W; p += blockDim.x) {
        FV s = (FV)0;
        for (int w = 0; w < kObjWarps; ++w) s += shAcc[(size_t)w * W + p];
        out[p] = s;
    }
}

template <typename FV>
__global__ void objective_reduce_kernel(const ClassDesc *__restrict__ desc, const FV *__restrict__ partial,
                                        int32_t L, int32_t W, int32_t maxBlocks, FV *__restrict__ partValues)
{
    int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)L * W) return;
    int l = (int)(idx / W), p = (int)(idx % W);
    int nb = (desc[l].M + kObjRowsPerCta - 1) / kObjRowsPerCta;
    FV s = (FV)0;
    for (int b = 0; b < nb; ++b) s += partial[((int64_t)l * maxBlocks + b) * W + p];
    partValues[idx] = s;
}

// one CTA, fixed strided partials then a fixed tree: reproducible
template <typename FV>
__global__ void __launch_bounds__(256, 1) objective_total_kernel(const FV *__restrict__ partValues, int64_t n,
                                                             FV *__restrict__ total)
{
    __shared__ FV sh[256];
    FV s = (FV)0;
    for (int64_t i = threadIdx.x; i < n; i += 256) s += partValues[i];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if ((int)threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) *total = sh[0];
}

template <typename SV, typename FV>
static rcd_status run_objective(rcd_ctx *ctx, const Sizes &sz, const ClassDesc *descDev,
                                const std::vector<ClassDesc> &descHost, const void *S, const int32_t *perm,
                                const int32_t *assignment, void *partValues, void *total, void *scratch,
                                cudaStream_t st)
{
    const int maxBlocks = (int)((sz.maxM + kObjRowsPerCta - 1) / kObjRowsPerCta);
    const size_t smem = (size_t)kObjWarps * sz.W * (sizeof(FV) + sizeof(int32_t));
    if ((int64_t)smem > ctx->maxSmemOptin - 1024)
        return fail(ctx, RCD_ERR_UNSUPPORTED, "W=%d needs %zu bytes of shared memory in the objective kernel", sz.W, smem);
    if (sz.L > 65535) return fail(ctx, RCD_ERR_UNSUPPORTED, "objective: more than 65535 classes");
    RCD_CUDA(ctx, cudaFuncSetAttribute(objective_rows_kernel<SV, FV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (maxBlocks > 0) {
        dim3 grid(maxBlocks, sz.L);
        objective_rows_kernel<SV, FV><<<grid, kObjWarps * 32, smem, st>>>(descDev, (const SV *)S, perm, assignment, sz.W,
                                                                         maxBlocks, (FV *)scratch);
        ctx->kernelLaunches++;
    }
    int64_t n = (int64_t)sz.L * sz.W;
    objective_reduce_kernel<FV><<<(unsigned)((n + 127) / 128), 128, 0, st>>>(descDev, (const FV *)scratch, sz.L, sz.W,
                                                                           maxBlocks, (FV *)partValues);
    objective_total_kernel<FV><<<1, 256, 0, st>>>((const FV *)partValues, n, (FV *)total);
    ctx->kernelLaunches += 2;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

rcd_status launch_objective(rcd_ctx *ctx, rcd_feat_dtype dtype, const Sizes &sz, const ClassDesc *descDev,
                            const std::vector<ClassDesc> &descHost, const void *S, const int32_t *perm,
                            const int32_t *assignment, void *partValues, void *total, void *scratch,
                            cudaStream_t st)
{
    if (dtype == RCD_FEAT_I8)
        return run_objective<int32_t, long long>(ctx, sz, descDev, descHost, S, perm, assignment, partValues, total, scratch, st);
    return run_objective<float, double>(ctx, sz, descDev, descHost, S, perm, assignment, partValues, total, scratch, st);
}

}  // namespace rcd
