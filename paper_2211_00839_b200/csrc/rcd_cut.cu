// Algorithm 1 with the graph-cut objective of Section 4, item 2:
//     f(A) = sum_{v in V_l \ A} sum_{v' in A} S[v][v'].
// With S symmetric and tie_p[u] = sum_{a in A_p} S[u][a],
//     f(A_p u {u}) - f(A_p) = (sum_v S[v][u] - S[u][u]) - 2 tie_p[u] = base[u] - 2 tie_p[u],
// so a pick needs no pass over S at all: an argmax over M values, then tie_p += row v* of S.
// One CTA per class runs the class to completion (classes are independent); the whole objective
// costs O(M) per pick.  Values: int64 for int8 features (exact), double otherwise.
// The objective is not monotone (a sample that joins A stops being cut), gains may be negative;
// Algorithm 1 runs unchanged: least-f non-full block, argmax with lowest-index ties.
#include "rcd_internal.h"

#include <limits.h>
#include <type_traits>

namespace rcd {

constexpr int kCutThreads = 512;
constexpr int kCutMaxBlocks = 1024;

template <typename SV> struct CutArith { using FV = double; };
template <> struct CutArith<int32_t> { using FV = long long; };

template <typename SV>
struct CutParams {
    using FV = typename CutArith<SV>::FV;
    const ClassDesc *desc;
    const SV *S;
    FV *tie;            // [sum W*ld] tie_p[u]
    FV *base;           // [N]        column sum minus the diagonal entry, class-sorted order
    FV *fval;           // [L][W]
    const int32_t *quota;
    int32_t *pos;       // [N] >= 0 while the sample is unassigned
    const int32_t *perm;
    int32_t *assignment;
    int32_t *order;     // may be null
    int32_t *status;
    int32_t L, W;
};

template <typename SV>
__global__ void __launch_bounds__(kCutThreads, 2) cut_chain_kernel(CutParams<SV> prm)
{
    using FV = typename CutArith<SV>::FV;
    __shared__ FV shF[kCutMaxBlocks];
    __shared__ int32_t shRoom[kCutMaxBlocks];
    __shared__ unsigned long long shG[kCutThreads / 32];      // order-preserving images of the warps' best gains
    __shared__ int shV[kCutThreads / 32];
    __shared__ int shPick, shBlock;
    const int l = blockIdx.x;
    const ClassDesc c = prm.desc[l];
    const int W = prm.W;
    if (c.M == 0) {                                           // empty class: every block has value 0
        for (int p = threadIdx.x; p < W; p += kCutThreads) prm.fval[(int64_t)l * W + p] = 0;
        return;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const SV *Sl = prm.S + c.sOff;
    FV *base = prm.base + c.row0;
    FV *tie = prm.tie + c.vOff;
    int32_t *pos = prm.pos + c.row0;

    // base[u] = sum_v S[v][u] - S[u][u]  (row sum of the symmetric S, one warp per row, lanes in fixed order)
    for (int u = warp; u < c.M; u += kCutThreads / 32) {
        const SV *row = Sl + (int64_t)u * c.ld;
        FV acc = 0;
        for (int j = lane; j < c.M; j += 32) acc += (FV)row[j];
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) base[u] = acc - (FV)row[u];
    }
    for (int64_t i = threadIdx.x; i < (int64_t)W * c.ld; i += kCutThreads) tie[i] = 0;
    for (int u = threadIdx.x; u < c.M; u += kCutThreads) pos[u] = u;
    for (int p = threadIdx.x; p < W; p += kCutThreads) { shF[p] = 0; shRoom[p] = prm.quota[(int64_t)l * W + p]; }
    __syncthreads();

    for (int t = 0; t < c.M; ++t) {
        // j* = argmin over non-full blocks of f, ties -> lowest index
        if (warp == 0) {
            FV bestF = 0;
            int bestP = INT_MAX;
            for (int p = lane; p < W; p += 32)
                if (shRoom[p] > 0 && (bestP == INT_MAX || shF[p] < bestF)) { bestF = shF[p]; bestP = p; }
            // (three warp-wide reductions on an order-preserving image of f: least f, lowest index among equals)
            unsigned long long of = ordered_u64(bestF);
            warp_argmin_ordered(of, bestP);
            if (lane == 0) shBlock = bestP;
        }
        __syncthreads();
        const int j = shBlock;
        if (j == INT_MAX) {                                   // samples left but every block is full
            if (threadIdx.x == 0) atomicOr(prm.status, kDevNoCandidate);
            return;
        }
        // v* = argmax over the unassigned samples of base[u] - 2 tie_j[u], ties -> lowest index
        const FV *tj = tie + (int64_t)j * c.ld;
        FV bestG = 0;
        int bestV = INT_MAX;
#pragma unroll 4
        for (int u = threadIdx.x; u < c.M; u += kCutThreads) {
            const FV g = base[u] - 2 * tj[u];
            if (pos[u] >= 0 && (bestV == INT_MAX || g > bestG)) { bestG = g; bestV = u; }
        }
        // greatest gain, lowest index among equals: over the warp, then over the warps' results
        unsigned long long og = ordered_u64(bestG);
        warp_argmax_ordered(og, bestV);
        if (lane == 0) { shG[warp] = og; shV[warp] = bestV; }
        __syncthreads();
        if (warp == 0) {
            og = lane < kCutThreads / 32 ? shG[lane] : 0ull;
            bestV = lane < kCutThreads / 32 ? shV[lane] : INT_MAX;
            warp_argmax_ordered(og, bestV);
            if constexpr (std::is_same<FV, double>::value) bestG = from_ordered_u64_d(og);
            else bestG = from_ordered_u64_ll(og);
            if (lane == 0) {
                shPick = bestV;
                if (bestV != INT_MAX) {
                    shF[j] += bestG;
                    shRoom[j] -= 1;
                    pos[bestV] = -1;
                    const int global = prm.perm[c.row0 + bestV];
                    prm.assignment[global] = j;
                    if (prm.order) prm.order[c.row0 + t] = global;
                }
            }
        }
        __syncthreads();
        const int vstar = shPick;
        if (vstar == INT_MAX) {
            if (threadIdx.x == 0) atomicOr(prm.status, kDevBadState);
            return;
        }
        // tie_j[u] += S[v*][u]
        {
            FV *tw = tie + (int64_t)j * c.ld;
            const SV *row = Sl + (int64_t)vstar * c.ld;
            for (int u = threadIdx.x; u < c.M; u += kCutThreads) tw[u] += (FV)row[u];
        }
        __syncthreads();
    }
    for (int p = threadIdx.x; p < W; p += kCutThreads) prm.fval[(int64_t)l * W + p] = shF[p];
}

// f(A_p) for every block from the definition: per row v the sums r_p(v) = sum_{a in A_p} S[v][a], then
// f_p += r_p(v) for every block p that v is not in.  int64 sums are exact; fp64 sums inside a row are
// accumulated with shared-memory atomics, so their last bits can differ from run to run.
template <typename SV>
__global__ void __launch_bounds__(256, 4) cut_objective_rows_kernel(const ClassDesc *__restrict__ desc, const SV *__restrict__ S,
                                                                   const int32_t *__restrict__ perm,
                                                                   const int32_t *__restrict__ assignment, int32_t W,
                                                                   int32_t maxBlocks,
                                                                   typename CutArith<SV>::FV *__restrict__ partial)
{
    using FV = typename CutArith<SV>::FV;
    using AT = typename std::conditional<std::is_integral<SV>::value, unsigned long long, double>::type;
    extern __shared__ unsigned char shraw[];
    AT *shSum = reinterpret_cast<AT *>(shraw);                  // [8 warps][W] block totals of this CTA's rows
    AT *shRow = shSum + (size_t)8 * W;                          // [8 warps][W] sums of the current row
    const int l = blockIdx.y;
    const ClassDesc c = desc[l];
    const int first = blockIdx.x * 64;
    if (first >= c.M) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    AT *sum = shSum + (size_t)warp * W, *cur = shRow + (size_t)warp * W;
    for (int p = lane; p < W; p += 32) sum[p] = 0;
    const int32_t *pl = perm + c.row0;
    for (int r = warp; r < 64; r += 8) {
        const int v = first + r;
        if (v >= c.M) break;
        for (int p = lane; p < W; p += 32) cur[p] = 0;
        __syncwarp();
        const SV *row = S + c.sOff + (int64_t)v * c.ld;
        for (int a = lane; a < c.M; a += 32) {
            const int p = assignment[pl[a]];
            if (p >= 0 && p < W) atomicAdd(&cur[p], (AT)(FV)row[a]);       // int64 wraps like two's complement
        }
        __syncwarp();
        const int mine = assignment[pl[v]];
        for (int p = lane; p < W; p += 32) if (p != mine) sum[p] += cur[p];
        __syncwarp();
    }
    __syncthreads();
    FV *out = partial + ((int64_t)l * maxBlocks + blockIdx.x) * W;
    for (int p = threadIdx.x; p < W; p += blockDim.x) {
        AT s = 0;
        for (int w = 0; w < 8; ++w) s += shSum[(size_t)w * W + p];
        out[p] = (FV)s;
    }
}

template <typename FV>
__global__ void cut_objective_reduce_kernel(const ClassDesc *__restrict__ desc, const FV *__restrict__ partial, int32_t L,
                                            int32_t W, int32_t maxBlocks, FV *__restrict__ partValues)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)L * W) return;
    const int l = (int)(idx / W), p = (int)(idx % W);
    const int nb = (desc[l].M + 63) / 64;
    FV s = 0;
    for (int b = 0; b < nb; ++b) s += partial[((int64_t)l * maxBlocks + b) * W + p];
    partValues[idx] = s;
}

template <typename FV>
__global__ void __launch_bounds__(256, 1) cut_objective_total_kernel(const FV *__restrict__ partValues, int64_t n, FV *__restrict__ total)
{
    __shared__ FV sh[256];
    FV s = 0;
    for (int64_t i = threadIdx.x; i < n; i += 256) s += partValues[i];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if ((int)threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) *total = sh[0];
}

template <typename SV>
static rcd_status run_cut(rcd_ctx *ctx, const Sizes &sz, const Workspace &ws, int32_t *assignment, int32_t *order, cudaStream_t st)
{
    using FV = typename CutArith<SV>::FV;
    if (sz.W > kCutMaxBlocks) return fail(ctx, RCD_ERR_UNSUPPORTED, "graph cut: at most %d blocks", kCutMaxBlocks);
    CutParams<SV> prm;
    prm.desc = ws.desc;
    prm.S = (const SV *)ws.S;
    prm.tie = (FV *)ws.gains;
    prm.base = (FV *)ws.cutBase;
    prm.fval = (FV *)ws.fval;
    prm.quota = ws.quota;
    prm.pos = ws.pos;
    prm.perm = ws.perm;
    prm.assignment = assignment;
    prm.order = order;
    prm.status = ws.status;
    prm.L = sz.L;
    prm.W = sz.W;
    cut_chain_kernel<SV><<<sz.L, kCutThreads, 0, st>>>(prm);
    ctx->kernelLaunches++;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

rcd_status launch_cut(rcd_ctx *ctx, const Sizes &sz, const Workspace &ws, int32_t *assignment, int32_t *order, cudaStream_t st)
{
    if (sz.L == 0 || sz.maxM == 0) return RCD_OK;
    if (sz.floatArith) return run_cut<float>(ctx, sz, ws, assignment, order, st);
    return run_cut<int32_t>(ctx, sz, ws, assignment, order, st);
}

template <typename SV>
static rcd_status run_cut_objective(rcd_ctx *ctx, const Sizes &sz, const ClassDesc *descDev, const void *S, const int32_t *perm,
                                    const int32_t *assignment, void *partValues, void *total, void *scratch, cudaStream_t st)
{
    using FV = typename CutArith<SV>::FV;
    const int maxBlocks = (int)((sz.maxM + 63) / 64);
    const size_t smem = (size_t)16 * sz.W * 8;
    if ((int64_t)smem > ctx->maxSmemOptin - 1024) return fail(ctx, RCD_ERR_UNSUPPORTED, "W=%d too large for the cut objective kernel", sz.W);
    if (sz.L > 65535) return fail(ctx, RCD_ERR_UNSUPPORTED, "objective: more than 65535 classes");
    RCD_CUDA(ctx, cudaFuncSetAttribute(cut_objective_rows_kernel<SV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (maxBlocks > 0) {
        dim3 grid(maxBlocks, sz.L);
        cut_objective_rows_kernel<SV><<<grid, 256, smem, st>>>(descDev, (const SV *)S, perm, assignment, sz.W, maxBlocks, (FV *)scratch);
        ctx->kernelLaunches++;
    }
    const int64_t n = (int64_t)sz.L * sz.W;
    cut_objective_reduce_kernel<FV><<<(unsigned)((n + 127) / 128), 128, 0, st>>>(descDev, (const FV *)scratch, sz.L, sz.W, maxBlocks, (FV *)partValues);
    cut_objective_total_kernel<FV><<<1, 256, 0, st>>>((const FV *)partValues, n, (FV *)total);
    ctx->kernelLaunches += 2;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

rcd_status launch_cut_objective(rcd_ctx *ctx, const Sizes &sz, const ClassDesc *descDev, const void *S, const int32_t *perm,
                                const int32_t *assignment, void *partValues, void *total, void *scratch, cudaStream_t st)
{
    if (sz.floatArith) return run_cut_objective<float>(ctx, sz, descDev, S, perm, assignment, partValues, total, scratch, st);
    return run_cut_objective<int32_t>(ctx, sz, descDev, S, perm, assignment, partValues, total, scratch, st);
}

}  // namespace rcd
