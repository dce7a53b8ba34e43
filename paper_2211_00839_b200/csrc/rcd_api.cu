// Host side of the C ABI: argument checks, workspace layout, quotas, and the order in which the
// kernels of the other translation units are enqueued.
#include "rcd_internal.h"

#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>

namespace rcd {

rcd_status fail(rcd_ctx *ctx, rcd_status st, const char *fmt, ...)
{
    if (ctx) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        ctx->err = buf;
    }
    return st;
}

rcd_status cuda_fail(rcd_ctx *ctx, cudaError_t e, const char *what)
{
    return fail(ctx, RCD_ERR_CUDA, "CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
}

// Device-side errors of a call are collected in a status word inside the caller's workspace (the kernels'
// target, ctx->statusDev) and copied into the context's own word when the call has enqueued its last kernel:
// rcd_sync_status reads only the context's word, so it never touches a workspace the caller may have freed.
static cudaError_t status_begin(rcd_ctx *ctx, cudaStream_t st)
{
    ctx->statusDev = ctx->statusOwn;
    return cudaMemsetAsync(ctx->statusOwn, 0, sizeof(int32_t), st);
}
static cudaError_t status_publish(rcd_ctx *ctx, cudaStream_t st)
{
    cudaError_t e = cudaSuccess;
    if (ctx->statusDev && ctx->statusDev != ctx->statusOwn)
        e = cudaMemcpyAsync(ctx->statusOwn, ctx->statusDev, sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    ctx->statusDev = ctx->statusOwn;
    return e;
}

// Bump allocator over the caller's workspace.
struct Carver {
    unsigned char *base;
    size_t off = 0;
    template <typename T> T *take(size_t count)
    {
        off = align_up(off);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += count * sizeof(T);
        return p;
    }
};

size_t layout_workspace(void *base, rcd_feat_dtype dtype, const Sizes &sz, Workspace *ws)
{
    Carver c{static_cast<unsigned char *>(base)};
    const size_t L = (size_t)std::max<int32_t>(sz.L, 1), W = (size_t)std::max<int32_t>(sz.W, 1);
    const size_t N = (size_t)std::max<int64_t>(sz.N, 1);
    const size_t sElem = 4;                                     // int32 / fp32
    const size_t gElem = (sz.floatArith && !sz.graphCut) ? 4 : 8;   // fp32 gains / int64 gains, or 8-byte ties
    Workspace w{};
    // the head does not depend on the class sizes: it is used before they are known
    w.status = c.take<int32_t>(4);
    w.counts = c.take<int32_t>(L);
    w.nSweep = c.take<int32_t>(4);
    // everything below is placed once the class sizes are known
    w.desc = c.take<ClassDesc>(L);
    w.tilePrefix = c.take<int32_t>(L + 1);
    w.chunkHist = c.take<int32_t>((size_t)std::max<int32_t>(sz.nChunks, 1) * L);
    w.perm = c.take<int32_t>(N);
    w.Xs = c.take<unsigned char>(N * (size_t)sz.d * feat_bytes(dtype));
    w.S = c.take<unsigned char>((size_t)std::max<int64_t>(sz.sElems, 1) * sElem);
    w.gaussNorms = c.take<int32_t>(N);
    w.gaussPartial = c.take<double>(L * (size_t)((sz.maxM + 63) / 64 + 1));
    w.gaussSigma = c.take<float>(L);
    w.gaussScale = c.take<float>(L);
    w.cutBase = c.take<unsigned char>(sz.graphCut ? N * 8 : 8);
    w.cover = c.take<unsigned char>((size_t)std::max<int64_t>(sz.vElems, 1) * sElem);
    w.gains = c.take<unsigned char>((size_t)std::max<int64_t>(sz.vElems, 1) * gElem);
    w.fval = c.take<unsigned char>(L * W * 8);
    w.cnt = c.take<int32_t>(L * W);
    w.quota = c.take<int32_t>(L * W);
    w.valid = c.take<uint8_t>(L * W);
    w.cand = c.take<int32_t>(N);
    w.pos = c.take<int32_t>(N);
    w.nR = c.take<int32_t>(L);
    w.jstar = c.take<int32_t>(L);
    w.sweepN = c.take<int32_t>(L);
    w.sweepParts = c.take<int32_t>(L * kSparseMax);
    w.sweepMode = c.take<int32_t>(L);
    w.thr = c.take<unsigned char>((size_t)std::max<int64_t>(sz.vElems / (int64_t)W, 1) * sElem + 64);
    w.hitCount = c.take<unsigned long long>(L);
    w.sparseElems = c.take<unsigned long long>(L);
    w.sparseFrom = c.take<int32_t>(L);
    w.sweepCS = c.take<int32_t>(L);
    w.rowCtr = c.take<int32_t>(L);
    w.sweepList = c.take<int32_t>(3 * L);
    w.sync = c.take<ClassSync>(L);
    w.tickets = c.take<int32_t>(N + L);
    w.sweepF = c.take<long long>(L * 8);
    w.sizesSorted = c.take<int32_t>(L);
    w.classOrder = c.take<int32_t>(L);
    w.floorv = c.take<unsigned char>(L * kLazyBlocks * 8);
    w.theta = c.take<unsigned char>(L * kLazyBlocks * 8);
    w.sweepTheta = c.take<unsigned char>(L * kLazyBlocks * 8);
    w.lazyStat = c.take<int32_t>(L * 4);
    w.stepBytes = c.take<unsigned long long>((size_t)sz.maxM + 1);
    w.stepOps = c.take<unsigned long long>((size_t)sz.maxM + 1);
    w.phaseNs = c.take<unsigned long long>(kPhaseWords);   // phase clocks, the grid-barrier counter, threshold-pass and row-skipping counters
    w.bytes = align_up(c.off);
    if (ws) *ws = w;
    return w.bytes;
}

static int32_t chunks_for(int64_t N) { return (int32_t)((N + kGroupChunk - 1) / kGroupChunk); }

// Sizes for the promise "no class larger than Mmax".
static bool float_arith(const rcd_ctx *ctx, rcd_feat_dtype dtype)
{
    return dtype == RCD_FEAT_BF16 || ctx->cfg.similarity_kind == RCD_SIM_GAUSSIAN;
}

static Sizes bound_sizes(const rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d, int32_t L, int64_t Mmax, int32_t W)
{
    Sizes sz{};
    sz.floatArith = float_arith(ctx, dtype);
    sz.graphCut = ctx->cfg.objective == RCD_OBJ_GRAPH_CUT;
    sz.N = N; sz.d = d; sz.L = L; sz.W = W;
    if (Mmax > N) Mmax = N;
    sz.maxM = Mmax;
    sz.sElems = N * (int64_t)pad_row(Mmax);               // sum M_l * ld_l <= N * pad_row(Mmax)
    sz.vElems = (int64_t)W * (N + 7LL * L);               // sum W * ld_l,  ld_l <= M_l + 7
    sz.nChunks = chunks_for(N);
    return sz;
}

static rcd_status check_common(rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d, int32_t L, int32_t W)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    if (dtype != RCD_FEAT_I8 && dtype != RCD_FEAT_BF16) return fail(ctx, RCD_ERR_INVALID_ARG, "unknown feature dtype %d", (int)dtype);
    if (N < 0 || N > 0x7fffffffLL) return fail(ctx, RCD_ERR_INVALID_ARG, "N=%lld out of range", (long long)N);
    if (d <= 0) return fail(ctx, RCD_ERR_INVALID_ARG, "d=%lld must be positive", (long long)d);
    if (L <= 0) return fail(ctx, RCD_ERR_INVALID_ARG, "L=%d must be positive", L);
    if (W <= 0) return fail(ctx, RCD_ERR_INVALID_ARG, "W=%d must be positive", W);
    if (W > 1024) return fail(ctx, RCD_ERR_UNSUPPORTED, "W=%d: at most 1024 blocks are supported", W);
    if (dtype == RCD_FEAT_I8 && 16384LL * d > 0x7fffffffLL)
        return fail(ctx, RCD_ERR_UNSUPPORTED, "d=%lld: an int8 dot product could overflow int32", (long long)d);
    return RCD_OK;
}

static rcd_status check_capacities(rcd_ctx *ctx, const double *cap, int32_t W)
{
    if (!cap) return fail(ctx, RCD_ERR_INVALID_ARG, "capacities is null");
    for (int32_t j = 0; j < W; ++j)
        if (!(cap[j] > 0.0) || !std::isfinite(cap[j]))
            return fail(ctx, RCD_ERR_INVALID_ARG, "capacity %d is not a finite positive number", j);
    return RCD_OK;
}

// Largest-remainder apportionment of M samples over W blocks (Algorithm 1's C_{l,j} = |V_l| r_j / sum r, made integer).
// Shares are formed in IEEE double in index order (sum first, then M * r_j / sum, no contraction); every block gets
// the integer part of its share, and the samples still unplaced go one each to the blocks ranked by fractional part
// (a stable sort: equal fractions keep their index order, so ties fall to the lowest index).  Should rounding ever
// make the integer parts add up to more than M (a share that rounds up onto an integer; no input found does), the
// surplus is taken back from the other end of the same ranking.
static void quotas_host(int64_t M, const double *r, int32_t W, int32_t *out)
{
    volatile double sum = 0.0;
    for (int32_t j = 0; j < W; ++j) sum = sum + r[j];
    std::vector<double> frac((size_t)W);
    std::vector<int32_t> rank((size_t)W);
    int64_t placed = 0;
    for (int32_t j = 0; j < W; ++j) {
        volatile double numerator = (double)M * r[j];
        volatile double share = numerator / sum;
        const double whole = std::floor(share);
        out[j] = (int32_t)whole;
        frac[(size_t)j] = share - whole;
        placed += (int64_t)whole;
        rank[(size_t)j] = j;
    }
    std::stable_sort(rank.begin(), rank.end(), [&](int32_t a, int32_t b) { return frac[(size_t)a] > frac[(size_t)b]; });
    int64_t left = M - placed;
    for (size_t k = 0; left > 0; k = (k + 1) % (size_t)W, --left) out[rank[k]] += 1;
    for (size_t k = (size_t)W; left < 0 && k-- > 0;)
        if (out[rank[k]] > 0) { out[rank[k]] -= 1; ++left; }
}

// Shared front half of rcd_partition and rcd_objective: class sizes, descriptors, workspace
// layout, stable split, feature gather, similarity.
struct Prepared {
    Sizes sz{};
    Workspace ws{};
    std::vector<ClassDesc> desc;
};

static rcd_status prepare(rcd_ctx *ctx, const void *features, rcd_feat_dtype dtype, int64_t N, int64_t d,
                          const int32_t *labels, int32_t L, int32_t W, void *workspace, size_t workspaceBytes,
                          cudaStream_t st, Prepared *out)
{
    if (((uintptr_t)workspace) % kAlign != 0) return fail(ctx, RCD_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    // head of the workspace: status, counts
    Sizes head{};
    head.N = N; head.d = d; head.L = L; head.W = W; head.nChunks = chunks_for(N);
    head.floatArith = float_arith(ctx, dtype);
    head.graphCut = ctx->cfg.objective == RCD_OBJ_GRAPH_CUT;
    Workspace hw{};
    Sizes tiny = head;
    layout_workspace(workspace, dtype, tiny, &hw);
    size_t headBytes = (size_t)((unsigned char *)hw.desc - (unsigned char *)workspace);
    if (workspaceBytes < headBytes) return fail(ctx, RCD_ERR_WORKSPACE_TOO_SMALL, "workspace smaller than its %zu-byte head", headBytes);
    if ((size_t)L > ctx->hostStageInts) return fail(ctx, RCD_ERR_UNSUPPORTED, "L=%d exceeds the %zu classes the context can stage", L, ctx->hostStageInts);

    RCD_CUDA(ctx, cudaMemsetAsync(hw.status, 0, 4 * sizeof(int32_t), st));
    RCD_CUDA(ctx, cudaMemsetAsync(hw.counts, 0, (size_t)L * sizeof(int32_t), st));
    rcd_status rs = launch_count_labels(ctx, labels, N, L, hw.counts, hw.status, st);
    if (rs != RCD_OK) return rs;
    RCD_CUDA(ctx, cudaMemcpyAsync(ctx->hostStage, hw.counts, (size_t)L * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    RCD_CUDA(ctx, cudaMemcpyAsync(ctx->hostStage + L, hw.status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    RCD_CUDA(ctx, cudaStreamSynchronize(st));
    if (ctx->hostStage[L] & kDevBadLabel) return fail(ctx, RCD_ERR_INVALID_ARG, "a label lies outside [0, %d)", L);

    Prepared &P = *out;
    P.desc.resize((size_t)L);
    Sizes sz = head;
    int64_t row = 0, sOff = 0, vOff = 0, maxM = 0;
    for (int32_t l = 0; l < L; ++l) {
        ClassDesc c{};
        c.M = ctx->hostStage[l];
        c.ld = pad_row(c.M);
        c.row0 = (int32_t)row;
        c.sOff = sOff;
        c.vOff = vOff;
        row += c.M;
        sOff += (int64_t)c.M * c.ld;
        vOff += (int64_t)W * c.ld;
        maxM = std::max<int64_t>(maxM, c.M);
        P.desc[(size_t)l] = c;
    }
    if (row != N) return fail(ctx, RCD_ERR_INTERNAL, "class sizes sum to %lld, expected %lld", (long long)row, (long long)N);
    sz.sElems = sOff; sz.vElems = vOff; sz.maxM = maxM;
    size_t need = layout_workspace(workspace, dtype, sz, &P.ws);
    if (need > workspaceBytes)
        return fail(ctx, RCD_ERR_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, the class sizes found need %zu", workspaceBytes, need);
    P.sz = sz;
    ctx->statusDev = P.ws.status;

    RCD_CUDA(ctx, cudaMemcpyAsync(P.ws.desc, P.desc.data(), (size_t)L * sizeof(ClassDesc), cudaMemcpyHostToDevice, st));
    rs = launch_stable_split(ctx, labels, N, L, sz.nChunks, P.ws.chunkHist, P.ws.desc, P.ws.perm, st);
    if (rs != RCD_OK) return rs;
    rs = launch_gather_rows(ctx, features, P.ws.perm, N, d * (int64_t)feat_bytes(dtype), P.ws.Xs, st);
    if (rs != RCD_OK) return rs;
    if (ctx->cfg.profile >= 1) RCD_CUDA(ctx, cudaEventRecord(ctx->evPhase[1], st));
    SimClasses cls{};
    cls.src.table = P.ws.desc;
    cls.L = L;
    cls.maxM = maxM;
    {
        std::vector<int32_t> prefix((size_t)L + 1);
        int64_t run = 0;
        for (int32_t l = 0; l < L; ++l) {
            prefix[(size_t)l] = (int32_t)run;
            run += sim_tiles(P.desc[(size_t)l].M);
            if (run > 0x7fffffffLL) return fail(ctx, RCD_ERR_UNSUPPORTED, "too many similarity tiles");
        }
        prefix[(size_t)L] = (int32_t)run;
        cls.upperTiles = run;
        cls.tilePrefixDev = P.ws.tilePrefix;
        RCD_CUDA(ctx, cudaMemcpyAsync(P.ws.tilePrefix, prefix.data(), prefix.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    }
    rs = launch_similarity(ctx, P.ws.Xs, dtype, N, d, cls, P.ws.S, st);
    if (rs != RCD_OK) return rs;
    if (ctx->cfg.similarity_kind == RCD_SIM_GAUSSIAN) {
        rs = launch_gaussian(ctx, P.ws.Xs, dtype, N, d, cls, P.ws.S, P.ws.gaussNorms, P.ws.gaussPartial, P.ws.gaussSigma,
                             P.ws.gaussScale, st);
        if (rs != RCD_OK) return rs;
    }
    if (ctx->cfg.profile >= 1) RCD_CUDA(ctx, cudaEventRecord(ctx->evPhase[2], st));
    return RCD_OK;
}

}  // namespace rcd

using namespace rcd;

extern "C" {

const char *rcd_version(void) { return "rcd-b200 0.1 (sm_100a)"; }

const char *rcd_last_error(const rcd_ctx *ctx) { return ctx ? ctx->err.c_str() : ""; }

rcd_status rcd_create(rcd_ctx **out, int cuda_device, const rcd_config *cfg)
{
    if (!out) return RCD_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg) {
        if (cfg->sweep_batch_max != 0 && cfg->sweep_batch_max != 1 && cfg->sweep_batch_max != 2 &&
            cfg->sweep_batch_max != 4 && cfg->sweep_batch_max != 8)
            return RCD_ERR_INVALID_ARG;
        if (cfg->similarity_path != 0 && cfg->similarity_path != 2) return RCD_ERR_INVALID_ARG;
        if (cfg->profile < 0 || cfg->profile > 2) return RCD_ERR_INVALID_ARG;
        if (cfg->greedy_path < 0 || cfg->greedy_path > 4) return RCD_ERR_INVALID_ARG;
        if (cfg->similarity_kind != RCD_SIM_DOT && cfg->similarity_kind != RCD_SIM_GAUSSIAN) return RCD_ERR_INVALID_ARG;
        if (cfg->objective != RCD_OBJ_FACILITY && cfg->objective != RCD_OBJ_GRAPH_CUT) return RCD_ERR_INVALID_ARG;
        if (cfg->sweep_mode != 0 && cfg->sweep_mode != 1) return RCD_ERR_INVALID_ARG;
        if (cfg->async_group < 0 || cfg->async_group > 4096) return RCD_ERR_INVALID_ARG;
        if (cfg->async_help_min < 0) return RCD_ERR_INVALID_ARG;
        if (cfg->threshold_from < 0 || cfg->threshold_hit_shift < 0 || cfg->threshold_hit_shift > 30) return RCD_ERR_INVALID_ARG;
        if (cfg->lazy_mode != 0 && cfg->lazy_mode != 1) return RCD_ERR_INVALID_ARG;
        if (cfg->lazy_from < 0) return RCD_ERR_INVALID_ARG;
        if (cfg->dense_ring != 0 && cfg->dense_ring != 2) return RCD_ERR_INVALID_ARG;
        if (cfg->incremental < 0 || cfg->incremental > 2) return RCD_ERR_INVALID_ARG;
        if (cfg->incremental_max < 0 || cfg->incremental_max > 128) return RCD_ERR_INVALID_ARG;
    }
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || cuda_device < 0 || cuda_device >= count) {
        cudaGetLastError();
        return RCD_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cuda_device) != cudaSuccess) return RCD_ERR_CUDA;
    if (prop.major != 10) return RCD_ERR_UNSUPPORTED;     // the kernels are built for sm_100a only
    if (cudaSetDevice(cuda_device) != cudaSuccess) return RCD_ERR_CUDA;
    rcd_ctx *ctx = new (std::nothrow) rcd_ctx();
    if (!ctx) return RCD_ERR_INTERNAL;
    ctx->device = cuda_device;
    ctx->smCount = prop.multiProcessorCount;
    ctx->maxSmemOptin = (int)prop.sharedMemPerBlockOptin;
    ctx->cooperative = prop.cooperativeLaunch != 0;
    if (cfg) ctx->cfg = *cfg;
    ctx->hostStageInts = 1 << 20;
    if (cudaMallocHost((void **)&ctx->hostStage, (ctx->hostStageInts + 16) * sizeof(int32_t)) != cudaSuccess) {
        delete ctx;
        return RCD_ERR_CUDA;
    }
    if (cudaMalloc((void **)&ctx->statusOwn, 256) != cudaSuccess || cudaMemset(ctx->statusOwn, 0, 256) != cudaSuccess) {
        rcd_destroy(ctx);
        return RCD_ERR_CUDA;
    }
    for (auto &e : ctx->evPhase)
        if (cudaEventCreate(&e) != cudaSuccess) { rcd_destroy(ctx); return RCD_ERR_CUDA; }
    *out = ctx;
    return RCD_OK;
}

void rcd_destroy(rcd_ctx *ctx)
{
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    for (auto &e : ctx->evPhase) if (e) cudaEventDestroy(e);
    for (auto &e : ctx->evSweep) cudaEventDestroy(e);
    if (ctx->hostStage) cudaFreeHost(ctx->hostStage);
    if (ctx->statusOwn) cudaFree(ctx->statusOwn);
    delete ctx;
}

rcd_status rcd_sync_status(rcd_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaStreamSynchronize(st));
    int32_t word = 0;
    RCD_CUDA(ctx, cudaMemcpy(&word, ctx->statusOwn, sizeof word, cudaMemcpyDeviceToHost));
    if (word == 0) return RCD_OK;
    if (word & kDevBadLabel) return fail(ctx, RCD_ERR_INVALID_ARG, "device status %d: label out of range", word);
    if (word & kDevTimeout) return fail(ctx, RCD_ERR_TIMEOUT, "device status %d: a bounded wait inside a kernel ran out", word);
    return fail(ctx, RCD_ERR_INTERNAL, "device status %d: greedy state inconsistent", word);
}

rcd_status rcd_selftest_bounded_wait(rcd_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    RCD_CUDA(ctx, cudaMemsetAsync(ctx->statusOwn, 0, 64, st));
    ctx->statusDev = ctx->statusOwn;
    return launch_bounded_wait_selftest(ctx, (unsigned *)(ctx->statusOwn + 8), ctx->statusOwn, st);
}

rcd_status rcd_get_profile(rcd_ctx *ctx, rcd_profile *out)
{
    if (!ctx || !out) return RCD_ERR_INVALID_ARG;
    memset(out, 0, sizeof *out);
    out->kernel_launches = ctx->kernelLaunches;
    out->steps = ctx->steps;
    out->similarity_tc_launches = ctx->tcLaunches;
    if (!ctx->phaseValid) return RCD_OK;
    RCD_CUDA(ctx, cudaEventSynchronize(ctx->evPhase[4]));
    float ms = 0.f;
    int64_t lazyBytes = 0;      // bytes of the rows read by row-skipping passes (counted as they are read)
    RCD_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->evPhase[0], ctx->evPhase[4])); out->total_ms = ms;
    RCD_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->evPhase[0], ctx->evPhase[1])); out->group_ms = ms;
    RCD_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->evPhase[1], ctx->evPhase[2])); out->similarity_ms = ms;
    RCD_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->evPhase[2], ctx->evPhase[3])); out->greedy_ms = ms;
    if (ctx->phaseNsDev) {
        unsigned long long ns[kPhaseWords] = {};
        RCD_CUDA(ctx, cudaMemcpy(ns, ctx->phaseNsDev, sizeof ns, cudaMemcpyDeviceToHost));
        out->lazy_sweeps = (int64_t)ns[8];
        out->lazy_misses = (int64_t)ns[9];
        out->lazy_rows = (int64_t)ns[10];
        out->lazy_rows_skipped = (int64_t)ns[11];
        lazyBytes = (int64_t)ns[12];
        out->incremental_updates = (int64_t)ns[15];
        out->incremental_rows = (int64_t)ns[16];
        out->noted_picks = (int64_t)ns[17];
        out->threshold_pass_ns = (int64_t)ns[13];
        out->threshold_pass_bytes = (int64_t)ns[14];
        out->persistent_sweep_ns = (int64_t)ns[0];
        out->persistent_pick_ns = (int64_t)ns[1];
        out->threshold_hits = (int64_t)ns[3];
        out->threshold_elems = (int64_t)ns[4];
        out->threshold_max_blocks = (int64_t)ns[5];
        out->async_lull_ns = (int64_t)ns[6];
        out->async_visits = (int64_t)(ns[7] & 0xffffffffull);
        out->async_attempts = (int64_t)(ns[7] >> 32);
    }
    if (ctx->stepBytesDev && ctx->steps > 0) {
        std::vector<unsigned long long> bytes((size_t)ctx->steps + 1), ops((size_t)ctx->steps + 1);
        RCD_CUDA(ctx, cudaMemcpy(bytes.data(), ctx->stepBytesDev, bytes.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
        RCD_CUDA(ctx, cudaMemcpy(ops.data(), ctx->stepOpsDev, ops.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
        for (int64_t t = 0; t < ctx->steps; ++t) {
            if (bytes[(size_t)t] == 0) continue;
            out->sweep_bytes += (int64_t)bytes[(size_t)t];
            out->sweep_elem_ops += (int64_t)ops[(size_t)t];
            out->sweep_launches += 1;
            if (ctx->sweepEventsUsed >= 2 * (t + 1)) {
                RCD_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->evSweep[(size_t)(2 * t)], ctx->evSweep[(size_t)(2 * t + 1)]));
                out->sweep_ms += ms;
            }
        }
        out->sweep_bytes += lazyBytes;
    }
    return RCD_OK;
}

rcd_status rcd_quotas(int64_t M, const double *capacities_host, int32_t W, int32_t *quotas_host_out)
{
    if (M < 0 || M > 0x7fffffffLL || W <= 0 || !capacities_host || !quotas_host_out) return RCD_ERR_INVALID_ARG;
    for (int32_t j = 0; j < W; ++j)
        if (!(capacities_host[j] > 0.0) || !std::isfinite(capacities_host[j])) return RCD_ERR_INVALID_ARG;
    quotas_host(M, capacities_host, W, quotas_host_out);
    return RCD_OK;
}

// ---- downstream hook: per-worker index lists and batch sizes (Algorithm 2, initialisation) ----

struct ListsWorkspace {
    int32_t *status;      // [4]
    int32_t *counts;      // [W]
    ClassDesc *desc;      // [W] (only row0 is used: where a worker's list starts)
    int32_t *chunkHist;   // [nChunks][W]
    size_t bytes;
};

static size_t layout_lists(void *base, int64_t N, int32_t W, ListsWorkspace *out)
{
    Carver c{static_cast<unsigned char *>(base)};
    ListsWorkspace w{};
    const size_t Wn = (size_t)std::max<int32_t>(W, 1);
    w.status = c.take<int32_t>(4);
    w.counts = c.take<int32_t>(Wn);
    w.desc = c.take<ClassDesc>(Wn);
    w.chunkHist = c.take<int32_t>((size_t)std::max<int32_t>(chunks_for(N), 1) * Wn);
    w.bytes = align_up(c.off);
    if (out) *out = w;
    return w.bytes;
}

rcd_status rcd_worker_lists_workspace_bytes(rcd_ctx *ctx, int64_t N, int32_t W, size_t *bytes_out)
{
    if (!ctx || !bytes_out) return RCD_ERR_INVALID_ARG;
    if (N < 0 || N > 0x7fffffffLL || W <= 0) return fail(ctx, RCD_ERR_INVALID_ARG, "N=%lld or W=%d out of range", (long long)N, W);
    *bytes_out = layout_lists(nullptr, N, W, nullptr);
    return RCD_OK;
}

rcd_status rcd_worker_lists(rcd_ctx *ctx, const int32_t *assignment_dev, int64_t N, int32_t W, int64_t *offsets_dev,
                            int32_t *indices_dev, void *workspace_dev, size_t workspace_bytes, void *cuda_stream)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    if (N < 0 || N > 0x7fffffffLL || W <= 0) return fail(ctx, RCD_ERR_INVALID_ARG, "N=%lld or W=%d out of range", (long long)N, W);
    if (!offsets_dev || !workspace_dev || (N > 0 && (!assignment_dev || !indices_dev))) return fail(ctx, RCD_ERR_INVALID_ARG, "null device pointer");
    if (((uintptr_t)workspace_dev) % kAlign != 0) return fail(ctx, RCD_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    if ((size_t)W + 1 > ctx->hostStageInts) return fail(ctx, RCD_ERR_UNSUPPORTED, "W=%d exceeds the %zu blocks the context can stage", W, ctx->hostStageInts);
    ListsWorkspace ws{};
    const size_t need = layout_lists(workspace_dev, N, W, &ws);
    if (workspace_bytes < need) return fail(ctx, RCD_ERR_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    ctx->kernelLaunches = 0;
    RCD_CUDA(ctx, status_begin(ctx, st));
    ctx->statusDev = ws.status;
    RCD_CUDA(ctx, cudaMemsetAsync(ws.status, 0, 4 * sizeof(int32_t), st));
    RCD_CUDA(ctx, cudaMemsetAsync(ws.counts, 0, (size_t)W * sizeof(int32_t), st));
    // sizes of the lists (a histogram of the block numbers), read back: they fix where each list starts
    rcd_status rs = launch_count_labels(ctx, assignment_dev, N, W, ws.counts, ws.status, st);
    if (rs != RCD_OK) return rs;
    RCD_CUDA(ctx, cudaMemcpyAsync(ctx->hostStage, ws.counts, (size_t)W * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    RCD_CUDA(ctx, cudaMemcpyAsync(ctx->hostStage + W, ws.status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    RCD_CUDA(ctx, cudaStreamSynchronize(st));
    if (ctx->hostStage[W] & kDevBadLabel) return fail(ctx, RCD_ERR_INVALID_ARG, "an assignment entry lies outside [0, %d)", W);
    std::vector<ClassDesc> desc((size_t)W);
    std::vector<int64_t> offsets((size_t)W + 1);
    int64_t run = 0;
    for (int32_t j = 0; j < W; ++j) {
        ClassDesc c{};
        c.M = ctx->hostStage[j];
        c.row0 = (int32_t)run;
        desc[(size_t)j] = c;
        offsets[(size_t)j] = run;
        run += c.M;
    }
    offsets[(size_t)W] = run;
    if (run != N) return fail(ctx, RCD_ERR_INTERNAL, "list sizes sum to %lld, expected %lld", (long long)run, (long long)N);
    // (pageable host memory: the runtime stages these copies before it returns)
    RCD_CUDA(ctx, cudaMemcpyAsync(offsets_dev, offsets.data(), offsets.size() * sizeof(int64_t), cudaMemcpyHostToDevice, st));
    RCD_CUDA(ctx, cudaMemcpyAsync(ws.desc, desc.data(), desc.size() * sizeof(ClassDesc), cudaMemcpyHostToDevice, st));
    // a stable split by block number: inside a list the dataset indices ascend
    rs = launch_stable_split(ctx, assignment_dev, N, W, chunks_for(N), ws.chunkHist, ws.desc, indices_dev, st);
    if (rs != RCD_OK) return rs;
    RCD_CUDA(ctx, status_publish(ctx, st));
    return RCD_OK;
}

rcd_status rcd_batch_sizes_rule(int64_t B, const double *capacities_host, int32_t W, rcd_batch_rule rule, int64_t *batch_sizes_host_out)
{
    if (B <= 0 || W <= 0 || !capacities_host || !batch_sizes_host_out) return RCD_ERR_INVALID_ARG;
    if (rule != RCD_BATCH_PROPORTIONAL && rule != RCD_BATCH_AS_PRINTED) return RCD_ERR_INVALID_ARG;
    for (int32_t j = 0; j < W; ++j)
        if (!(capacities_host[j] > 0.0) || !std::isfinite(capacities_host[j])) return RCD_ERR_INVALID_ARG;
    for (int32_t j = 0; j < W; ++j) {
        const double x = rule == RCD_BATCH_PROPORTIONAL ? (double)B * capacities_host[j] / capacities_host[0]
                                                        : (double)B * capacities_host[0] / capacities_host[j];
        if (!(x < 9.0e18)) return RCD_ERR_INVALID_ARG;
        const int64_t b = (int64_t)std::floor(x + 0.5);
        batch_sizes_host_out[j] = b < 1 ? 1 : b;
    }
    return RCD_OK;
}

rcd_status rcd_batch_sizes(int64_t B, const double *capacities_host, int32_t W, int64_t *batch_sizes_host_out)
{
    return rcd_batch_sizes_rule(B, capacities_host, W, RCD_BATCH_PROPORTIONAL, batch_sizes_host_out);
}

rcd_status rcd_similarity(rcd_ctx *ctx, const void *X_dev, rcd_feat_dtype dtype, int64_t M, int64_t d,
                          int64_t batch, void *S_dev, int64_t ldS, void *cuda_stream)
{
    rcd_status rs = check_common(ctx, dtype, 0, d, 1, 1);
    if (rs != RCD_OK) return rs;
    if (M < 0 || batch < 0 || M > 0x7fffffffLL) return fail(ctx, RCD_ERR_INVALID_ARG, "M or batch negative");
    if (M == 0 || batch == 0) return RCD_OK;
    if (!X_dev || !S_dev) return fail(ctx, RCD_ERR_INVALID_ARG, "null device pointer");
    if (ldS % 4 != 0 || ldS < M || ldS > (M + 63) / 64 * 64)
        return fail(ctx, RCD_ERR_INVALID_ARG, "ldS must be a multiple of 4 in [M, M rounded up to 64] = [%lld, %lld], got %lld",
                    (long long)M, (long long)((M + 63) / 64 * 64), (long long)ldS);
    if (M * batch > 0x7fffffffLL) return fail(ctx, RCD_ERR_INVALID_ARG, "M*batch too large");
    if (((uintptr_t)X_dev) % 16 || ((uintptr_t)S_dev) % 16) return fail(ctx, RCD_ERR_INVALID_ARG, "X and S must be 16-byte aligned");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    SimClasses cls{};
    cls.src.table = nullptr;
    cls.src.uniM = (int32_t)M;
    cls.src.uniLd = (int32_t)ldS;
    cls.L = (int32_t)batch;
    cls.maxM = M;
    cls.tilePrefixDev = nullptr;
    cls.uniTiles = (int32_t)sim_tiles(M);
    cls.upperTiles = batch * (int64_t)cls.uniTiles;
    ctx->kernelLaunches = 0;
    ctx->tcLaunches = 0;
    RCD_CUDA(ctx, status_begin(ctx, st));
    return launch_similarity(ctx, X_dev, dtype, M * batch, d, cls, S_dev, st);
}

rcd_status rcd_similarity_gaussian_workspace_bytes(rcd_ctx *ctx, int64_t M, int64_t batch, size_t *bytes_out)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    if (!bytes_out || M < 0 || batch < 0 || M * batch > 0x7fffffffLL || batch > 0x7fffffffLL)
        return fail(ctx, RCD_ERR_INVALID_ARG, "bad M, batch or null output");
    *bytes_out = gaussian_scratch_bytes(M * batch, (int32_t)batch, M) + kAlign;
    return RCD_OK;
}

rcd_status rcd_similarity_gaussian(rcd_ctx *ctx, const void *X_dev, rcd_feat_dtype dtype, int64_t M, int64_t d, int64_t batch,
                                   void *S_dev, int64_t ldS, float *sigma_dev_or_null, void *workspace_dev,
                                   size_t workspace_bytes, void *cuda_stream)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    // every argument is checked before anything is launched or written
    if (M > 0 && batch > 0) {
        if (batch > 65535) return fail(ctx, RCD_ERR_UNSUPPORTED, "Gaussian similarity: more than 65535 classes");
        if (M * batch > 0x7fffffffLL) return fail(ctx, RCD_ERR_INVALID_ARG, "M*batch too large");
        if (!workspace_dev || ((uintptr_t)workspace_dev) % kAlign) return fail(ctx, RCD_ERR_INVALID_ARG, "workspace null or not 256-byte aligned");
        if (workspace_bytes < gaussian_scratch_bytes(M * batch, (int32_t)batch, M))
            return fail(ctx, RCD_ERR_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, need %zu", workspace_bytes,
                        gaussian_scratch_bytes(M * batch, (int32_t)batch, M));
    }
    rcd_status rs = rcd_similarity(ctx, X_dev, dtype, M, d, batch, S_dev, ldS, cuda_stream);
    if (rs != RCD_OK || M == 0 || batch == 0) return rs;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    unsigned char *w = (unsigned char *)workspace_dev;
    void *norms = w;                                  w += align_up((size_t)(M * batch) * 4);
    double *partial = (double *)w;                    w += align_up((size_t)batch * (size_t)((M + 63) / 64) * 8);
    float *sigma = (float *)w;                        w += align_up((size_t)batch * 4);
    float *scale = (float *)w;
    SimClasses cls{};
    cls.src.table = nullptr;
    cls.src.uniM = (int32_t)M;
    cls.src.uniLd = (int32_t)ldS;
    cls.L = (int32_t)batch;
    cls.maxM = M;
    rs = launch_gaussian(ctx, X_dev, dtype, M * batch, d, cls, S_dev, norms, partial, sigma, scale, st);
    if (rs != RCD_OK) return rs;
    if (sigma_dev_or_null)
        RCD_CUDA(ctx, cudaMemcpyAsync(sigma_dev_or_null, sigma, (size_t)batch * sizeof(float), cudaMemcpyDeviceToDevice, st));
    return RCD_OK;
}

rcd_status rcd_partition_workspace_bytes(rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d, int32_t L,
                                         int64_t M_max, int32_t W, size_t *bytes_out)
{
    rcd_status rs = check_common(ctx, dtype, N, d, L, W);
    if (rs != RCD_OK) return rs;
    if (!bytes_out || M_max < 0) return fail(ctx, RCD_ERR_INVALID_ARG, "bad M_max or null output");
    Sizes sz = bound_sizes(ctx, dtype, N, d, L, M_max, W);
    *bytes_out = layout_workspace(nullptr, dtype, sz, nullptr);
    return RCD_OK;
}

rcd_status rcd_partition(rcd_ctx *ctx, const void *features_dev, rcd_feat_dtype dtype, int64_t N, int64_t d,
                         const int32_t *labels_dev, int32_t L, const double *capacities_host, int32_t W,
                         int32_t *assignment_dev, int32_t *order_dev_or_null, void *part_values_dev_or_null,
                         void *workspace_dev, size_t workspace_bytes, void *cuda_stream)
{
    rcd_status rs = check_common(ctx, dtype, N, d, L, W);
    if (rs != RCD_OK) return rs;
    rs = check_capacities(ctx, capacities_host, W);
    if (rs != RCD_OK) return rs;
    if (N > 0 && (!features_dev || !labels_dev || !assignment_dev)) return fail(ctx, RCD_ERR_INVALID_ARG, "null device pointer");
    if (!workspace_dev) return fail(ctx, RCD_ERR_INVALID_ARG, "workspace is null");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    ctx->kernelLaunches = 0;
    ctx->tcLaunches = 0;
    ctx->steps = 0;
    ctx->phaseValid = false;
    ctx->stepBytesDev = nullptr;
    ctx->stepOpsDev = nullptr;
    ctx->phaseNsDev = nullptr;
    ctx->sweepEventsUsed = 0;
    const bool prof = ctx->cfg.profile >= 1;
    RCD_CUDA(ctx, status_begin(ctx, st));
    if (prof) RCD_CUDA(ctx, cudaEventRecord(ctx->evPhase[0], st));

    Prepared P;
    rs = prepare(ctx, features_dev, dtype, N, d, labels_dev, L, W, workspace_dev, workspace_bytes, st, &P);
    if (rs != RCD_OK) return rs;

    std::vector<int32_t> quota((size_t)L * W);
    for (int32_t l = 0; l < L; ++l) quotas_host(P.desc[(size_t)l].M, capacities_host, W, quota.data() + (size_t)l * W);
    RCD_CUDA(ctx, cudaMemcpyAsync(P.ws.quota, quota.data(), quota.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));

    if (P.sz.graphCut) rs = launch_cut(ctx, P.sz, P.ws, assignment_dev, order_dev_or_null, st);
    else rs = launch_greedy(ctx, P.sz.floatArith ? RCD_FEAT_BF16 : RCD_FEAT_I8, P.sz, P.ws, P.desc, assignment_dev, order_dev_or_null, st);
    if (rs != RCD_OK) return rs;
    if (prof) RCD_CUDA(ctx, cudaEventRecord(ctx->evPhase[3], st));
    if (part_values_dev_or_null) {
        if (P.sz.maxM == 0) RCD_CUDA(ctx, cudaMemsetAsync(part_values_dev_or_null, 0, (size_t)L * W * 8, st));
        else RCD_CUDA(ctx, cudaMemcpyAsync(part_values_dev_or_null, P.ws.fval, (size_t)L * W * 8, cudaMemcpyDeviceToDevice, st));
    }
    RCD_CUDA(ctx, status_publish(ctx, st));
    if (prof) {
        RCD_CUDA(ctx, cudaEventRecord(ctx->evPhase[4], st));
        ctx->phaseValid = true;
    }
    return RCD_OK;
}

// Host-buffer variant: staging areas for features, labels and the three outputs sit behind the
// device workspace proper.
static size_t host_tail_bytes(rcd_feat_dtype dtype, int64_t N, int64_t d, int32_t L, int32_t W)
{
    const size_t featB = align_up((size_t)std::max<int64_t>(N, 1) * (size_t)d * feat_bytes(dtype));
    const size_t vecB = align_up((size_t)std::max<int64_t>(N, 1) * 4);
    const size_t valB = align_up((size_t)L * W * 8);
    return featB + 3 * vecB + valB;
}

rcd_status rcd_partition_host_workspace_bytes(rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d, int32_t L,
                                              int64_t M_max, int32_t W, size_t *bytes_out)
{
    rcd_status rs = check_common(ctx, dtype, N, d, L, W);
    if (rs != RCD_OK) return rs;
    if (!bytes_out || M_max < 0) return fail(ctx, RCD_ERR_INVALID_ARG, "bad M_max or null output");
    Sizes sz = bound_sizes(ctx, dtype, N, d, L, M_max, W);
    *bytes_out = layout_workspace(nullptr, dtype, sz, nullptr) + host_tail_bytes(dtype, N, d, L, W) + kAlign;
    return RCD_OK;
}

rcd_status rcd_partition_host(rcd_ctx *ctx, const void *features_host, rcd_feat_dtype dtype, int64_t N, int64_t d,
                              const int32_t *labels_host, int32_t L, const double *capacities_host, int32_t W,
                              int32_t *assignment_host, int32_t *order_host_or_null, void *part_values_host_or_null,
                              void *workspace_dev, size_t workspace_bytes, void *cuda_stream)
{
    rcd_status rs = check_common(ctx, dtype, N, d, L, W);
    if (rs != RCD_OK) return rs;
    rs = check_capacities(ctx, capacities_host, W);
    if (rs != RCD_OK) return rs;
    if (N > 0 && (!features_host || !labels_host || !assignment_host)) return fail(ctx, RCD_ERR_INVALID_ARG, "null host pointer");
    if (!workspace_dev || ((uintptr_t)workspace_dev) % kAlign) return fail(ctx, RCD_ERR_INVALID_ARG, "workspace null or not 256-byte aligned");
    // The staging areas are placed from the END of the workspace so that the inner workspace can
    // use whatever the true class sizes need.
    const size_t featB = align_up((size_t)std::max<int64_t>(N, 1) * (size_t)d * feat_bytes(dtype));
    const size_t vecB = align_up((size_t)std::max<int64_t>(N, 1) * 4);
    const size_t tail = host_tail_bytes(dtype, N, d, L, W);
    if (workspace_bytes < tail + kAlign) return fail(ctx, RCD_ERR_WORKSPACE_TOO_SMALL, "workspace smaller than the staging areas (%zu bytes)", tail);
    size_t innerBytes = (workspace_bytes - tail) / kAlign * kAlign;
    unsigned char *base = (unsigned char *)workspace_dev;
    unsigned char *feat = base + innerBytes;
    int32_t *lab = (int32_t *)(feat + featB);
    int32_t *asg = (int32_t *)((unsigned char *)lab + vecB);
    int32_t *ord = (int32_t *)((unsigned char *)asg + vecB);
    void *val = (unsigned char *)ord + vecB;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    if (N > 0) {
        RCD_CUDA(ctx, cudaMemcpyAsync(feat, features_host, (size_t)N * (size_t)d * feat_bytes(dtype), cudaMemcpyHostToDevice, st));
        RCD_CUDA(ctx, cudaMemcpyAsync(lab, labels_host, (size_t)N * 4, cudaMemcpyHostToDevice, st));
    }
    rs = rcd_partition(ctx, feat, dtype, N, d, lab, L, capacities_host, W, asg, order_host_or_null ? ord : nullptr,
                       part_values_host_or_null ? val : nullptr, workspace_dev, innerBytes, st);
    if (rs != RCD_OK) return rs;
    if (N > 0) {
        RCD_CUDA(ctx, cudaMemcpyAsync(assignment_host, asg, (size_t)N * 4, cudaMemcpyDeviceToHost, st));
        if (order_host_or_null) RCD_CUDA(ctx, cudaMemcpyAsync(order_host_or_null, ord, (size_t)N * 4, cudaMemcpyDeviceToHost, st));
    }
    if (part_values_host_or_null)
        RCD_CUDA(ctx, cudaMemcpyAsync(part_values_host_or_null, val, (size_t)L * W * 8, cudaMemcpyDeviceToHost, st));
    return rcd_sync_status(ctx, st);
}

// Objective scratch: per class and row block, W partial sums.
static size_t objective_scratch_bytes(int32_t L, int64_t Mmax, int32_t W)
{
    size_t blocks = (size_t)((Mmax + 63) / 64);
    return align_up(std::max<size_t>(1, (size_t)L * blocks * (size_t)W * 8));
}

rcd_status rcd_objective_workspace_bytes(rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d, int32_t L,
                                         int64_t M_max, int32_t W, size_t *bytes_out)
{
    rcd_status rs = check_common(ctx, dtype, N, d, L, W);
    if (rs != RCD_OK) return rs;
    if (!bytes_out || M_max < 0) return fail(ctx, RCD_ERR_INVALID_ARG, "bad M_max or null output");
    Sizes sz = bound_sizes(ctx, dtype, N, d, L, M_max, W);
    *bytes_out = layout_workspace(nullptr, dtype, sz, nullptr) + objective_scratch_bytes(L, std::min(M_max, N), W);
    return RCD_OK;
}

rcd_status rcd_objective(rcd_ctx *ctx, const void *features_dev, rcd_feat_dtype dtype, int64_t N, int64_t d,
                         const int32_t *labels_dev, int32_t L, const int32_t *assignment_dev, int32_t W,
                         void *part_values_dev, void *total_dev, void *workspace_dev, size_t workspace_bytes,
                         void *cuda_stream)
{
    rcd_status rs = check_common(ctx, dtype, N, d, L, W);
    if (rs != RCD_OK) return rs;
    if (!part_values_dev || !total_dev) return fail(ctx, RCD_ERR_INVALID_ARG, "null output pointer");
    if (N > 0 && (!features_dev || !labels_dev || !assignment_dev)) return fail(ctx, RCD_ERR_INVALID_ARG, "null device pointer");
    if (!workspace_dev) return fail(ctx, RCD_ERR_INVALID_ARG, "workspace is null");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    RCD_CUDA(ctx, status_begin(ctx, st));
    const int savedProfile = ctx->cfg.profile;
    ctx->cfg.profile = 0;
    Prepared P;
    rs = prepare(ctx, features_dev, dtype, N, d, labels_dev, L, W, workspace_dev, workspace_bytes, st, &P);
    ctx->cfg.profile = savedProfile;
    if (rs != RCD_OK) return rs;
    size_t scratchB = objective_scratch_bytes(L, P.sz.maxM, W);
    if (P.ws.bytes + scratchB > workspace_bytes)
        return fail(ctx, RCD_ERR_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, objective needs %zu", workspace_bytes, P.ws.bytes + scratchB);
    void *scratch = (unsigned char *)workspace_dev + P.ws.bytes;
    if (P.sz.graphCut)
        rs = launch_cut_objective(ctx, P.sz, P.ws.desc, P.ws.S, P.ws.perm, assignment_dev, part_values_dev, total_dev, scratch, st);
    else
        rs = launch_objective(ctx, P.sz.floatArith ? RCD_FEAT_BF16 : RCD_FEAT_I8, P.sz, P.ws.desc, P.desc, P.ws.S, P.ws.perm, assignment_dev,
                              part_values_dev, total_dev, scratch, st);
    if (rs != RCD_OK) return rs;
    RCD_CUDA(ctx, status_publish(ctx, st));
    return RCD_OK;
}

}  // extern "C"
