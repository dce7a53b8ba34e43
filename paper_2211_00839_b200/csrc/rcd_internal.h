// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include <string>
#include <vector>

#include "rcd.h"

namespace rcd {

constexpr int kMaxSweepBatch = 8;          // blocks refreshed by one dense pass over S
constexpr int kSparseMax = 64;             // blocks refreshed by one threshold pass over S
constexpr int kSweepThreads = 512;         // sweep CTA: 16 warps, one CTA per SM
constexpr int kSelectThreads = 512;        // pick/update CTA: one per class
constexpr int kLazyBlocks = 64;            // row skipping keeps a floor per block for classes of up to this many blocks
constexpr int kPhaseWords = 20;            // 64-bit counters a greedy launch keeps (phase clocks, barrier, pass statistics)
constexpr size_t kAlign = 256;

// Device-side status bits (OR-ed into the status word).
enum : int {
    kDevOk = 0,
    kDevBadLabel = 1,          // a label outside [0, L)
    kDevNoCandidate = 2,       // a class had samples left but no block could take one
    kDevBadState = 4,          // internal consistency check failed
    kDevTimeout = 8,           // a bounded wait inside a kernel ran out
};

// Hand-off word of one class between the CTA that makes its picks and the CTAs that sweep it (the
// asynchronous greedy kernel).  `epoch` is a sequence lock: even = sweep number epoch/2 is published
// and its parameters are stable, odd = the class belongs to its pick CTA (or is finished).
struct ClassSync {
    int32_t epoch;
    int32_t nGroups;   // row groups (tickets) of the published sweep
    int32_t done;      // row groups of the published sweep whose gains are written
    int32_t seq;       // order number of the published sweep (sweep number x L + class)
    int32_t pad_[2];   // (the word fills one 32-byte sector: the counters of two classes never share one)
    int32_t nR;        // of the published sweep: samples of the class still unassigned
    int32_t cfg;       //   blocks it refreshes | warps per row group << 8 | (1 = threshold pass) << 16
};
static_assert(sizeof(ClassSync) == 32, "one 32-byte sector per class");

// One class, as the kernels see it.  Built on the host once the class sizes are known.
struct ClassDesc {
    int32_t M;        // samples in the class
    int32_t ld;       // row pitch of S and of the per-block vectors, in elements (a multiple of 4; pad_row(M) inside rcd_partition)
    int32_t row0;     // first row of the class in class-sorted sample order
    int32_t pad_;
    int64_t sOff;     // element offset of S_l
    int64_t vOff;     // element offset of the class's [W][ld] arrays (coverage, gains)
};

// Where a kernel finds the descriptor of class l: a table in device memory, or (table == null)
// `L` classes of equal size laid out back to back.
struct DescSource {
    const ClassDesc *table;
    int32_t uniM, uniLd;
    __host__ __device__ ClassDesc get(int l) const
    {
        if (table) return table[l];
        ClassDesc c;
        c.M = uniM; c.ld = uniLd; c.row0 = l * uniM; c.pad_ = 0;
        c.sOff = (int64_t)l * uniM * uniLd; c.vOff = 0;
        return c;
    }
};

// The classes a similarity launch covers.
struct SimClasses {
    DescSource src;
    int32_t L;
    int64_t maxM;
    // tensor-core kernel: 128 x 256 tiles that reach the diagonal or lie above it, listed class after class
    const int32_t *tilePrefixDev;   // [L+1] first tile index of every class (null: equal classes)
    int32_t uniTiles;               // tiles per class when the classes are equal
    int64_t upperTiles;             // tiles in all
};

// Pointers into the caller's workspace for one rcd_partition call.
struct Workspace {
    // grouping
    int32_t *counts;        // [L]
    int32_t *chunkHist;     // [nChunks][L]
    int32_t *perm;          // [N] class-sorted position -> dataset index
    void *Xs;               // [N][d] features in class-sorted order
    // per class
    ClassDesc *desc;        // [L]
    int32_t *tilePrefix;    // [L+1] first upper-triangle tile of every class (tensor-core similarity)
    void *S;                // similarity matrices
    void *gaussNorms;       // [N] squared norms of the class-sorted rows (int32 / float)
    double *gaussPartial;   // [L][ceil(maxM/64)] per-row-block sums of pairwise distances
    float *gaussSigma;      // [L] bandwidth of every class
    float *gaussScale;      // [L] 1 / (2 sigma^2)
    void *cutBase;          // [N] graph cut: column sum minus diagonal of every sample (int64 / double)
    void *cover;            // [sum W*ld] coverage vectors (int32 / float)
    void *gains;            // [sum W*ld] stored gains (int64 / float)
    void *fval;             // [L][W] tracked f (int64 / double)
    int32_t *cnt;           // [L][W]
    int32_t *quota;         // [L][W]
    uint8_t *valid;         // [L][W] 1 = stored gains of that block are current
    int32_t *cand;          // [N] unassigned samples of each class (class-local ids), compact
    int32_t *pos;           // [N] position of each sample in cand
    int32_t *nR;            // [L] unassigned count
    int32_t *jstar;         // [L] block chosen for the next pick (-1: none)
    int32_t *sweepN;        // [L] blocks to refresh in the next sweep (0: none)
    int32_t *sweepParts;    // [L][kSparseMax]
    int32_t *sweepMode;     // [L] dense / threshold pass
    void *thr;              // [sum ld] threshold vector of every class (int32 / float)
    unsigned long long *hitCount;   // [L]
    unsigned long long *sparseElems; // [L]
    int32_t *sparseFrom;    // [L]
    int32_t *sweepCS;       // [L] warps per row group in the next sweep
    int32_t *rowCtr;        // [L] ticket counter over row groups of the running sweep
    ClassSync *sync;        // [L] asynchronous kernel: hand-off words
    int32_t *tickets;       // [N + L] asynchronous kernel: one ticket counter per (class, sweep number), never reused
    int32_t *sizesSorted;   // [L] class sizes, ascending
    int32_t *classOrder;    // [L] classes by descending size
    void *floorv;           // [L][kLazyBlocks] per block: every stored gain at or above it is exact (int64 / double)
    void *theta;            // [L][kLazyBlocks] per block: floor its next row-skipping pass will establish
    void *sweepTheta;       // [L][kLazyBlocks] floors of the blocks the class's next pass lists, in list order (int64 / fp32)
    int32_t *lazyStat;      // [L][4] row-skipping passes of the class, misses, members needed before rows are skipped
    long long *sweepF;      // [L][8] asynchronous kernel, int8 features: f of the first blocks in the sweep's list
    int32_t *sweepList;     // [3][L] classes that sweep in a step (three lists in rotation)
    int32_t *nSweep;        // [3] (+1 pad)
    unsigned long long *stepBytes;   // [steps+1] bytes the sweep of step t has to read
    unsigned long long *stepOps;     // [steps+1] element x block pairs of that sweep
    unsigned long long *phaseNs;     // [6] sweep-/pick-phase ns of the persistent kernel, barrier counter, threshold-pass hits / elements / max blocks
    int32_t *status;        // [1]
    size_t bytes;           // total bytes laid out
};

struct Sizes {
    int64_t N, d;
    int32_t L, W;
    int64_t sElems;         // sum M_l * ld_l
    int64_t vElems;         // sum W * ld_l
    int64_t maxM;
    int32_t nChunks;
    bool floatArith;        // fp32 S / fp32 gains / double f (bf16 features, or the Gaussian kernel)
    bool graphCut;          // graph-cut objective: the gains array holds 8-byte ties
};

constexpr int kGroupChunk = 1024;           // samples per chunk of the stable class split

inline size_t feat_bytes(rcd_feat_dtype t) { return t == RCD_FEAT_I8 ? 1 : 2; }
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
inline int32_t pad4(int64_t m) { return (int32_t)((m + 3) / 4 * 4); }
// Row pitch of S and of the per-block vectors inside rcd_partition / rcd_objective: a multiple of 8
// elements, so that every row starts on a 32-byte boundary (one memory sector): the 16-byte pieces that
// the sweeps copy then pair up into whole sectors.
inline int32_t pad_row(int64_t m) { return (int32_t)((m + 7) / 8 * 8); }

// Tiles the tensor-core similarity kernel computes for a class of M samples: 128 rows x 256 columns each, those that
// reach the diagonal or lie above it (row block tm pairs with the column blocks from tm / 2 on).
inline int64_t sim_tiles(int64_t M)
{
    const int64_t rowBlocks = (M + 127) / 128, colBlocks = (M + 255) / 256;
    int64_t n = 0;
    for (int64_t tm = 0; tm < rowBlocks; ++tm) n += colBlocks - tm / 2;
    return n;
}

// Lays the workspace out at `base` (may be null to measure).  Returns total bytes.
size_t layout_workspace(void *base, rcd_feat_dtype dtype, const Sizes &sz, Workspace *ws);

}  // namespace rcd

struct rcd_ctx {
    int device = 0;
    int smCount = 0;
    int maxSmemOptin = 0;
    bool cooperative = false;           // device supports cooperative launches
    rcd_config cfg{};
    std::string err;
    int32_t *hostStage = nullptr;       // pinned, counts / status read-back
    int32_t *statusOwn = nullptr;       // device status word for calls that take no workspace
    size_t hostStageInts = 0;
    // profiling
    cudaEvent_t evPhase[5]{};           // start, after group, after similarity, after greedy, end
    bool phaseValid = false;
    std::vector<cudaEvent_t> evSweep;   // 2 per step
    int64_t sweepEventsUsed = 0;
    int64_t kernelLaunches = 0;
    int64_t tcLaunches = 0;
    int64_t steps = 0;
    const unsigned long long *stepBytesDev = nullptr;
    const unsigned long long *stepOpsDev = nullptr;
    const unsigned long long *phaseNsDev = nullptr;
    const int32_t *statusDev = nullptr;
};

namespace rcd {

rcd_status fail(rcd_ctx *ctx, rcd_status st, const char *fmt, ...);
rcd_status cuda_fail(rcd_ctx *ctx, cudaError_t e, const char *what);

#define RCD_CUDA(ctx, call)                                            \
    do {                                                               \
        cudaError_t e__ = (call);                                      \
        if (e__ != cudaSuccess) return ::rcd::cuda_fail(ctx, e__, #call); \
    } while (0)

// ---- launchers implemented in the .cu files (all asynchronous on `st`) ----

// class split
rcd_status launch_count_labels(rcd_ctx *ctx, const int32_t *labels, int64_t N, int32_t L, int32_t *counts,
                               int32_t *status, cudaStream_t st);
rcd_status launch_stable_split(rcd_ctx *ctx, const int32_t *labels, int64_t N, int32_t L, int32_t nChunks,
                               int32_t *chunkHist, const ClassDesc *descDev, int32_t *perm, cudaStream_t st);
rcd_status launch_gather_rows(rcd_ctx *ctx, const void *X, const int32_t *perm, int64_t N, int64_t rowBytes,
                              void *Xs, cudaStream_t st);

// similarity: S_l = Xs_l Xs_l^T for every class described by desc
rcd_status launch_similarity(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t Ntot, int64_t d,
                             const SimClasses &cls, void *S, cudaStream_t st);

// Gaussian-kernel similarity: transforms the dot products in S in place
rcd_status launch_gaussian(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t N, int64_t d, const SimClasses &cls,
                           void *S, void *norms, double *partial, float *sigma, float *scale, cudaStream_t st);
size_t gaussian_scratch_bytes(int64_t N, int32_t L, int64_t maxM);

// greedy loop
rcd_status launch_greedy(rcd_ctx *ctx, rcd_feat_dtype dtype, const Sizes &sz, const Workspace &ws,
                         const std::vector<ClassDesc> &descHost, int32_t *assignment, int32_t *order,
                         cudaStream_t st);

rcd_status launch_bounded_wait_selftest(rcd_ctx *ctx, unsigned *counter, int32_t *status, cudaStream_t st);

// graph-cut objective: the whole greedy loop, and f from an assignment
rcd_status launch_cut(rcd_ctx *ctx, const Sizes &sz, const Workspace &ws, int32_t *assignment, int32_t *order, cudaStream_t st);
rcd_status launch_cut_objective(rcd_ctx *ctx, const Sizes &sz, const ClassDesc *descDev, const void *S, const int32_t *perm,
                                const int32_t *assignment, void *partValues, void *total, void *scratch, cudaStream_t st);

// objective from an assignment
rcd_status launch_objective(rcd_ctx *ctx, rcd_feat_dtype dtype, const Sizes &sz, const ClassDesc *descDev,
                            const std::vector<ClassDesc> &descHost, const void *S, const int32_t *perm,
                            const int32_t *assignment, void *partValues, void *total, void *scratch,
                            cudaStream_t st);


#ifdef __CUDACC__
// ---- warp-wide reductions of (value, index) pairs by 32-bit redux instead of shuffle ladders ----
// Order-preserving images in unsigned integers (a < b exactly when image(a) < image(b); -0.0 is taken as +0.0).
__device__ __forceinline__ unsigned long long ordered_u64(long long x) { return (unsigned long long)x ^ 0x8000000000000000ull; }
__device__ __forceinline__ unsigned long long ordered_u64(double x)
{
    const unsigned long long b = (unsigned long long)__double_as_longlong(x + 0.0);
    return b ^ ((b >> 63) ? ~0ull : 0x8000000000000000ull);
}
__device__ __forceinline__ unsigned ordered_u32(float x)
{
    const unsigned b = __float_as_uint(x + 0.0f);
    return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float from_ordered_u32(unsigned o) { return __uint_as_float(o ^ ((o >> 31) ? 0x80000000u : 0xffffffffu)); }

// Maximum of a 64-bit key over the warp (two 32-bit warp reductions: high words, then low words among the lanes that
// hold the greatest high word).
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long k)
{
    const unsigned hi = (unsigned)(k >> 32), lo = (unsigned)k;
    const unsigned mhi = __reduce_max_sync(0xffffffffu, hi);
    const unsigned mlo = __reduce_max_sync(0xffffffffu, hi == mhi ? lo : 0u);
    return ((unsigned long long)mhi << 32) | mlo;
}
// Arg-maximum of (ordered image of the value, index) pairs over the warp: the greatest value, and among the lanes that
// hold it the lowest index; lanes without a candidate pass index INT_MAX.  Three warp-wide reductions.
__device__ __forceinline__ void warp_argmax_ordered(unsigned long long &ord, int &idx)
{
    const bool has = idx != 0x7fffffff;
    const unsigned hi = has ? (unsigned)(ord >> 32) : 0u, lo = has ? (unsigned)ord : 0u;
    const unsigned mhi = __reduce_max_sync(0xffffffffu, hi);
    const unsigned mlo = __reduce_max_sync(0xffffffffu, (has && hi == mhi) ? lo : 0u);
    const int mi = __reduce_min_sync(0xffffffffu, (has && hi == mhi && lo == mlo) ? idx : 0x7fffffff);
    ord = ((unsigned long long)mhi << 32) | mlo;
    idx = mi;
}
// The same for the least value (lowest index among equals).
__device__ __forceinline__ void warp_argmin_ordered(unsigned long long &ord, int &idx)
{
    unsigned long long inv = ~ord;
    warp_argmax_ordered(inv, idx);
    ord = ~inv;
}
__device__ __forceinline__ long long from_ordered_u64_ll(unsigned long long o) { return (long long)(o ^ 0x8000000000000000ull); }
__device__ __forceinline__ double from_ordered_u64_d(unsigned long long o)
{
    return __longlong_as_double((long long)(o ^ ((o >> 63) ? 0x8000000000000000ull : ~0ull)));
}
#endif

}  // namespace rcd
