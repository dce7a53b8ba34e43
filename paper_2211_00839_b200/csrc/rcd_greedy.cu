// The greedy loop of Algorithm 1 with the facility-location objective, for all classes together.
//
// Per class the device keeps, for every block p: a coverage vector cover_p[i] =
// max(0, max_{v' in A_p} S[i][v']), the tracked value f_p = sum_i cover_p[i], the count and the
// quota, and a row of stored marginal gains G_p[v] = sum_i max(0, S[v][i] - cover_p[i])
// (GreedyStep's f(A_p u {v}) - f(A_p); S is symmetric).  G_p stays correct until block p itself
// receives a sample, so a pass over S is only needed when the chosen block's row is out of date,
// and that pass refreshes up to `sweep_batch_max` out-of-date blocks at once.
//
// The loop advances in rounds.  A round is
//   a sweep phase  every class that asked for a sweep gets one.  Persistent CTAs (one per SM)
//                  serve the classes; teams of 1-16 warps pull groups of rows, each warp streams
//                  its 128-column chunks of those rows with 128-bit loads against the coverage
//                  vectors staged in shared memory, reduces with warp shuffles, the team writes G;
//   a pick phase   one CTA per class makes pick after pick (argmax of G_{j*} over the unassigned
//                  samples with a warp-shuffle reduction and lowest-index ties, coverage / value /
//                  count update, removal of v* from the candidate list, choice of the next block
//                  j* = least f among the non-full blocks) until the next block's gains are out of
//                  date, and then asks for the class's next sweep.
// Classes are independent, so each class makes exactly the picks Algorithm 1 prescribes whatever
// the interleaving.  The whole loop is one cooperative launch (greedy_persistent_kernel, phases
// separated by a bounded grid barrier); sweep_kernel / chain_kernel are the same two phases as
// separate launches, used when every sweep is to be timed on its own.
#include "rcd_internal.h"

#include <limits.h>
#include <algorithm>
#include <type_traits>

namespace rcd {

template <typename SV> struct Arith;
template <> struct Arith<int32_t> {
    using GV = long long;   // gains
    using FV = long long;   // tracked f
    static constexpr bool kInt = true;
};
template <> struct Arith<float> {
    using GV = float;
    using FV = double;
    static constexpr bool kInt = false;
};

template <typename SV>
struct GreedyParams {
    using GV = typename Arith<SV>::GV;
    using FV = typename Arith<SV>::FV;
    const ClassDesc *desc;
    const SV *S;
    SV *cover;
    GV *gains;
    FV *fval;
    int32_t *cnt;
    const int32_t *quota;
    uint8_t *valid;
    int32_t *cand;
    int32_t *pos;
    int32_t *nR;
    int32_t *jstar;
    int32_t *sweepN;
    int32_t *sweepParts;    // [L][kSparseMax] blocks the class's next sweep refreshes
    int32_t *sweepMode;     // [L] 0 = dense pass (coverage vectors in shared memory), 1 = threshold pass
    SV *thr;                // per class [ld]: min over the listed blocks of their coverage (threshold pass)
    unsigned long long *hitCount;   // [L] elements above the threshold in the class's last threshold pass
    unsigned long long *sparseElems; // [L] elements that pass compared (0: the last pass was dense)
    int32_t *sparseFrom;    // [L] members every out-of-date block must have before the next threshold pass is tried
    int32_t *sweepCS;       // warps that share one row group in the next sweep (1, 2, 4, 8 or 16)
    int32_t *rowCtr;
    int32_t *sweepList;
    int32_t *nSweep;
    unsigned long long *stepBytes;
    unsigned long long *stepOps;
    unsigned long long *phaseNs;    // [0..1] time block 0 spent in sweep / pick phases (persistent kernel), [2] grid-barrier
                                    // counter, [3..5] threshold passes: elements above the threshold / elements compared / most blocks in one pass,
                                    // [6..7] asynchronous kernel: ns the first sweep CTA found nothing to sweep, its visits
    unsigned *barrier;              // arrival counter of the persistent kernel's grid barrier
    int32_t *status;
    const int32_t *perm;
    int32_t *assignment;
    int32_t *order;         // may be null
    int32_t L, W;
    int32_t batchMax;       // 1, 2, 4 or 8
    int32_t smemBytes;      // dynamic shared memory of the sweep kernel
    int32_t segIters;       // int path: chunk iterations a 32-bit partial sum can take without overflow
    int32_t sweepWarps;     // warps of one sweep launch (CTAs x 16)
    uint32_t one;           // the value 1, opaque to the compiler (see accumulate_chunk)
    int32_t hitShift;           // a threshold pass with more than 1 element in 2^hitShift above the threshold makes the class wait
    int32_t sparseMinMembers;   // threshold passes start once every out-of-date block has this many members (<0: never)
    // asynchronous kernel (greedy_async_kernel); asyncMode = 0 everywhere else
    ClassSync *sync;            // [L] hand-off words
    int32_t *tickets;           // [N + L] ticket counter of sweep k of class l at tickets[row0_l + l + k]
    long long *sweepF;          // [L][kMaxSweepBatch] int8 features: f of the blocks a dense pass refreshes
    int32_t asyncMode;
    int32_t nPick;              // CTAs [0, nPick) make picks, the others sweep
    int32_t helpMin;            // row groups a sweep must have left for a sweep CTA that is not at home there
    int32_t asyncGroup;         // sweeps published one after another that are served together (by CTA home position)
    // row skipping (lazy evaluation of GreedyStep's argmax): see plan_decide / sweep_class_lazy / pick_chain
    FV *floorv;                 // [L][kLazyBlocks] every stored gain of the block at or above this value is exact
    FV *theta;                  // [L][kLazyBlocks] the floor the block's next row-skipping pass establishes
    GV *sweepTheta;             // [L][kLazyBlocks] those floors for the blocks of the class's next pass, in list order
    int32_t *lazyStat;          // [L][4] row-skipping passes, misses
    int32_t lazyFrom;           // members every listed block must have before a pass skips rows (< 0: never)
    int32_t incremental;        // 1 = a pick updates the stored gains of its block in place (see delta_term) instead of leaving them to a pass
    int32_t deltaMax;           //     ... when the pick raised the block's coverage in at most this many columns (<= kDeltaMax)
    int32_t denseRing;          // 8-block dense passes stream through shared-memory rings when the coverage vectors leave room
    const int32_t *classOrder;  // [L] classes by descending size (the order in which the one-CTA-per-class loop draws them)
    const int32_t *sizesSorted; // [L] class sizes in ascending order
    int32_t minM;               // smallest non-empty class
    int32_t nonEmpty;           // classes that hold at least one sample
};

__host__ __device__ inline int rows_per_group(int P) { return P == 8 ? 4 : 8; }

// ---------------------------------------------------------------------------------------------
// Choice of the next block and of the blocks the next sweep refreshes.  The class's block values
// and flags live in shared memory while its CTA works on it (plan_load), so a chain of picks
// re-reads nothing from global memory; plan_decide is run by warp 0.
constexpr int kMaxBlocks = 1024;
template <typename FV>
struct PlanShared {
    FV f[kMaxBlocks];              // tracked f of every block
    int32_t room[kMaxBlocks];      // quota - count
    int32_t quota[kMaxBlocks];
    uint8_t open[kMaxBlocks];      // bit 0: block is not full, bit 1: its stored gains are out of date
    int32_t nextJ;                 // plan_decide's answer: block of the next pick (-1: none)
    int32_t needSweep;             //                       1 = that pick must wait for a sweep
    int32_t sweepBlocks;           //                       blocks in the scheduled sweep's list
    int32_t sweepSparse;           //                       1 = the scheduled sweep is a threshold pass
    int32_t sweepLazy;             //                       1 = ... that skips rows below the blocks' floors
    // Row skipping.  Stored gains never grow when a block grows (diminishing returns, Section 3.1), so an
    // out-of-date stored gain is an upper bound of the current one.  floorv[p]: every stored gain of block p at
    // or above it was recomputed since p last changed (exact); theta[p]: the floor the next pass will use.
    FV floorv[kLazyBlocks];
    FV theta[kLazyBlocks];
    int32_t lazySweeps, lazyMisses;
};

template <typename T> __device__ __forceinline__ T lowest_value();
template <> __device__ __forceinline__ long long lowest_value<long long>() { return LLONG_MIN; }
template <> __device__ __forceinline__ double lowest_value<double>() { return -INFINITY; }
template <> __device__ __forceinline__ float lowest_value<float>() { return -INFINITY; }
template <typename T> __device__ __forceinline__ T highest_value();
template <> __device__ __forceinline__ long long highest_value<long long>() { return LLONG_MAX; }
template <> __device__ __forceinline__ double highest_value<double>() { return INFINITY; }

// Rows one ticket of a sweep stands for: R rows of a dense pass, two of a threshold pass, 32 of a row-skipping
// pass (one per lane: most of them are skipped).
constexpr int kLazyRows = 32;

template <typename SV>
__device__ __forceinline__ void plan_load(const GreedyParams<SV> &prm, int l, PlanShared<typename Arith<SV>::FV> &sh)
{
    const int W = prm.W;
    for (int p = threadIdx.x; p < W; p += blockDim.x) {
        const int64_t at = (int64_t)l * W + p;
        const int quota = prm.quota[at];
        const int room = quota - prm.cnt[at];
        sh.f[p] = prm.fval[at];
        sh.room[p] = room;
        sh.quota[p] = quota;
        sh.open[p] = (uint8_t)((room > 0 ? 1 : 0) | (prm.valid[at] ? 0 : 2));
        if (p < kLazyBlocks) {
            sh.floorv[p] = prm.floorv[(int64_t)l * kLazyBlocks + p];
            sh.theta[p] = prm.theta[(int64_t)l * kLazyBlocks + p];
        }
    }
    if (threadIdx.x == 0) {
        sh.lazySweeps = prm.lazyStat[4 * l];
        sh.lazyMisses = prm.lazyStat[4 * l + 1];
    }
}

// The counterpart of plan_load for what a chain changes of the row-skipping state (block values and counts are
// written as the picks are made).
template <typename SV>
__device__ __forceinline__ void plan_store_lazy(const GreedyParams<SV> &prm, int l, const PlanShared<typename Arith<SV>::FV> &sh)
{
    const int n = min(prm.W, kLazyBlocks);
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        prm.floorv[(int64_t)l * kLazyBlocks + p] = sh.floorv[p];
        prm.theta[(int64_t)l * kLazyBlocks + p] = sh.theta[p];
    }
    if (threadIdx.x == 0) {
        prm.lazyStat[4 * l] = sh.lazySweeps;
        prm.lazyStat[4 * l + 1] = sh.lazyMisses;
    }
}

// Warp 0 only.  nR = samples of the class still unassigned.
constexpr int kSparseQueue = 256;                                  // threshold pass: queue entries per warp
constexpr int kSparseRows = 2;                                     // threshold pass: rows per warp and ticket
constexpr int kSparseStages = 8;                                   // threshold pass: ring of chunks of S per warp
constexpr int kSparseRingBytes = kSparseStages * kSparseRows * 512;   // rows x 32 lanes x 16 bytes per stage
constexpr int kSparseWarpBytes = kSparseRingBytes + kSparseQueue * 8; // ring + queue
constexpr int kSparseQueueBytes = kSparseWarpBytes * (kSweepThreads / 32);
// The rings are the destination of 16-byte asynchronous copies whose sources (rows of S) start on 32-byte
// boundaries: the dynamic shared memory is declared 128-byte aligned and the rings start on a 128-byte
// boundary behind the threshold vector, so that a copy never straddles two 32-byte sectors (a ring that
// starts 16 bytes off such a boundary doubles the sectors fetched per copy).
__host__ __device__ inline int thr_bytes_aligned(int bytes) { return (bytes + 127) & ~127; }
static_assert(kSparseWarpBytes % 128 == 0, "per-warp rings must keep the 128-byte alignment");

// What plan_decide reads from global memory when it has to schedule a sweep.  A chain of picks schedules
// at most one (its last pick), so the chain loads these at its start, under the first argmax, instead of
// waiting for them at the end.  `remaining` is decremented by other classes' chains at any time: it may only
// steer decisions that cannot change a result (the integer path, where every sum is exact); the
// floating-point path, whose sums depend on how a pass splits its columns, uses classes_alongside().
struct PlanGlobals {
    int32_t remaining;              // unfinished classes
    int32_t from;                   // sparseFrom[l]
    unsigned long long elems;       // sparseElems[l]
    unsigned long long hits;        // hitCount[l] (added to by the sweeping CTAs)
};
template <typename SV>
__device__ __forceinline__ PlanGlobals plan_globals(const GreedyParams<SV> &prm, int l)
{
    PlanGlobals g;
    g.remaining = *(volatile int32_t *)&prm.nSweep[3];
    g.from = *(volatile int32_t *)&prm.sparseFrom[l];
    g.elems = *(volatile unsigned long long *)&prm.sparseElems[l];
    g.hits = *(volatile unsigned long long *)&prm.hitCount[l];
    return g;
}

// How many classes are taken to be still unfinished when a class has made `made` picks: those larger than
// `made` samples.  A function of the class's own progress and of the class sizes only, so that the shape of a
// floating-point sweep (dense or threshold pass, warps per row group: they fix the order of its additions)
// never depends on the timing of other classes.  Whole warp; the same value in every lane.
template <typename SV>
__device__ __forceinline__ int classes_alongside(const GreedyParams<SV> &prm, int made)
{
    if (made < prm.minM) return prm.nonEmpty;
    const int lane = threadIdx.x & 31;
    int n = 0;
    for (int i = lane; i < prm.L; i += 32) n += __ldg(prm.sizesSorted + i) > made ? 1 : 0;
    for (int off = 16; off > 0; off >>= 1) n += __shfl_xor_sync(0xffffffffu, n, off);
    return n;
}

template <typename SV>
__device__ void plan_decide(const GreedyParams<SV> &prm, int l, const ClassDesc &c, int nR, int nextStep,
                            PlanShared<typename Arith<SV>::FV> &sh, const PlanGlobals *pre = nullptr)
{
    using FV = typename Arith<SV>::FV;
    using GV = typename Arith<SV>::GV;
    const int lane = threadIdx.x & 31;
    const int W = prm.W;
    uint8_t *valid = prm.valid + (int64_t)l * W;
    if (nR == 0) {
        if (lane == 0) { prm.jstar[l] = -1; prm.sweepN[l] = 0; sh.nextJ = -1; sh.needSweep = 0; }
        return;
    }

    {
        if (W <= 32) {
            // At most one block per lane and nothing out of date (the usual case once stored gains are corrected in place):
            // the next block is the argmin of f over the non-full blocks, lowest index on ties, and no pass is due.
            const uint8_t o = lane < W ? sh.open[lane] : (uint8_t)0;
            const bool cand = (o & 1) != 0;
            const unsigned candMask = __ballot_sync(0xffffffffu, cand);
            const unsigned staleMask = __ballot_sync(0xffffffffu, cand && (o & 2));
            if (candMask != 0 && staleMask == 0) {
                const unsigned long long fo = cand ? ordered_u64(sh.f[lane]) : ~0ull;     // (same order as f itself)
                const unsigned hi = (unsigned)(fo >> 32);
                const unsigned lo = (unsigned)fo;
                const unsigned mhi = __reduce_min_sync(0xffffffffu, hi);
                const unsigned mlo = __reduce_min_sync(0xffffffffu, (cand && hi == mhi) ? lo : 0xffffffffu);
                const unsigned eq = __ballot_sync(0xffffffffu, cand && hi == mhi && lo == mlo);
                const int jnext = __ffs(eq) - 1;
                if (lane == 0) { prm.jstar[l] = jnext; prm.sweepN[l] = 0; sh.nextJ = jnext; sh.needSweep = 0; }
                return;
            }
        }
    }
    // j* = argmin over non-full blocks of f, ties -> lowest index
    FV bestF = 0;
    int bestP = INT_MAX;
    int nStale = 0;
    int fewest = INT_MAX;                          // members of the emptiest out-of-date non-full block
    int floorsKnown = 1;                           // every out-of-date non-full block has a floor for a row-skipping pass
    for (int p = lane; p < W; p += 32) {
        const uint8_t o = sh.open[p];
        if (o & 1) {
            const FV fp = sh.f[p];
            if (bestP == INT_MAX || fp < bestF) { bestF = fp; bestP = p; }
            if (o & 2) {
                ++nStale;
                fewest = min(fewest, sh.quota[p] - sh.room[p]);
                if (p >= kLazyBlocks || !(sh.theta[p] > lowest_value<FV>())) floorsKnown = 0;
            }
        }
    }
    for (int off = 16; off > 0; off >>= 1) {
        FV oF = __shfl_xor_sync(0xffffffffu, bestF, off);
        int oP = __shfl_xor_sync(0xffffffffu, bestP, off);
        nStale += __shfl_xor_sync(0xffffffffu, nStale, off);
        fewest = min(fewest, __shfl_xor_sync(0xffffffffu, fewest, off));
        floorsKnown &= __shfl_xor_sync(0xffffffffu, floorsKnown, off);
        if (oP != INT_MAX && (bestP == INT_MAX || oF < bestF || (oF == bestF && oP < bestP))) { bestF = oF; bestP = oP; }
    }
    if (bestP == INT_MAX) {
        if (lane == 0) {
            prm.jstar[l] = -1; prm.sweepN[l] = 0; sh.nextJ = -1; sh.needSweep = 0;
            atomicOr(prm.status, kDevNoCandidate);
        }
        return;
    }
    const int jstar = bestP;
    if (!(sh.open[jstar] & 2)) {
        if (lane == 0) { prm.jstar[l] = jstar; prm.sweepN[l] = 0; sh.nextJ = jstar; sh.needSweep = 0; }
        return;
    }
    // how many blocks one pass can refresh: bounded by the configuration, by the shared memory
    // that holds their coverage vectors and by the number of out-of-date blocks
    int cap = prm.batchMax;
    while (cap > 1 && (int64_t)cap * c.ld * (int64_t)sizeof(SV) > prm.smemBytes) cap >>= 1;
    // Threshold pass: once every out-of-date block has a few members, almost no S[v][i] exceeds the
    // blocks' coverage, so the pass only compares S with one threshold vector and touches the
    // blocks' coverage per exceeding element: it can refresh up to kSparseMax blocks at once.
    // A threshold pass is tried when every out-of-date block has sparseFrom[l] members; if more than
    // 1 element in 32 turned out to be above the threshold, the next try waits until the blocks
    // have twice the members they had.  Near the end of a class (few rows left) the dense pass,
    // which can split the columns of a row over several warps, keeps more warps busy.
    // (everything the decision reads from global memory: loaded by the caller beforehand, or here, back to
    // back: one trip to memory)
    PlanGlobals g;
    if (pre) g = *pre;
    else g = plan_globals(prm, l);
    int remaining = g.remaining;
    if constexpr (!Arith<SV>::kInt) remaining = classes_alongside(prm, c.M - nR);
    if (prm.asyncMode == 2) remaining = 1;                   // the class has its CTA to itself
    int from = 0;
    if (lane == 0) {
        from = g.from;
        if (g.elems) {
            atomicAdd(&prm.phaseNs[3], g.hits);
            atomicAdd(&prm.phaseNs[4], g.elems);
            if ((g.hits << prm.hitShift) > g.elems) { from = 2 * fewest; prm.sparseFrom[l] = from; }
            prm.hitCount[l] = 0;
            prm.sparseElems[l] = 0;
        }
    }
    from = __shfl_sync(0xffffffffu, from, 0);
    const int64_t together0 = max(remaining, 1);
    // Row skipping: a threshold pass may leave out every row whose stored gains lie below the listed blocks'
    // floors (they stay upper bounds).  Tried once the blocks have lazyFrom members; a class where, after a few
    // misses, more than a quarter of such passes ended in one (the best stored gain fell below its floor) stops trying.
    const bool lazyWanted = prm.lazyFrom >= 0 && W <= kLazyBlocks && floorsKnown && fewest >= prm.lazyFrom &&
                            (sh.lazyMisses <= 8 || 4 * sh.lazyMisses <= sh.lazySweeps);
    const bool sparse = prm.sparseMinMembers >= 0 && prm.batchMax > 1 && (nStale > 1 || lazyWanted) && fewest >= from &&
                        (int64_t)thr_bytes_aligned(c.ld * (int)sizeof(SV)) + kSparseQueueBytes <= prm.smemBytes &&
                        (lazyWanted || together0 * ((nR + kSparseRows - 1) / kSparseRows) * 4 >= prm.sweepWarps);
    if (sparse) cap = kSparseMax;
    const bool lazy = sparse && lazyWanted;
    // n blocks are refreshed; the dense pass is instantiated for lists of 1, 2, 4, 8, so its list is
    // padded with copies of j* up to the next power of two (same bytes read, identical values written)
    const int n = nStale < cap ? nStale : cap;
    int P = 1;
    while (P < n) P *= 2;
    if (sparse) P = n;
    int32_t *parts = prm.sweepParts + (int64_t)l * kSparseMax;
    GV *listTheta = prm.sweepTheta + (int64_t)l * kLazyBlocks;
    if (lane == 0) {
        parts[0] = jstar; valid[jstar] = 1; sh.open[jstar] = 1;
        if (jstar < kLazyBlocks) {
            sh.floorv[jstar] = lazy ? sh.theta[jstar] : lowest_value<FV>();
            listTheta[0] = lazy ? (GV)sh.theta[jstar] : lowest_value<GV>();
        }
    }
    __syncwarp();
    if (nStale <= cap) {
        // every out-of-date non-full block is listed: after j* in index order (the order of the list does not
        // enter any result: each block's gains are summed by themselves)
        int k = 1;
        for (int p0 = 0; p0 < W; p0 += 32) {
            const int p = p0 + lane;
            const bool take = p < W && sh.open[p] == 3;
            const unsigned m = __ballot_sync(0xffffffffu, take);
            if (take) {
                const int at = k + __popc(m & ((1u << lane) - 1u));
                parts[at] = p;
                valid[p] = 1;
                sh.open[p] = 1;
                if (p < kLazyBlocks) {
                    sh.floorv[p] = lazy ? sh.theta[p] : lowest_value<FV>();
                    if (at < kLazyBlocks) listTheta[at] = lazy ? (GV)sh.theta[p] : lowest_value<GV>();
                }
            }
            k += __popc(m);
        }
        __syncwarp();
    } else
    for (int k = 1; k < n; ++k) {
        // next out-of-date non-full block of least f: the one most likely to be chosen soon
        FV qF = 0;
        int qP = INT_MAX;
        for (int p = lane; p < W; p += 32) {
            if (sh.open[p] == 3) {
                const FV fp = sh.f[p];
                if (qP == INT_MAX || fp < qF) { qF = fp; qP = p; }
            }
        }
        for (int off = 16; off > 0; off >>= 1) {
            FV oF = __shfl_xor_sync(0xffffffffu, qF, off);
            int oP = __shfl_xor_sync(0xffffffffu, qP, off);
            if (oP != INT_MAX && (qP == INT_MAX || oF < qF || (oF == qF && oP < qP))) { qF = oF; qP = oP; }
        }
        if (lane == 0) {
            parts[k] = qP; valid[qP] = 1; sh.open[qP] = 1;
            if (qP < kLazyBlocks) sh.floorv[qP] = lowest_value<FV>();     // (more blocks than one list holds: never a row-skipping pass)
        }
        __syncwarp();
    }
    if (lane == 0) for (int k = n; k < P; ++k) parts[k] = jstar;
    // warps per row group: enough that the row groups of the classes that sweep together (every
    // unfinished class, once per round) cover every warp of the launch, at least one 128-column chunk per warp
    const int R = lazy ? kLazyRows : (sparse ? kSparseRows : rows_per_group(P));
    const int64_t nGroups = (nR + R - 1) / R;
    const int rem = remaining;                                        // unfinished classes: they all sweep in the same round
    const int64_t together = rem > 1 ? rem : 1;
    const int chunks = (c.ld + 127) / 128;
    int CS = 1;
    while (!sparse && CS < 16 && 2 * CS <= chunks && 2 * CS * together * nGroups <= prm.sweepWarps) CS *= 2;
    if (lane == 0) {
        sh.nextJ = jstar;
        sh.needSweep = 1;
        sh.sweepBlocks = P;
        sh.sweepSparse = sparse ? 1 : 0;
        sh.sweepLazy = lazy ? 1 : 0;
        prm.sweepMode[l] = lazy ? 2 : (sparse ? 1 : 0);
        if (sparse) {
            // (a row-skipping pass compares only the rows it reads: its hit rate does not steer the back-off)
            prm.sparseElems[l] = lazy ? 0ull : (unsigned long long)nR * (unsigned long long)c.M;
            atomicMax(&prm.phaseNs[5], (unsigned long long)P);
        }
        if (lazy) {
            sh.lazySweeps += 1;
            atomicAdd(&prm.phaseNs[8], 1ull);
        }
        prm.jstar[l] = jstar;
        prm.sweepN[l] = P;
        prm.sweepCS[l] = CS;
        prm.rowCtr[l] = 0;
        if (prm.asyncMode == 2) {
            // (one CTA runs the class from its first pick to its last: nothing to publish)
        } else if (prm.asyncMode) {
            ClassSync &sy = prm.sync[l];                   // published with the epoch by the caller
            sy.nGroups = (int32_t)nGroups;
            sy.nR = nR;
            sy.cfg = P | (CS << 8) | ((lazy ? 2 : (sparse ? 1 : 0)) << 16);
            if constexpr (Arith<SV>::kInt) {
                if (!sparse)
                    for (int k = 0; k < P; ++k) prm.sweepF[(int64_t)l * kMaxSweepBatch + k] = (long long)sh.f[parts[k]];
            }
        } else {
            int par = nextStep % 3;
            int slot = atomicAdd(&prm.nSweep[par], 1);
            prm.sweepList[(int64_t)par * prm.L + slot] = l;
        }
        if (lazy) {
            // what the pass reads whatever it finds: the threshold vector, the candidate list and the stored gains of
            // the listed blocks; the rows of S it does read are counted by the warps that read them
            atomicAdd(&prm.stepBytes[nextStep], (unsigned long long)((int64_t)c.ld * sizeof(SV) + (int64_t)nR * (4 + (int64_t)n * sizeof(GV))));
        } else {
            atomicAdd(&prm.stepBytes[nextStep], (unsigned long long)((int64_t)nR * c.ld + (int64_t)(sparse ? 1 : n) * c.ld) * sizeof(SV));
            atomicAdd(&prm.stepOps[nextStep], (unsigned long long)((int64_t)nR * c.M * (sparse ? 1 : n)));
            if (sparse) atomicAdd(&prm.phaseNs[14], (unsigned long long)((int64_t)nR * c.ld + c.ld) * sizeof(SV));
        }
    }
}

// ---------------------------------------------------------------------------------------------
template <typename SV>
__global__ void __launch_bounds__(kSelectThreads, 4) init_kernel(GreedyParams<SV> prm)
{
    using FV = typename Arith<SV>::FV;
    __shared__ PlanShared<FV> shPlan;
    const int l = blockIdx.x;
    const ClassDesc c = prm.desc[l];
    const int W = prm.W;
    SV *cover = prm.cover + c.vOff;
    for (int64_t i = threadIdx.x; i < (int64_t)W * c.ld; i += blockDim.x) cover[i] = 0;
    for (int v = threadIdx.x; v < c.M; v += blockDim.x) {
        prm.cand[c.row0 + v] = v;
        prm.pos[c.row0 + v] = v;
    }
    for (int p = threadIdx.x; p < W; p += blockDim.x) {
        prm.cnt[(int64_t)l * W + p] = 0;
        prm.fval[(int64_t)l * W + p] = (FV)0;
        prm.valid[(int64_t)l * W + p] = 0;
    }
    for (int p = threadIdx.x; p < kLazyBlocks; p += blockDim.x) {
        prm.floorv[(int64_t)l * kLazyBlocks + p] = lowest_value<FV>();
        prm.theta[(int64_t)l * kLazyBlocks + p] = lowest_value<FV>();
    }
    if (threadIdx.x < 4) prm.lazyStat[4 * l + threadIdx.x] = 0;
    if (threadIdx.x == 0) {
        prm.nR[l] = c.M;
        prm.sparseFrom[l] = prm.sparseMinMembers;
        prm.sparseElems[l] = 0;
        prm.hitCount[l] = 0;
        if (c.M > 0) atomicAdd(&prm.nSweep[3], 1);         // classes still to finish
        if (prm.asyncMode == 1) {
            prm.sync[l].epoch = c.M > 0 ? 0 : 1;           // sweep 0 is published by this kernel
            prm.sync[l].done = 0;
            prm.sync[l].seq = l;
            prm.sync[l].nGroups = 0;                       // (plan_decide below sets it)

        }
    }
    __syncthreads();
    plan_load(prm, l, shPlan);
    __syncthreads();
    if (threadIdx.x < 32) plan_decide(prm, l, c, c.M, 0, shPlan);
}

// ---------------------------------------------------------------------------------------------
// Streaming 128-bit load that does not allocate in L1 (S is read once per pass; the coverage
// vectors sit in shared memory).
__device__ __forceinline__ int4 ld_stream(const int4 *p)
{
    int4 v;
    asm("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// The same load as a volatile statement: it stays where it is written (the compiler neither sinks it into the
// branch that uses its result nor merges it with a neighbour), so that several of them are in flight at once.
__device__ __forceinline__ int4 ld_stream_here(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Barrier over the `threads` threads of one team of warps (named barriers 1..15; 0 is the CTA's).
__device__ __forceinline__ void team_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" :: "r"(id), "r"(threads) : "memory");
}

// Sum NA per-lane partials over the 32 lanes so that lane k ends with the total of partial
// k / (32/NA): each step hands half of the values to the partner lane (xor offset) and adds the
// partner's copy of the half that stays, then plain butterflies finish the remaining offsets.
// The order of additions is fixed, so fp32 results are reproducible.
template <typename T, int N>
struct WarpMultiReduce {
    static __device__ __forceinline__ T run(T (&v)[N], int off, int lane)
    {
        T w[N / 2];
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            T send = up ? v[i] : v[i + N / 2];
            T keep = up ? v[i + N / 2] : v[i];
            w[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
        return WarpMultiReduce<T, N / 2>::run(w, off >> 1, lane);
    }
};
template <typename T>
struct WarpMultiReduce<T, 1> {
    static __device__ __forceinline__ T run(T (&v)[1], int off, int lane)
    {
        T x = v[0];
        for (; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
        return x;
    }
};

// acc + x computed as x * one + acc: an integer multiply-add issues on the FMA pipe, so the adds
// of the integer path do not compete with the max operations for the ALU pipe.
__device__ __forceinline__ uint32_t add_on_fma_pipe(uint32_t x, uint32_t one, uint32_t acc)
{
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(x), "r"(one), "r"(acc));
    return r;
}

template <typename SV, int P, int R>
__device__ __forceinline__ void accumulate_chunk(uint32_t one, const int4 (&s)[R], const int4 *shCover, int ld4, int cc,
                                                 typename std::conditional<Arith<SV>::kInt, uint32_t, float>::type (&acc)[P * R])
{
#pragma unroll
    for (int p = 0; p < P; ++p) {
        const int4 m = shCover[p * ld4 + cc];
        if constexpr (Arith<SV>::kInt) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                uint32_t a = acc[r * P + p];
                a = add_on_fma_pipe((uint32_t)max(s[r].x, m.x), one, a);
                a = add_on_fma_pipe((uint32_t)max(s[r].y, m.y), one, a);
                a = add_on_fma_pipe((uint32_t)max(s[r].z, m.z), one, a);
                a = add_on_fma_pipe((uint32_t)max(s[r].w, m.w), one, a);
                acc[r * P + p] = a;
            }
        } else {
            const float m0 = __int_as_float(m.x), m1 = __int_as_float(m.y);
            const float m2 = __int_as_float(m.z), m3 = __int_as_float(m.w);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float a = acc[r * P + p];
                a += fmaxf(__int_as_float(s[r].x) - m0, 0.f);
                a += fmaxf(__int_as_float(s[r].y) - m1, 0.f);
                a += fmaxf(__int_as_float(s[r].z) - m2, 0.f);
                a += fmaxf(__int_as_float(s[r].w) - m3, 0.f);
                acc[r * P + p] = a;
            }
        }
    }
}

// One class, P blocks.  The CTA's 16 warps form teams of CS warps; a team pulls a group of R rows
// from the class's ticket counter and its warps take interleaved 128-column chunks of those rows,
// so that a sweep with few rows left still spreads over every warp of the GPU.  Per-warp partial
// sums meet in shared memory and are added in warp order (fixed, reproducible).
// 16 bytes global -> shared without passing through registers (completion: cp.async.wait_group).
__device__ __forceinline__ void async_copy16(int4 *smemDst, const int4 *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"((uint32_t)__cvta_generic_to_shared(smemDst)), "l"(src) : "memory");
}

// kRing: the rows stream through a per-warp ring of asynchronous copies in shared memory (`ring`, kDenseStages
// chunks of R rows per warp) instead of one register buffer ahead: a warp of a CTA that sweeps a class alone has
// a few hundred instructions of work per chunk, far less than a trip to memory takes, so it needs several
// chunks in flight to keep its issue slots busy.  Each lane reads back only the pieces it copied itself.
constexpr int kDenseStages = 4;
__host__ __device__ inline int dense_ring_bytes(int R) { return (kSweepThreads / 32) * kDenseStages * R * 512; }

template <typename SV, int P, int R, bool kRing = false>
__device__ __forceinline__ void sweep_class(const GreedyParams<SV> &prm, int l, const ClassDesc &c, int nR, int CS,
                                            const int4 *shCover, const long long *shF, const int32_t *parts,
                                            int *shTicket, typename Arith<SV>::GV *shPart,
                                            int32_t *ticket, int32_t *done, int firstTicket, int4 *ring = nullptr)
{
    using GV = typename Arith<SV>::GV;
    using AccT = typename std::conditional<Arith<SV>::kInt, uint32_t, float>::type;
    constexpr int NA = P * R;
    constexpr bool kPrefetch = (R <= 4);          // second register buffer only where it fits
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int team = warp / CS, wIn = warp - team * CS;
    const int teamThreads = CS * 32, barId = 1 + team;
    const int ld4 = c.ld >> 2;
    const int nGroups = (nR + R - 1) / R;
    const int stride = CS * 32;
    const SV *Sl = prm.S + c.sOff;
    const int32_t *cand = prm.cand + c.row0;
    GV *G = prm.gains + c.vOff;
    GV *myPart = shPart + (team * CS) * 32;       // [CS][32] for this team (teams are CS-aligned)
    // `ticket` hands out the row groups.  firstTicket >= 0: the CTA has already drawn one ticket per
    // team (firstTicket + team); `done` (may be null) counts the row groups whose gains are written.
    bool preDrawn = firstTicket >= 0;
    int finished = 0;                             // row groups of this sweep this team has completed

    for (;;) {
        int g = 0;
        if (preDrawn) {
            g = firstTicket + team;
            preDrawn = false;
        } else if (CS == 1) {
            if (lane == 0) g = atomicAdd(ticket, 1);
            g = __shfl_sync(0xffffffffu, g, 0);
        } else {
            if (wIn == 0 && lane == 0) shTicket[team] = atomicAdd(ticket, 1);
            team_sync(barId, teamThreads);
            g = shTicket[team];
        }
        if (g >= nGroups) break;
        const int k0 = g * R;
        int vrow[R];
        const int4 *rp[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            int k = k0 + r;
            vrow[r] = __ldcg(cand + (k < nR ? k : nR - 1));
            rp[r] = reinterpret_cast<const int4 *>(Sl + (int64_t)vrow[r] * c.ld);
        }
        GV total;
        const int first = wIn * 32 + lane;
        // (kRing) this lane's chunks c0, c0 + stride, ... below cEnd through the warp's ring, kDenseStages - 1 ahead
        auto ring_stream = [&](int c0, int cEnd, AccT (&acc)[NA]) {
            int4 *rg = ring + (threadIdx.x >> 5) * (kDenseStages * R * 32) + lane;
            int ci = c0;
#pragma unroll
            for (int st = 0; st < kDenseStages - 1; ++st) {
                if (ci < cEnd) {
#pragma unroll
                    for (int r = 0; r < R; ++r) async_copy16(rg + (st * R + r) * 32, rp[r] + ci);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                ci += stride;
            }
            int stage = 0;
            for (int cc = c0; cc < cEnd; cc += stride) {
                int ahead = stage + kDenseStages - 1;
                if (ahead >= kDenseStages) ahead -= kDenseStages;
                if (ci < cEnd) {
#pragma unroll
                    for (int r = 0; r < R; ++r) async_copy16(rg + (ahead * R + r) * 32, rp[r] + ci);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                ci += stride;
                asm volatile("cp.async.wait_group %0;" :: "n"(kDenseStages - 1) : "memory");
                int4 sr[R];
#pragma unroll
                for (int r = 0; r < R; ++r) sr[r] = rg[(stage * R + r) * 32];
                accumulate_chunk<SV, P, R>(prm.one, sr, shCover, ld4, cc, acc);
                if (++stage == kDenseStages) stage = 0;
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        };
        (void)ring_stream;
        if constexpr (Arith<SV>::kInt) {
            // sum_i max(S[v][i], cover[i]) in unsigned 32-bit partials (every term is in [0, 2^31)),
            // widened to 64 bits every segIters iterations; the gain is that sum minus f_p.
            unsigned long long tot = 0;
            // every lane runs every segment (the shuffles below need the whole warp), whether or
            // not its own columns reach into it
            const int segLen = prm.segIters * stride;
            for (int base = 0; base < ld4; base += segLen) {
                AccT acc[NA];
#pragma unroll
                for (int i = 0; i < NA; ++i) acc[i] = 0u;
                const int c0 = base + first;
                const int cEnd = min(ld4, base + segLen);
                if constexpr (kRing) {
                    ring_stream(c0, cEnd, acc);
                } else if constexpr (kPrefetch) {
                    int4 cur[R], nxt[R];
                    if (c0 < cEnd) {
#pragma unroll
                        for (int r = 0; r < R; ++r) cur[r] = ld_stream(rp[r] + c0);
                    }
                    for (int cc = c0; cc < cEnd; cc += stride) {
                        const int cn = cc + stride;
                        if (cn < cEnd) {
#pragma unroll
                            for (int r = 0; r < R; ++r) nxt[r] = ld_stream(rp[r] + cn);
                        }
                        accumulate_chunk<SV, P, R>(prm.one, cur, shCover, ld4, cc, acc);
#pragma unroll
                        for (int r = 0; r < R; ++r) cur[r] = nxt[r];
                    }
                } else {
                    for (int cc = c0; cc < cEnd; cc += stride) {
                        int4 s[R];
#pragma unroll
                        for (int r = 0; r < R; ++r) s[r] = ld_stream(rp[r] + cc);
                        accumulate_chunk<SV, P, R>(prm.one, s, shCover, ld4, cc, acc);
                    }
                }
                unsigned long long wide[NA / 2];
                {
                    const bool up = (lane & 16) != 0;
#pragma unroll
                    for (int i = 0; i < NA / 2; ++i) {
                        uint32_t send = up ? acc[i] : acc[i + NA / 2];
                        uint32_t keep = up ? acc[i + NA / 2] : acc[i];
                        wide[i] = (unsigned long long)keep + (unsigned long long)__shfl_xor_sync(0xffffffffu, send, 16);
                    }
                }
                tot += WarpMultiReduce<unsigned long long, NA / 2>::run(wide, 8, lane);
            }
            total = (GV)tot;
        } else {
            AccT acc[NA];
#pragma unroll
            for (int i = 0; i < NA; ++i) acc[i] = 0.f;
            if constexpr (kRing) {
                ring_stream(first, ld4, acc);
            } else if constexpr (kPrefetch) {
                int4 cur[R], nxt[R];
                if (first < ld4) {
#pragma unroll
                    for (int r = 0; r < R; ++r) cur[r] = ld_stream(rp[r] + first);
                }
                for (int cc = first; cc < ld4; cc += stride) {
                    const int cn = cc + stride;
                    if (cn < ld4) {
#pragma unroll
                        for (int r = 0; r < R; ++r) nxt[r] = ld_stream(rp[r] + cn);
                    }
                    accumulate_chunk<SV, P, R>(prm.one, cur, shCover, ld4, cc, acc);
#pragma unroll
                    for (int r = 0; r < R; ++r) cur[r] = nxt[r];
                }
            } else {
                for (int cc = first; cc < ld4; cc += stride) {
                    int4 s[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) s[r] = ld_stream(rp[r] + cc);
                    accumulate_chunk<SV, P, R>(prm.one, s, shCover, ld4, cc, acc);
                }
            }
            total = WarpMultiReduce<float, NA>::run(acc, 16, lane);
        }
        // lane k holds partial k / (32/NA) = r * P + p of this warp's columns
        if (CS > 1) {
            myPart[wIn * 32 + lane] = total;
            team_sync(barId, teamThreads);
            if (wIn == 0) {
                GV sum = myPart[lane];
                for (int w = 1; w < CS; ++w) sum += myPart[w * 32 + lane];
                total = sum;
            }
        }
        constexpr int kShare = 32 / NA;
        if (wIn == 0 && (lane % kShare) == 0) {
            const int idx = lane / kShare;
            const int r = idx / P, p = idx % P;
            if (k0 + r < nR) {
                GV gain;
                if constexpr (Arith<SV>::kInt) gain = total - shF[p];
                else gain = total;
                int row = 0;
#pragma unroll
                for (int q = 0; q < R; ++q) if (q == r) row = vrow[q];
                G[(int64_t)parts[p] * c.ld + row] = gain;
            }
        }
        ++finished;
    }
    // The row groups this team finished are reported together, once the sweep's tickets have run out for it: the
    // class's pick CTA only needs the total, and one fence then covers the gains of all of them.
    if (done != nullptr && wIn == 0 && finished > 0) {
        __syncwarp();
        if (lane == 0) { __threadfence(); atomicAdd(done, finished); }
    }
}

// Threshold pass over one class.  shThr[i] = min over the P listed blocks of cover_p[i]: an element
// S[v][i] <= shThr[i] adds nothing to any listed block's gain, and once the blocks have some
// members that is true of all but a few elements per row.  The warp therefore only compares its R
// rows against the threshold (one compare per element, whatever P is) and appends the elements
// above it to a small queue in shared memory.  The queue is drained with the lanes arranged as
// (queue slot, block): lane (s, p) fetches cover_p[i] for the s-th queued element and adds
// max(0, S[v][i] - cover_p[i]) to its running sum for that element's row, so 32 / P' elements
// (P' = P rounded up to a power of two) are in flight at once.  The slots' sums are added at the
// end of the row group.  With more than 32 blocks every lane serves blocks p and p + 32.

// What a warp of a threshold pass keeps for the whole pass.
template <typename SV, int A>
struct SparseWarp {
    int4 *ring;                 // the warp's ring of chunks of S
    uint2 *queue;               // the warp's queue of elements above the threshold
    const int4 *shThr;          // threshold vector (shared memory)
    int ld4, lane;
    unsigned below;             // lanes below this one
    int Pp, slots, slot;        // lanes per queue slot, slots, this lane's slot
    int myPart[A];              // blocks this lane serves (-1: none)
    const SV *myCov[A];         // their coverage vectors
};

template <typename SV, int A>
__device__ __forceinline__ void sparse_setup(SparseWarp<SV, A> &w, const GreedyParams<SV> &prm, const ClassDesc &c, int P,
                                             const int4 *shThr, const int32_t *parts, uint2 *warpArea)
{
    w.ring = reinterpret_cast<int4 *>(warpArea);                    // per warp: ring, then queue
    w.queue = warpArea + kSparseRingBytes / 8;
    w.shThr = shThr;
    w.ld4 = c.ld >> 2;
    w.lane = threadIdx.x & 31;
    w.below = (1u << w.lane) - 1u;
    const SV *cover = prm.cover + c.vOff;
    int Pp = 1;                                                     // lanes per queue slot
    while (Pp < P && Pp < 32) Pp *= 2;
    w.Pp = Pp;
    w.slots = 32 / Pp;
    w.slot = w.lane / Pp;
#pragma unroll
    for (int a = 0; a < A; ++a) {
        const int p = (w.lane & (Pp - 1)) + 32 * a;
        w.myPart[a] = p < P ? parts[p] : -1;
        w.myCov[a] = cover + (int64_t)(w.myPart[a] < 0 ? parts[0] : w.myPart[a]) * c.ld;
    }
}

// Adds the queued elements to the lanes' running sums: lane (slot, block) fetches the block's coverage of the
// element's column and adds max(0, S - cover) to the sum of the element's row.
template <typename SV, int A>
__device__ __forceinline__ void sparse_drain(const SparseWarp<SV, A> &w, int &qn, typename Arith<SV>::GV (&acc)[kSparseRows][A])
{
    using GV = typename Arith<SV>::GV;
    constexpr int R = kSparseRows;
    __syncwarp();
    for (int i0 = w.slot; i0 < qn; i0 += 2 * w.slots) {
        uint2 e[2];
        bool ok[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int i = i0 + u * w.slots;
            ok[u] = i < qn;
            e[u] = w.queue[ok[u] ? i : i0];
        }
        GV d[2][A];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int col = (int)(e[u].x & 0x0fffffffu);
#pragma unroll
            for (int a = 0; a < A; ++a) {
                const SV cv = __ldcg(w.myCov[a] + col);
                if constexpr (Arith<SV>::kInt) {
                    const int dd = (int)e[u].y - cv;
                    d[u][a] = (ok[u] && w.myPart[a] >= 0 && dd > 0) ? (GV)dd : (GV)0;
                } else {
                    const float dd = __uint_as_float(e[u].y) - cv;
                    d[u][a] = (ok[u] && w.myPart[a] >= 0 && dd > 0.f) ? dd : 0.f;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int r = (int)(e[u].x >> 28);
#pragma unroll
            for (int rr = 0; rr < R; ++rr)
#pragma unroll
                for (int a = 0; a < A; ++a) acc[rr][a] += (r == rr) ? d[u][a] : (GV)0;
        }
    }
    __syncwarp();
    qn = 0;
}

// Streams nRows (<= kSparseRows) rows of S against the threshold vector: elements above it are queued and the
// queue is drained into acc whenever it is nearly full.  On return every copy has landed and the last
// elements are still in the queue (qn of them): the caller drains them when it has issued what it wants to
// overlap with that.
// S streams through a ring in shared memory filled by asynchronous copies, kSparseStages - 1 chunks ahead;
// every lane reads back only the 16-byte pieces it copied itself, so waiting for its own copy groups is all
// the synchronisation the ring needs.
template <typename SV, int A>
__device__ __forceinline__ void sparse_stream(const SparseWarp<SV, A> &w, const int4 *const (&rp)[kSparseRows], int nRows,
                                              typename Arith<SV>::GV (&acc)[kSparseRows][A], unsigned &hits, int &qn)
{
    constexpr int R = kSparseRows;
    const int lane = w.lane, ld4 = w.ld4;
    auto issue = [&](int base, int st) {
        const int cc = base + lane;
        if (cc < ld4) {
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (r < nRows) async_copy16(w.ring + (st * R + r) * 32 + lane, rp[r] + cc);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
#pragma unroll
    for (int st = 0; st < kSparseStages - 1; ++st) issue(st * 32, st);
    int stage = 0;
    for (int base = 0; base < ld4; base += 32) {                // every lane runs every chunk: ballots below
        const int cc = base + lane;
        const bool inside = cc < ld4;
        {
            int ahead = stage + kSparseStages - 1;
            if (ahead >= kSparseStages) ahead -= kSparseStages;
            issue(base + (kSparseStages - 1) * 32, ahead);       // past the row's end: an empty group
        }
        asm volatile("cp.async.wait_group %0;" :: "n"(kSparseStages - 1) : "memory");
        int4 t = make_int4(0, 0, 0, 0);
        if (inside) t = w.shThr[cc];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            int4 s = make_int4(0, 0, 0, 0);
            unsigned h = 0;
            if (inside && r < nRows) {
                s = w.ring[(stage * R + r) * 32 + lane];
                if constexpr (Arith<SV>::kInt) {
                    h = (s.x > t.x ? 1u : 0u) | (s.y > t.y ? 2u : 0u) | (s.z > t.z ? 4u : 0u) | (s.w > t.w ? 8u : 0u);
                } else {
                    h = (__int_as_float(s.x) > __int_as_float(t.x) ? 1u : 0u) | (__int_as_float(s.y) > __int_as_float(t.y) ? 2u : 0u) |
                        (__int_as_float(s.z) > __int_as_float(t.z) ? 4u : 0u) | (__int_as_float(s.w) > __int_as_float(t.w) ? 8u : 0u);
                }
            }
            if (__any_sync(0xffffffffu, h != 0)) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool mine = (h >> e) & 1u;
                    const unsigned m = __ballot_sync(0xffffffffu, mine);
                    if (mine) {
                        const int sv = e == 0 ? s.x : (e == 1 ? s.y : (e == 2 ? s.z : s.w));
                        w.queue[qn + __popc(m & w.below)] = make_uint2((unsigned)(cc * 4 + e) | ((unsigned)r << 28), (unsigned)sv);
                    }
                    qn += __popc(m);
                }
                if (qn > kSparseQueue - 128) { hits += qn; sparse_drain<SV, A>(w, qn, acc); }
            }
        }
        if (++stage == kSparseStages) stage = 0;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

template <typename SV, int A>
__device__ __noinline__ void sweep_class_sparse(const GreedyParams<SV> &prm, int l, const ClassDesc c, int nR, int P,
                                                   const int4 *shThr, const int32_t *parts, uint2 *queue,
                                                   int32_t *ticket, int32_t *done, int firstTicket)
{
    using GV = typename Arith<SV>::GV;
    constexpr int R = kSparseRows;
    SparseWarp<SV, A> w;
    sparse_setup<SV, A>(w, prm, c, P, shThr, parts, queue);
    const int lane = w.lane;
    const int nGroups = (nR + R - 1) / R;
    const SV *Sl = prm.S + c.sOff;
    const int32_t *cand = prm.cand + c.row0;
    GV *G = prm.gains + c.vOff;
    unsigned hits = 0;
    int finished = 0;                                               // row groups of this sweep this warp has completed
    // The warp's ticket (firstTicket >= 0: one per warp was drawn by the CTA) and the rows it names.  The next
    // ticket is drawn while the current rows stream, and its row indices are loaded under the drain and the
    // stores that end a row group, so that neither trip to memory is waited for between two row groups.
    int g = 0;
    if (firstTicket >= 0) {
        g = firstTicket + (threadIdx.x >> 5);
    } else {
        if (lane == 0) g = atomicAdd(ticket, 1);
        g = __shfl_sync(0xffffffffu, g, 0);
    }
    int rowOf[R];
#pragma unroll
    for (int r = 0; r < R; ++r) rowOf[r] = 0;
    if (g < nGroups) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int k = g * R + r;
            rowOf[r] = __ldcg(cand + (k < nR ? k : nR - 1));
        }
    }
    for (;;) {
        if (g >= nGroups) break;
        const int k0 = g * R;
        const int4 *rp[R];
#pragma unroll
        for (int r = 0; r < R; ++r) rp[r] = reinterpret_cast<const int4 *>(Sl + (int64_t)rowOf[r] * c.ld);
        int gDrawn = 0;
        if (lane == 0) gDrawn = atomicAdd(ticket, 1);
        GV acc[R][A];                                               // running sums of this lane, [row][block of the lane]
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int a = 0; a < A; ++a) acc[r][a] = 0;
        int qn = 0;                                                 // queued elements (same in every lane)
        sparse_stream<SV, A>(w, rp, R, acc, hits, qn);
        const int gNext = __shfl_sync(0xffffffffu, gDrawn, 0);
        int rowNext[R];
#pragma unroll
        for (int r = 0; r < R; ++r) rowNext[r] = 0;
        if (gNext < nGroups) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int k = gNext * R + r;
                rowNext[r] = __ldcg(cand + (k < nR ? k : nR - 1));
            }
        }
        if (qn) { hits += qn; sparse_drain<SV, A>(w, qn, acc); }
#pragma unroll
        for (int r = 0; r < R; ++r) {
#pragma unroll
            for (int a = 0; a < A; ++a) {
                GV t = acc[r][a];
                for (int off = w.Pp; off < 32; off <<= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
                if (w.slot == 0 && k0 + r < nR && w.myPart[a] >= 0) G[(int64_t)w.myPart[a] * c.ld + rowOf[r]] = t;
            }
        }
        ++finished;
        g = gNext;
#pragma unroll
        for (int r = 0; r < R; ++r) rowOf[r] = rowNext[r];
    }
    if (done != nullptr) {
        // The row groups this warp finished are reported together, once the sweep's tickets have run out for it (the
        // class's pick CTA only needs the total); their hit count and gains are in place before they count as done.
        if (finished > 0) {
            __syncwarp();
            if (lane == 0) {
                if (hits) atomicAdd(&prm.hitCount[l], (unsigned long long)hits);
                __threadfence();
                atomicAdd(done, finished);
            }
        }
    } else if (lane == 0 && hits) {
        atomicAdd(&prm.hitCount[l], (unsigned long long)hits);
    }
}

// Row-skipping threshold pass (the exact lazy rule for GreedyStep's argmax).  A stored gain of a block that has
// grown since it was computed is an upper bound of the current gain (diminishing returns), so a row whose
// stored gains lie below the floors of all listed blocks (shTheta[k] for parts[k]) cannot be needed before
// those floors are lowered: it is left out and keeps its upper bounds.  Every other row is recomputed for all
// listed blocks, exactly as in sweep_class_sparse.  Afterwards every stored gain of parts[k] at or above
// shTheta[k] is exact: an entry that was not recomputed was below the floor and still is.
// A ticket stands for kLazyRows consecutive entries of the candidate list, one per lane; the lanes look their
// rows' stored gains up, and the warp then streams the rows that are needed, two at a time.
template <typename SV, int A>
__device__ __noinline__ void sweep_class_lazy(const GreedyParams<SV> &prm, int l, const ClassDesc c, int nR, int P,
                                                 const int4 *shThr, const int32_t *parts, const typename Arith<SV>::GV *shTheta,
                                                 uint2 *queue, int32_t *ticket, int32_t *done, int firstTicket)
{
    using GV = typename Arith<SV>::GV;
    constexpr int R = kSparseRows;
    SparseWarp<SV, A> w;
    sparse_setup<SV, A>(w, prm, c, P, shThr, parts, queue);
    const int lane = w.lane;
    const int nTickets = (nR + kLazyRows - 1) / kLazyRows;
    const SV *Sl = prm.S + c.sOff;
    const int32_t *cand = prm.cand + c.row0;
    GV *G = prm.gains + c.vOff;
    unsigned hits = 0;
    int finished = 0, rowsRead = 0, rowsSeen = 0;
    int g = 0;
    if (firstTicket >= 0) {
        g = firstTicket + (threadIdx.x >> 5);
    } else {
        if (lane == 0) g = atomicAdd(ticket, 1);
        g = __shfl_sync(0xffffffffu, g, 0);
    }
    while (g < nTickets) {
        int gDrawn = 0;
        if (lane == 0) gDrawn = atomicAdd(ticket, 1);               // (the next ticket: in flight under this one's work)
        const int k = g * kLazyRows + lane;
        const int v = k < nR ? __ldcg(cand + k) : -1;
        bool need = false;
        if (v >= 0) {
            for (int k0 = 0; k0 < P; k0 += 4) {                     // four independent look-ups at a time
                GV b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) b[u] = __ldcg(G + (int64_t)parts[k0 + u < P ? k0 + u : 0] * c.ld + v);
#pragma unroll
                for (int u = 0; u < 4; ++u) need = need || (k0 + u < P && b[u] >= shTheta[k0 + u]);
            }
        }
        unsigned mask = __ballot_sync(0xffffffffu, need);
        rowsSeen += __popc(__ballot_sync(0xffffffffu, v >= 0));
        while (mask) {
            const int i0 = __ffs(mask) - 1;
            mask &= mask - 1;
            int i1 = i0, nRows = 1;
            if (mask) { i1 = __ffs(mask) - 1; mask &= mask - 1; nRows = 2; }
            int rowOf[R];
            rowOf[0] = __shfl_sync(0xffffffffu, v, i0);
            rowOf[1] = __shfl_sync(0xffffffffu, v, i1);
            const int4 *rp[R];
#pragma unroll
            for (int r = 0; r < R; ++r) rp[r] = reinterpret_cast<const int4 *>(Sl + (int64_t)rowOf[r] * c.ld);
            GV acc[R][A];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int a = 0; a < A; ++a) acc[r][a] = 0;
            int qn = 0;
            sparse_stream<SV, A>(w, rp, nRows, acc, hits, qn);
            if (qn) { hits += qn; sparse_drain<SV, A>(w, qn, acc); }
#pragma unroll
            for (int r = 0; r < R; ++r) {
#pragma unroll
                for (int a = 0; a < A; ++a) {
                    GV t = acc[r][a];
                    for (int off = w.Pp; off < 32; off <<= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
                    if (w.slot == 0 && r < nRows && w.myPart[a] >= 0) G[(int64_t)w.myPart[a] * c.ld + rowOf[r]] = t;
                }
            }
            rowsRead += nRows;
        }
        ++finished;
        g = __shfl_sync(0xffffffffu, gDrawn, 0);
    }
    if (finished > 0) {
        __syncwarp();
        if (lane == 0) {
            atomicAdd(&prm.phaseNs[10], (unsigned long long)rowsRead);
            atomicAdd(&prm.phaseNs[11], (unsigned long long)(rowsSeen - rowsRead));
            atomicAdd(&prm.phaseNs[12], (unsigned long long)rowsRead * (unsigned long long)c.ld * sizeof(SV));
            if (done != nullptr) {
                __threadfence();                                    // the gains are in place before the tickets count as done
                atomicAdd(done, finished);
            }
        }
    }
}

// Shared-memory arrays a CTA needs to serve sweeps (beside the dynamic area that holds the coverage vectors).
template <typename SV>
struct SweepShared {
    long long f[kMaxSweepBatch];
    int32_t parts[kSparseMax];
    typename Arith<SV>::GV theta[kLazyBlocks];
    int ticket[kSweepThreads / 32];
    typename Arith<SV>::GV part[kSweepThreads];
};

// One CTA (kSweepThreads threads) works on the scheduled sweep of class l until its tickets run out: stages the
// coverage vectors (or the threshold vector) of the listed blocks in shCover and calls the pass the class asked for.
// Several CTAs may serve the same sweep; they share its ticket counter rowCtr[l].
template <typename SV>
__device__ __forceinline__ void sweep_serve_class(const GreedyParams<SV> &prm, int l, int4 *shCover, SweepShared<SV> &sh)
{
    const ClassDesc c = prm.desc[l];
    const int nR = prm.nR[l];
    const int P = prm.sweepN[l];
    const int CS = prm.sweepCS[l];
    const int ld4 = c.ld >> 2;
    const int32_t *parts = prm.sweepParts + (int64_t)l * kSparseMax;
    if (prm.sweepMode[l]) {
        // threshold pass: one vector in shared memory, the blocks' coverage stays in global memory
        const int4 *thr = reinterpret_cast<const int4 *>(prm.thr + c.vOff / prm.W);
        for (int i = threadIdx.x; i < ld4; i += blockDim.x) shCover[i] = thr[i];
        const bool lazy = prm.sweepMode[l] == 2;
        if (threadIdx.x < P) {
            sh.parts[threadIdx.x] = parts[threadIdx.x];
            if (lazy) sh.theta[threadIdx.x] = prm.sweepTheta[(int64_t)l * kLazyBlocks + threadIdx.x];
        }
        __syncthreads();
        uint2 *queue = reinterpret_cast<uint2 *>(reinterpret_cast<char *>(shCover) + thr_bytes_aligned(c.ld * (int)sizeof(SV)) + (threadIdx.x >> 5) * kSparseWarpBytes);
        if (lazy) {
            if (P <= 32) sweep_class_lazy<SV, 1>(prm, l, c, nR, P, shCover, sh.parts, sh.theta, queue, &prm.rowCtr[l], nullptr, -1);
            else sweep_class_lazy<SV, 2>(prm, l, c, nR, P, shCover, sh.parts, sh.theta, queue, &prm.rowCtr[l], nullptr, -1);
        } else if (P <= 32) sweep_class_sparse<SV, 1>(prm, l, c, nR, P, shCover, sh.parts, queue, &prm.rowCtr[l], nullptr, -1);
        else sweep_class_sparse<SV, 2>(prm, l, c, nR, P, shCover, sh.parts, queue, &prm.rowCtr[l], nullptr, -1);
    } else {
        const int4 *cov = reinterpret_cast<const int4 *>(prm.cover + c.vOff);
        for (int i = threadIdx.x; i < P * ld4; i += blockDim.x) {
            int p = i / ld4, cc = i - p * ld4;
            shCover[i] = cov[(int64_t)parts[p] * ld4 + cc];
        }
        if (threadIdx.x < P) {
            sh.parts[threadIdx.x] = parts[threadIdx.x];
            if constexpr (Arith<SV>::kInt) sh.f[threadIdx.x] = prm.fval[(int64_t)l * prm.W + parts[threadIdx.x]];
        }
        __syncthreads();
        switch (P) {
        case 1: sweep_class<SV, 1, 8>(prm, l, c, nR, CS, shCover, sh.f, sh.parts, sh.ticket, sh.part, &prm.rowCtr[l], nullptr, -1); break;
        case 2: sweep_class<SV, 2, 8>(prm, l, c, nR, CS, shCover, sh.f, sh.parts, sh.ticket, sh.part, &prm.rowCtr[l], nullptr, -1); break;
        case 4: sweep_class<SV, 4, 8>(prm, l, c, nR, CS, shCover, sh.f, sh.parts, sh.ticket, sh.part, &prm.rowCtr[l], nullptr, -1); break;
        default: {
            const int covBytes = thr_bytes_aligned(8 * c.ld * (int)sizeof(SV));
            if (prm.denseRing && covBytes + dense_ring_bytes(4) <= prm.smemBytes)
                sweep_class<SV, 8, 4, true>(prm, l, c, nR, CS, shCover, sh.f, sh.parts, sh.ticket, sh.part, &prm.rowCtr[l], nullptr, -1,
                                            reinterpret_cast<int4 *>(reinterpret_cast<char *>(shCover) + covBytes));
            else
                sweep_class<SV, 8, 4>(prm, l, c, nR, CS, shCover, sh.f, sh.parts, sh.ticket, sh.part, &prm.rowCtr[l], nullptr, -1);
            break;
        }
        }
    }
    __syncthreads();
}

// The sweep of greedy step `step`, run by every CTA of the launch (kSweepThreads threads each).
template <typename SV>
__device__ __forceinline__ void sweep_step(const GreedyParams<SV> &prm, int step, int4 *shCover)
{
    __shared__ SweepShared<SV> shSweep;
    __shared__ int shGo;
    // three lists in rotation: this step reads list step%3, its picks fill (step+1)%3, and the one
    // after that is cleared here, a full step (and at least one barrier / launch boundary) before use
    const int par = step % 3;
    const int nS = prm.nSweep[par];
    if (blockIdx.x == 0 && threadIdx.x == 0) prm.nSweep[(step + 2) % 3] = 0;
    if (nS == 0) return;
    // Every CTA has a home position in the list (CTAs spread evenly over the sweeping classes) and
    // serves, again and again, the nearest class at or after it that still has row groups to hand
    // out.  One parallel look at all ticket counters finds that class; a class whose tickets have
    // run out stays that way for the rest of the round, so the loop ends.
    const int start = (int)(((int64_t)blockIdx.x * nS) / gridDim.x);
    for (;;) {
        if (threadIdx.x == 0) shGo = INT_MAX;
        __syncthreads();
        for (int s = threadIdx.x; s < nS; s += blockDim.x) {
            const int ls = prm.sweepList[(int64_t)par * prm.L + s];
            const int ms = prm.sweepMode[ls];
            const int Rs = ms == 2 ? kLazyRows : (ms ? kSparseRows : rows_per_group(prm.sweepN[ls]));
            const int groups = (prm.nR[ls] + Rs - 1) / Rs;
            if (*(volatile int32_t *)&prm.rowCtr[ls] < groups) {
                int dist = s - start;
                if (dist < 0) dist += nS;
                atomicMin(&shGo, dist);
            }
        }
        __syncthreads();
        const int go = shGo;
        if (go == INT_MAX) break;
        int s = start + go;
        if (s >= nS) s -= nS;
        sweep_serve_class(prm, prm.sweepList[(int64_t)par * prm.L + s], shCover, shSweep);
    }
}

template <typename SV>
__global__ void __launch_bounds__(kSweepThreads, 1) sweep_kernel(const __grid_constant__ GreedyParams<SV> prm, int step)
{
    extern __shared__ __align__(128) int4 shCover[];
    cudaGridDependencySynchronize();              // the previous launch (select / init) has finished
    cudaTriggerProgrammaticLaunchCompletion();
    sweep_step(prm, step, shCover);
}

// ---------------------------------------------------------------------------------------------
// Element-wise maximum of two 16-byte pieces (int32 or fp32 lanes).
template <typename SV>
__device__ __forceinline__ int4 max_int4(int4 a, int4 b)
{
    if constexpr (Arith<SV>::kInt) {
        a.x = max(a.x, b.x); a.y = max(a.y, b.y); a.z = max(a.z, b.z); a.w = max(a.w, b.w);
    } else {
        a.x = __float_as_int(fmaxf(__int_as_float(a.x), __int_as_float(b.x)));
        a.y = __float_as_int(fmaxf(__int_as_float(a.y), __int_as_float(b.y)));
        a.z = __float_as_int(fmaxf(__int_as_float(a.z), __int_as_float(b.z)));
        a.w = __float_as_int(fmaxf(__int_as_float(a.w), __int_as_float(b.w)));
    }
    return a;
}

template <typename SV>
__device__ __forceinline__ int4 min_int4(int4 a, int4 b)
{
    if constexpr (Arith<SV>::kInt) {
        a.x = min(a.x, b.x); a.y = min(a.y, b.y); a.z = min(a.z, b.z); a.w = min(a.w, b.w);
    } else {
        a.x = __float_as_int(fminf(__int_as_float(a.x), __int_as_float(b.x)));
        a.y = __float_as_int(fminf(__int_as_float(a.y), __int_as_float(b.y)));
        a.z = __float_as_int(fminf(__int_as_float(a.z), __int_as_float(b.z)));
        a.w = __float_as_int(fminf(__int_as_float(a.w), __int_as_float(b.w)));
    }
    return a;
}


// Finishes a coverage update whose operands were copied to shared memory earlier (row v* in
// scratch[0, ld4), the old coverage in scratch[ld4, 2 ld4)): dst[i] = max of the two.
// thrAcc (may be null): running element-wise minimum of the coverage vectors updated in this chain.
template <typename SV>
__device__ __forceinline__ void fold_pending(int4 *dst, const int4 *scratch, int ld4, int4 *thrAcc)
{
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    for (int i = threadIdx.x; i < ld4; i += kSelectThreads) {
        const int4 m = max_int4<SV>(scratch[ld4 + i], scratch[i]);
        dst[i] = m;
        if (thrAcc) thrAcc[i] = min_int4<SV>(thrAcc[i], m);
    }
}

// The picks of class l in round `round`, by one CTA of kSelectThreads threads: pick after pick
// (GreedyStep's argmax over the stored gains of the chosen block, then the bookkeeping of
// Algorithm 1's "A := A u {v*}, R := R \ {v*}" and the choice of the next block) until the next
// block's stored gains are out of date -- then a sweep is scheduled for round + 1 -- or the class
// is finished.  Inside the chain nothing waits on the coverage update: a pick only needs stored
// gains, so row v* is folded into the coverage vector while the next block is being chosen.
// own: 0 = the CTA may serve other classes between two chains of this one (all state is read from and
// written to global memory); 1 / 2 = the CTA serves this class only, first / later chain: the block table,
// the candidate list with its inverse, the dataset indices of the class's samples and the chain's loop
// state (keep[0] = samples left, keep[1] = next block) stay in shared memory between chains, so that a
// pick waits for one trip to memory only -- the loads of the stored gains, served by L2 (ld.cg).
constexpr int kPickMiss = -2;      // shPick: the best stored gain was not known to be exact

// Incremental update of stored gains.  When block j receives v*, its coverage rises from o_i to n_i = S[v*][i] in the
// columns i where S[v*][i] > o_i, and nowhere else.  The gain of a candidate v for j is sum_i max(0, S[v][i] - cover_i),
// so it falls by exactly
//     max(0, S[v][i] - o_i) - max(0, S[v][i] - n_i)
// for each such column, and S[v][i] = S[i][v] (S is symmetric: a Gram matrix): one row of S per risen column, read
// contiguously, updates the gains of all candidates at once.  Once a block has a few members a pick raises a handful
// of columns, so the block's stored gains stay exact for the price of a few rows instead of a pass over all of S.
constexpr int kDeltaMax = 128;     // columns one pick may raise and still be handled this way
template <typename SV>
__device__ __forceinline__ typename Arith<SV>::GV delta_term(int x, int o, int n)
{
    using GV = typename Arith<SV>::GV;
    if constexpr (Arith<SV>::kInt) {
        const GV a = (GV)x - (GV)o, b = (GV)x - (GV)n;
        return (a > 0 ? a : (GV)0) - (b > 0 ? b : (GV)0);
    } else {
        const float xf = __int_as_float(x);
        return fmaxf(xf - __int_as_float(o), 0.f) - fmaxf(xf - __int_as_float(n), 0.f);
    }
}
template <typename SV>
__device__ __forceinline__ bool rose(int r, int o)
{
    if constexpr (Arith<SV>::kInt) return r > o;
    else return __int_as_float(r) > __int_as_float(o);
}

// A (gain, index) pair as one key, for classes of at most 8192 samples: a greater key is a greater gain, or the same gain
// at a lower index; 0 means none.  Integer gains (never negative, far below 2^50 for such classes): gain << 13 |
// (8191 - index).  fp32 gains: order-preserving image of the gain << 32 | (8191 - index).
__device__ __forceinline__ unsigned long long note_key(long long gain, int v) { return ((unsigned long long)gain << 13) | (unsigned long long)(8191 - v); }
__device__ __forceinline__ unsigned long long note_key(float gain, int v) { return ((unsigned long long)ordered_u32(gain) << 32) | (unsigned long long)(8191 - v); }
__device__ __forceinline__ int key_index(unsigned long long key) { return 8191 - (int)(key & 8191ull); }
__device__ __forceinline__ void key_gain(unsigned long long key, long long &g) { g = (long long)(key >> 13); }
__device__ __forceinline__ void key_gain(unsigned long long key, float &g) { g = from_ordered_u32((unsigned)(key >> 32)); }

// kDelta: compiled with the incremental update of stored gains.
template <typename SV, bool kDelta = false>
__device__ __forceinline__ void pick_chain(const GreedyParams<SV> &prm, int l, int round, int4 *scratch, int scratchBytes,
                                           int own = 0, int *keep = nullptr)
{
    using GV = typename Arith<SV>::GV;
    using FV = typename Arith<SV>::FV;
    __shared__ PlanShared<FV> shPlan;
    __shared__ GV shG[kSelectThreads / 32];
    __shared__ int shV[kSelectThreads / 32];
    __shared__ unsigned long long shKey[kSelectThreads / 32];
    __shared__ int shPick;
    const ClassDesc c = prm.desc[l];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ld4 = c.ld >> 2;
    // resident state: behind the three ld-sized pieces of the scratch area used below
    const bool res = own != 0 && keep != nullptr && scratch != nullptr && (int64_t)6 * c.ld * (int64_t)sizeof(SV) <= scratchBytes;
    int32_t *shPos = reinterpret_cast<int32_t *>(scratch + 3 * ld4);
    int32_t *shCand = shPos + c.ld;
    int32_t *shPerm = shCand + c.ld;
    int nR, j;
    if (res && own == 2) {
        nR = keep[0];
        j = keep[1];
    } else {
        nR = prm.nR[l];
        j = prm.jstar[l];
    }
    if (nR == 0 || j < 0) {
        if (keep && threadIdx.x == 0) { keep[0] = nR; keep[1] = j; }
        return;
    }
    int32_t *cand = prm.cand + c.row0;
    int32_t *pos = prm.pos + c.row0;
    __shared__ int32_t shChain[kSparseMax];         // blocks that received a sample in this chain
    __shared__ int shChainOk;
    if (!(res && own == 2)) {
        plan_load(prm, l, shPlan);
        if (res) {
            for (int v = threadIdx.x; v < c.M; v += kSelectThreads) {
                shPos[v] = pos[v];
                shCand[v] = cand[v];
                shPerm[v] = prm.perm[c.row0 + v];
            }
        }
        __syncthreads();
    }
    // Folding row v* into the coverage vector is off the critical path (a pick reads stored gains,
    // never the coverage).  When the caller lends enough shared memory, row v* and the coverage
    // vector are fetched with asynchronous copies once v* is known, and the max/store happens one
    // pick later, after the next argmax; each thread consumes exactly the pieces it copied.
    const bool defer = scratch != nullptr && (int64_t)2 * c.ld * (int64_t)sizeof(SV) <= scratchBytes;
    int4 *pendDst = nullptr;
    // (incremental update of stored gains: rows of at most three 16-byte pieces per thread, and room for the list of
    // raised columns behind the resident state)
    const bool deltaAllowed = kDelta && prm.incremental && defer && ld4 <= 3 * kSelectThreads &&
                              (int64_t)6 * c.ld * (int64_t)sizeof(SV) + (int64_t)kDeltaMax * 16 <= scratchBytes;
    // The threshold vector of a coming threshold pass is the element-wise minimum of the listed blocks'
    // coverage.  Those blocks are, as a rule, exactly the ones that receive a sample in this chain (every
    // other block's stored gains stay valid), and each receives one: so the minimum is taken as the
    // updated vectors pass through fold_pending, in the third ld-sized piece of the scratch area.  A block
    // of the chain that is not listed (it became full) only lowers the threshold, which keeps the pass exact.
    int4 *thrAcc = (defer && (int64_t)3 * c.ld * (int64_t)sizeof(SV) <= scratchBytes) ? scratch + 2 * ld4 : nullptr;
    if (thrAcc) {
        int4 top;
        if constexpr (Arith<SV>::kInt) top = make_int4(INT_MAX, INT_MAX, INT_MAX, INT_MAX);
        else top = make_int4(0x7f800000, 0x7f800000, 0x7f800000, 0x7f800000);      // +infinity
        for (int i = threadIdx.x; i < ld4; i += kSelectThreads) thrAcc[i] = top;
    }
    int chainLen = 0;
    __shared__ int shRaised[2];                            // integer path: raised columns of the pick in hand (slot: pick parity)
    // The next v* of a block, noted ahead of time.  When the stored gains of block p are corrected in place they all stand
    // in registers, so every warp notes its best unassigned candidate among them.  At p's next turn the best of those is
    // the argmax, unless it has been assigned meanwhile (the stored gains of p do not change in between): then no stored
    // gain is loaded and the pick needs neither of the argmax's two barriers.  Blocks 0..kCacheBlocks-1; the notes sit
    // behind the list of raised columns.
    constexpr int kCacheBlocks = 16;
    constexpr int kWarps = kSelectThreads / 32;
    __shared__ uint8_t shNoted[kCacheBlocks];
    unsigned long long *noteK = reinterpret_cast<unsigned long long *>(scratch + 6 * ld4 + kDeltaMax);   // [kCacheBlocks][kWarps] keys
    const bool notes = kDelta && deltaAllowed && prm.lazyFrom < 0 && c.M <= 8192 &&
                       (int64_t)6 * c.ld * (int64_t)sizeof(SV) + (int64_t)kDeltaMax * 16 +
                       (int64_t)kCacheBlocks * kWarps * (int64_t)sizeof(unsigned long long) <= scratchBytes;
    if (threadIdx.x < kCacheBlocks) shNoted[threadIdx.x] = 0;       // (a pass may have rewritten any block's stored gains)
    if (threadIdx.x == 0) shRaised[0] = shRaised[1] = 0;
    __syncthreads();
    __shared__ unsigned long long shStat[4];               // corrections of this chain: how many, rows of S, bytes; picks from a note (thread 0 only)
    if (threadIdx.x == 0) shStat[0] = shStat[1] = shStat[2] = shStat[3] = 0ull;
    __shared__ PlanGlobals shPre;
    if (threadIdx.x == 0) shPre = plan_globals(prm, l);     // (in flight under the first argmax; read after its barriers)

    for (;;) {
        const int par = chainLen & 1;
        if (threadIdx.x == 0) shRaised[par ^ 1] = 0;        // (the next pick's slot: read last before the previous pick's final barrier)
        const GV *G = prm.gains + c.vOff + (int64_t)j * c.ld;
        // v* = argmax over the unassigned samples, ties -> lowest class-local index.  Walks all
        // samples with independent, coalesced loads (pos[v] < 0 marks an assigned sample).
        GV bestG = 0;
        int bestV = INT_MAX;
        bool fast = false;                                  // v* comes from the notes: no argmax
        if constexpr (kDelta) {
            if (notes && j < kCacheBlocks && shNoted[j]) {
                const unsigned long long key = warp_max_u64(lane < kWarps ? noteK[j * kWarps + lane] : 0ull);
                if (key) { key_gain(key, bestG); bestV = key_index(key); }
                fast = bestV != INT_MAX && (res ? shPos[bestV] : pos[bestV]) >= 0;
                if (!fast) { bestG = 0; bestV = INT_MAX; }
            }
        }
        if (fast) {
            if (res && chainLen == 0 && threadIdx.x == 0) __threadfence();
            if (pendDst) {
                fold_pending<SV>(pendDst, scratch, ld4, thrAcc);
                pendDst = nullptr;
            }
        } else {
        // batches of kArgmaxBatch samples per thread: all loads of a batch are issued before the
        // first comparison, so a class of up to kArgmaxBatch * kSelectThreads samples costs one
        // memory round trip
        constexpr int kArgmaxBatch = 12;
        for (int v0 = threadIdx.x; v0 < c.M; v0 += kArgmaxBatch * kSelectThreads) {
            GV g[kArgmaxBatch];
            int ps[kArgmaxBatch];
#pragma unroll
            for (int i = 0; i < kArgmaxBatch; ++i) {
                const int v = v0 + i * kSelectThreads;
                ps[i] = -1;
                g[i] = 0;
                if (v < c.M) {
                    if (res) { g[i] = __ldcg(G + v); ps[i] = shPos[v]; }
                    else { g[i] = G[v]; ps[i] = pos[v]; }
                }
            }
#pragma unroll
            for (int i = 0; i < kArgmaxBatch; ++i) {
                const int v = v0 + i * kSelectThreads;
                if (ps[i] >= 0 && (bestV == INT_MAX || g[i] > bestG)) { bestG = g[i]; bestV = v; }
            }
        }
        // (thread 0 of a CTA that owns its class has just marked the class as taken: that store is ordered
        // before everything the chain writes; the fence completes together with the loads above)
        if (res && chainLen == 0 && threadIdx.x == 0) __threadfence();
        if (pendDst) {                                  // finish the previous pick's coverage update
            fold_pending<SV>(pendDst, scratch, ld4, thrAcc);
            pendDst = nullptr;
        }
        // (gain, index) as one key where the class is small enough and no floors are kept (row-skipping passes off): the
        // two reductions are then two warp-wide maxima each instead of shuffle ladders over pairs
        const bool packed = c.M <= 8192 && prm.lazyFrom < 0;
        if (packed) {
            const unsigned long long key = warp_max_u64(bestV != INT_MAX ? note_key(bestG, bestV) : 0ull);
            if (lane == 0) shKey[warp] = key;
        } else {
            for (int off = 16; off > 0; off >>= 1) {
                GV oG = __shfl_xor_sync(0xffffffffu, bestG, off);
                int oV = __shfl_xor_sync(0xffffffffu, bestV, off);
                if (oV != INT_MAX && (bestV == INT_MAX || oG > bestG || (oG == bestG && oV < bestV))) { bestG = oG; bestV = oV; }
            }
            if (lane == 0) { shG[warp] = bestG; shV[warp] = bestV; }
        }
        __syncthreads();
        if (warp == 0) {
            // The least of the warps' best stored gains: at least one unassigned sample per warp lies at or above it,
            // so a later row-skipping pass with this floor recomputes the few dozen best-placed candidates of the block.
            FV low = lowest_value<FV>();
            if (packed) {
                const unsigned long long key = warp_max_u64(lane < kSelectThreads / 32 ? shKey[lane] : 0ull);
                bestG = 0;
                bestV = INT_MAX;
                if (key) { key_gain(key, bestG); bestV = key_index(key); }
            } else {
                bestG = lane < kSelectThreads / 32 ? shG[lane] : (GV)0;
                bestV = lane < kSelectThreads / 32 ? shV[lane] : INT_MAX;
                low = bestV != INT_MAX ? (FV)bestG : highest_value<FV>();
                for (int off = 16; off > 0; off >>= 1) {
                    GV oG = __shfl_xor_sync(0xffffffffu, bestG, off);
                    int oV = __shfl_xor_sync(0xffffffffu, bestV, off);
                    const FV oLow = __shfl_xor_sync(0xffffffffu, low, off);
                    if (oLow < low) low = oLow;
                    if (oV != INT_MAX && (bestV == INT_MAX || oG > bestG || (oG == bestG && oV < bestV))) { bestG = oG; bestV = oV; }
                }
            }
            if (lane == 0) {
                shPick = bestV;
                if (bestV != INT_MAX && j < kLazyBlocks && (FV)bestG < shPlan.floorv[j]) {
                    // A miss: the best stored gain lies below the floor of the block's last pass, so it may be an
                    // upper bound only.  Nothing is picked; the block asks for a pass over every row.
                    shPick = kPickMiss;
                    shPlan.open[j] = (uint8_t)(shPlan.open[j] | 2);
                    shPlan.theta[j] = lowest_value<FV>();
                    shPlan.lazyMisses += 1;
                    atomicAdd(&prm.phaseNs[9], 1ull);
                    prm.valid[(int64_t)l * prm.W + j] = 0;
                } else if (bestV != INT_MAX) {
                    // block j has received a sample: value, room, and its stored gains are now out of date
                    shPlan.f[j] += (FV)bestG;
                    const int room = shPlan.room[j] - 1;
                    shPlan.room[j] = room;
                    shPlan.open[j] = (uint8_t)((room > 0 ? 1 : 0) | 2);
                    if (j < kLazyBlocks) shPlan.theta[j] = low;
                    prm.valid[(int64_t)l * prm.W + j] = 0;     // (plan_decide, same lane, may set it again)
                }
            }
            __syncwarp();
        }
        __syncthreads();
        }
        if (!fast && shPick == kPickMiss) {
            // (the chain ends here: its last act is to schedule the pass this block needs)
            if (warp == 0) plan_decide(prm, l, c, nR, round + 1, shPlan, &shPre);
            __syncthreads();
            j = shPlan.nextJ;
            break;
        }
        if (threadIdx.x == 0 && chainLen < kSparseMax) shChain[chainLen] = j;
        ++chainLen;
        const int vstar = fast ? bestV : shPick;
        // (fast: thread 0 books the pick in the plan after the next barrier, so the room still counts this sample)
        const int roomAfter = fast ? shPlan.room[j] - 1 : shPlan.room[j];
        auto book_fast = [&]() {                             // thread 0, fast picks: what warp 0 does after an argmax
            shStat[3] += 1ull;
            shPlan.f[j] += (FV)bestG;
            shPlan.room[j] = roomAfter;
            shPlan.open[j] = (uint8_t)((roomAfter > 0 ? 1 : 0) | 2);
            const int64_t at = (int64_t)l * prm.W + j;
            prm.valid[at] = 0;
            prm.fval[at] = shPlan.f[j];
            prm.cnt[at] = shPlan.quota[j] - roomAfter;
        };
        if (vstar == INT_MAX || vstar < 0 || vstar >= c.M) {
            if (threadIdx.x == 0) atomicOr(prm.status, kDevBadState);
            j = -1;
            break;
        }
        // warp 0: next block (shared memory only).  last warp: global bookkeeping of this pick.
        // everybody else meanwhile starts fetching row v* and the coverage vector.
        const int4 *row = reinterpret_cast<const int4 *>(prm.S + c.sOff + (int64_t)vstar * c.ld);
        int4 *cov = reinterpret_cast<int4 *>(prm.cover + c.vOff + (int64_t)j * c.ld);
        // (one thread: the sample leaves the candidate list.  After an argmax its barriers lie between this and every read
        // of the list; a fast pick has none, and a warp that runs ahead must not change what the others still test their
        // noted candidate against: there it waits for the pick's next barrier)
        auto book_sample = [&]() {
            if (res) {
                // everything this needs is in shared memory: stores only, nothing to wait for
                const int global = shPerm[vstar];
                prm.assignment[global] = j;
                if (prm.order) prm.order[c.row0 + (c.M - nR)] = global;
                const int k = shPos[vstar];
                const int lastV = shCand[nR - 1];
                shCand[k] = lastV;
                shPos[lastV] = k;
                shPos[vstar] = -1;
                cand[k] = lastV;                                // (the sweeps read the list from global memory)
            } else {
                const int global = prm.perm[c.row0 + vstar];
                prm.assignment[global] = j;
                if (prm.order) prm.order[c.row0 + (c.M - nR)] = global;
                const int k = pos[vstar];
                const int lastV = cand[nR - 1];
                cand[k] = lastV;
                pos[lastV] = k;
                pos[vstar] = -1;
            }
            prm.nR[l] = nR - 1;
            if (nR == 1) atomicSub(&prm.nSweep[3], 1);        // one class fewer to finish
        };
        if (threadIdx.x == kSelectThreads - 32 && !fast) {
            const int64_t at = (int64_t)l * prm.W + j;
            prm.fval[at] = shPlan.f[j];
            prm.cnt[at] = shPlan.quota[j] - shPlan.room[j];
            book_sample();
        }
        if (kDelta && deltaAllowed && nR > 1 && roomAfter > 0) {
            // Incremental update: fold row v* into the coverage vector now, find the columns it raised, and if they are
            // few correct the stored gains of block j by one row of S per column; the block then stays up to date.
            for (int i = threadIdx.x; i < ld4; i += kSelectThreads) {
                async_copy16(scratch + i, row + i);
                async_copy16(scratch + ld4 + i, cov + i);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            GV *Gj = prm.gains + c.vOff + (int64_t)j * c.ld;
            GV gj[3][4];                                        // this thread's columns of the block's stored gains
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const int i = (int)threadIdx.x + k * kSelectThreads;
#pragma unroll
                for (int q = 0; q < 4; ++q) gj[k][q] = 0;
                if (i < ld4) {
                    if constexpr (Arith<SV>::kInt) {
                        const longlong2 a = __ldcg(reinterpret_cast<const longlong2 *>(Gj + 4 * i));
                        const longlong2 b = __ldcg(reinterpret_cast<const longlong2 *>(Gj + 4 * i) + 1);
                        gj[k][0] = a.x; gj[k][1] = a.y; gj[k][2] = b.x; gj[k][3] = b.y;
                    } else {
                        const float4 a = __ldcg(reinterpret_cast<const float4 *>(Gj + 4 * i));
                        gj[k][0] = a.x; gj[k][1] = a.y; gj[k][2] = a.z; gj[k][3] = a.w;
                    }
                }
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            int cnt = 0;
            unsigned mask = 0;
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const int i = (int)threadIdx.x + k * kSelectThreads;
                if (i < ld4) {
                    const int4 r = scratch[i], o = scratch[ld4 + i];
                    const int4 m = max_int4<SV>(o, r);
                    if (thrAcc) thrAcc[i] = min_int4<SV>(thrAcc[i], m);
                    const unsigned b = (rose<SV>(r.x, o.x) ? 1u : 0u) | (rose<SV>(r.y, o.y) ? 2u : 0u) |
                                       (rose<SV>(r.z, o.z) ? 4u : 0u) | (rose<SV>(r.w, o.w) ? 8u : 0u);
                    if (b) cov[i] = m;                            // (elsewhere the vector keeps its value)
                    mask |= b << (4 * k);
                    cnt += __popc(b);
                }
            }
            int4 *list = scratch + 6 * ld4;                      // (column, old coverage, new coverage, -)
            int total;
            bool few;
            if constexpr (Arith<SV>::kInt) {
                // integer corrections are exact in any order: the threads that found raised columns append them
                int at = cnt ? atomicAdd(&shRaised[par], cnt) : 0;
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    const int i = (int)threadIdx.x + k * kSelectThreads;
                    const unsigned b = (mask >> (4 * k)) & 15u;
                    if (b) {
                        const int4 r = scratch[i], o = scratch[ld4 + i];
                        if ((b & 1u) && at < kDeltaMax) list[at++] = make_int4(4 * i + 0, o.x, r.x, 0);
                        if ((b & 2u) && at < kDeltaMax) list[at++] = make_int4(4 * i + 1, o.y, r.y, 0);
                        if ((b & 4u) && at < kDeltaMax) list[at++] = make_int4(4 * i + 2, o.z, r.z, 0);
                        if ((b & 8u) && at < kDeltaMax) list[at++] = make_int4(4 * i + 3, o.w, r.w, 0);
                    }
                }
                __syncthreads();
                total = shRaised[par];
                few = total <= prm.deltaMax;
            } else {
            // where this thread's columns go in the list: an exclusive prefix sum over the CTA, so that the list (and with it
            // the order of the floating-point corrections) does not depend on timing
            int incl = cnt;
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += t;
            }
            if (lane == 31) shV[warp] = incl;                    // (the argmax is over: its per-warp array is free)
            __syncthreads();
            int base = 0; total = 0;
#pragma unroll
            for (int w = 0; w < kSelectThreads / 32; ++w) {
                const int t = shV[w];
                if (w < warp) base += t;
                total += t;
            }
            few = total <= prm.deltaMax;
            if (few) {
                int at = base + incl - cnt;
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    const int i = (int)threadIdx.x + k * kSelectThreads;
                    const unsigned b = (mask >> (4 * k)) & 15u;
                    if (b) {
                        const int4 r = scratch[i], o = scratch[ld4 + i];
                        if (b & 1u) list[at++] = make_int4(4 * i + 0, o.x, r.x, 0);
                        if (b & 2u) list[at++] = make_int4(4 * i + 1, o.y, r.y, 0);
                        if (b & 4u) list[at++] = make_int4(4 * i + 2, o.z, r.z, 0);
                        if (b & 8u) list[at++] = make_int4(4 * i + 3, o.w, r.w, 0);
                    }
                }
            }
            __syncthreads();
            }
            if (fast && threadIdx.x == 0) book_fast();
            if (fast && threadIdx.x == kSelectThreads - 32) book_sample();
            unsigned changed = 0;                                // bit k: the correction moved one of this thread's gains of piece k
            if (few) {
                const SV *Sl = prm.S + c.sOff;
                if (ld4 <= kSelectThreads) {
                    // short rows (one 16-byte piece per thread): twelve rows of S in flight per thread
                    const int i = (int)threadIdx.x;
                    for (int e0 = 0; e0 < total; e0 += 12) {
                        int4 x[12];
#pragma unroll
                        for (int q = 0; q < 12; ++q) {
                            const int col = list[e0 + q < total ? e0 + q : e0].x;
                            const int4 *rp = reinterpret_cast<const int4 *>(Sl + (int64_t)col * c.ld);
                            x[q] = i < ld4 ? ld_stream_here(rp + i) : make_int4(0, 0, 0, 0);
                        }
#pragma unroll
                        for (int q = 0; q < 12; ++q) {
                            if (e0 + q < total) {
                                const int4 ent = list[e0 + q];              // (shared memory, the same word for every thread)
                                const auto d0 = delta_term<SV>(x[q].x, ent.y, ent.z), d1 = delta_term<SV>(x[q].y, ent.y, ent.z);
                                const auto d2 = delta_term<SV>(x[q].z, ent.y, ent.z), d3 = delta_term<SV>(x[q].w, ent.y, ent.z);
                                gj[0][0] -= d0; gj[0][1] -= d1; gj[0][2] -= d2; gj[0][3] -= d3;
                                changed |= (d0 != 0 || d1 != 0 || d2 != 0 || d3 != 0) ? 1u : 0u;
                            }
                        }
                    }
                } else {
                    for (int e0 = 0; e0 < total; e0 += 4) {
                        int4 x[4][3];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int col = list[e0 + q < total ? e0 + q : e0].x;
                            const int4 *rp = reinterpret_cast<const int4 *>(Sl + (int64_t)col * c.ld);
#pragma unroll
                            for (int k = 0; k < 3; ++k) {
                                const int i = (int)threadIdx.x + k * kSelectThreads;
                                x[q][k] = (i < ld4 && e0 + q < total) ? ld_stream_here(rp + i) : make_int4(0, 0, 0, 0);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (e0 + q < total) {
                                const int4 ent = list[e0 + q];
#pragma unroll
                                for (int k = 0; k < 3; ++k) {
                                    const auto d0 = delta_term<SV>(x[q][k].x, ent.y, ent.z), d1 = delta_term<SV>(x[q][k].y, ent.y, ent.z);
                                    const auto d2 = delta_term<SV>(x[q][k].z, ent.y, ent.z), d3 = delta_term<SV>(x[q][k].w, ent.y, ent.z);
                                    gj[k][0] -= d0; gj[k][1] -= d1; gj[k][2] -= d2; gj[k][3] -= d3;
                                    changed |= (d0 != 0 || d1 != 0 || d2 != 0 || d3 != 0) ? (1u << k) : 0u;
                                }
                            }
                        }
                    }
                }
                if (total > 0) {
#pragma unroll
                    for (int k = 0; k < 3; ++k) {
                        const int i = (int)threadIdx.x + k * kSelectThreads;
                        if (i < ld4 && ((changed >> k) & 1u)) {        // (most gains keep their value: nothing to store)
                            if constexpr (Arith<SV>::kInt) {
                                reinterpret_cast<longlong2 *>(Gj + 4 * i)[0] = make_longlong2(gj[k][0], gj[k][1]);
                                reinterpret_cast<longlong2 *>(Gj + 4 * i)[1] = make_longlong2(gj[k][2], gj[k][3]);
                            } else {
                                *reinterpret_cast<float4 *>(Gj + 4 * i) = make_float4(gj[k][0], gj[k][1], gj[k][2], gj[k][3]);
                            }
                        }
                    }
                }
                if (threadIdx.x == 0) {
                    // block j is up to date again
                    shPlan.open[j] = (uint8_t)1;
                    prm.valid[(int64_t)l * prm.W + j] = 1;
                    shStat[0] += 1ull;
                    shStat[1] += (unsigned long long)total;
                    shStat[2] += (unsigned long long)(total + 2) * (unsigned long long)c.ld * sizeof(SV) + 2ull * c.ld * sizeof(GV);
                }
            }
            if (notes && j < kCacheBlocks) {
                if (few) {
                    // the corrected gains stand in registers: this warp's best unassigned candidate among them
                    unsigned long long nk = 0ull;
#pragma unroll
                    for (int k = 0; k < 3; ++k) {
                        const int i = (int)threadIdx.x + k * kSelectThreads;
                        if (i < ld4) {
                            // (resident list: the four marks of this piece in one 16-byte read)
                            int4 mk = make_int4(0, 0, 0, 0);
                            if (res) mk = reinterpret_cast<const int4 *>(shPos)[i];
                            const int mark[4] = {mk.x, mk.y, mk.z, mk.w};
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int v = 4 * i + q;
                                // (v* may or may not have left the list yet: named explicitly)
                                if (v < c.M && v != vstar && (res ? mark[q] : pos[v]) >= 0) {
                                    const unsigned long long kk = note_key(gj[k][q], v);
                                    if (kk > nk) nk = kk;
                                }
                            }
                        }
                    }
                    nk = warp_max_u64(nk);
                    if (lane == 0) noteK[j * kWarps + warp] = nk;
                }
                if (threadIdx.x == 0) shNoted[j] = few ? 1 : 0;
            }
            // (a compiler barrier: without it the correction above and the choice of the next block below are scheduled
            // into one another, and a pick takes 3 us longer -- C2 66 ms instead of 47 ms, measured)
            asm volatile("" ::: "memory");
            if (warp == 0) {
                __syncwarp();
                plan_decide(prm, l, c, nR - 1, round + 1, shPlan, &shPre);
            }
        } else {
            if (fast) {
                __syncthreads();                            // (everybody has read the room of block j)
                if (threadIdx.x == 0) book_fast();
                if (threadIdx.x == kSelectThreads - 32) book_sample();
            }
            if (threadIdx.x == 0 && notes && j < kCacheBlocks) shNoted[j] = 0;     // (the block's stored gains are out of date)
            if (warp == 0) {
                __syncwarp();
                plan_decide(prm, l, c, nR - 1, round + 1, shPlan, &shPre);
            }
            // cover_j <- max(cover_j, S[v*][.])
            if (defer) {
                for (int i = threadIdx.x; i < ld4; i += kSelectThreads) {
                    async_copy16(scratch + i, row + i);
                    async_copy16(scratch + ld4 + i, cov + i);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                pendDst = cov;
            } else {
#pragma unroll 2
                for (int i = threadIdx.x; i < ld4; i += kSelectThreads) cov[i] = max_int4<SV>(cov[i], row[i]);
            }
        }
        __syncthreads();
        nR -= 1;
        j = shPlan.nextJ;
        if (nR == 0 || j < 0 || shPlan.needSweep) break;
    }
    if (threadIdx.x == 0 && shStat[0]) {
        if (shStat[3]) atomicAdd(&prm.phaseNs[17], shStat[3]);
        atomicAdd(&prm.phaseNs[15], shStat[0]);
        atomicAdd(&prm.phaseNs[16], shStat[1]);
        atomicAdd(&prm.phaseNs[12], shStat[2]);
    }
    if (keep && threadIdx.x == 0) { keep[0] = nR; keep[1] = j; }     // (j = -1 after an inconsistency: the class is given up)
    if (!res) plan_store_lazy(prm, l, shPlan);                       // (a CTA that owns its class keeps this state in shared memory)
    if (pendDst) fold_pending<SV>(pendDst, scratch, ld4, thrAcc);
    if (shPlan.needSweep && shPlan.sweepSparse) {
        // threshold of the coming pass: element-wise minimum of the listed blocks' coverage vectors
        const int P = shPlan.sweepBlocks;
        const int32_t *parts = prm.sweepParts + (int64_t)l * kSparseMax;
        const int4 *cov = reinterpret_cast<const int4 *>(prm.cover + c.vOff);
        int4 *thr = reinterpret_cast<int4 *>(prm.thr + c.vOff / prm.W);
        // is every listed block one of this chain's?  (then the running minimum is the threshold)
        if (threadIdx.x == 0) shChainOk = (thrAcc != nullptr && chainLen <= kSparseMax) ? 1 : 0;
        __syncthreads();
        if (shChainOk && threadIdx.x < P) {
            const int p = parts[threadIdx.x];
            bool found = false;
            for (int k = 0; k < chainLen; ++k) found = found || shChain[k] == p;
            if (!found) shChainOk = 0;
        }
        __syncthreads();
        if (shChainOk) {
            for (int i = threadIdx.x; i < ld4; i += kSelectThreads) thr[i] = thrAcc[i];
        } else {
            // (each thread reads back exactly the pieces of the coverage vectors it wrote itself)
            for (int i = threadIdx.x; i < ld4; i += kSelectThreads) {
                int4 m = cov[(int64_t)parts[0] * ld4 + i];
                for (int k0 = 1; k0 < P; k0 += 8) {                     // eight independent loads at a time
                    int4 t[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) t[u] = cov[(int64_t)parts[k0 + u < P ? k0 + u : 0] * ld4 + i];
#pragma unroll
                    for (int u = 0; u < 8; ++u) m = min_int4<SV>(m, t[u]);
                }
                thr[i] = m;
            }
        }
    }
}

// Picks of round `round`: every class advances until it needs a sweep (or is finished).
template <typename SV>
__global__ void __launch_bounds__(kSelectThreads, 2) chain_kernel(GreedyParams<SV> prm, int round)
{
    cudaGridDependencySynchronize();              // the sweep of this round has finished
    cudaTriggerProgrammaticLaunchCompletion();
    pick_chain(prm, blockIdx.x, round, nullptr, 0);
}

// ---------------------------------------------------------------------------------------------
// The whole greedy loop in one cooperative launch.  A round = one sweep phase (every class that
// asked for a sweep, all CTAs) and one pick phase (class l by CTA l mod gridDim.x: picks until the
// class needs its next sweep), separated by grid barriers.  Control flow is uniform across the
// grid: the number of unfinished classes is read after a barrier and not touched before the next.
// Barrier over all CTAs of a cooperative launch (all co-resident): one arrival counter that only
// grows, so round k waits for k * gridDim.x arrivals.  The wait is bounded; when it runs out (or
// another CTA has already reported that) the timeout bit is set in the status word and the caller
// leaves its loop.  Thread 0's fences order this CTA's writes before its arrival and make the other
// CTAs' writes visible after the wait (the fence drops stale L1 lines of this SM).
constexpr unsigned kBarrierSpinLimit = 1u << 21;       // polls of about a microsecond each: a second or two
__device__ __forceinline__ bool grid_barrier(unsigned *counter, unsigned expected, int32_t *status,
                                             unsigned spinLimit = kBarrierSpinLimit)
{
    __shared__ int shOk;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        int ok = 1;
        unsigned spins = 0;
        while (*(volatile unsigned *)counter < expected) {
            if ((++spins & 1023u) == 0 && ((*(volatile int32_t *)status & kDevTimeout) || spins >= spinLimit)) {
                atomicOr(status, kDevTimeout);
                ok = 0;
                break;
            }
        }
        __threadfence();
        shOk = ok;
    }
    __syncthreads();
    return shOk != 0;
}

__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// (The loop keeps next to nothing in registers across the two phases -- the phase clocks of CTA 0
// sit in shared memory, the barrier's target is recomputed from the round number -- so that the
// sweep's inner loop gets the whole register budget.)
template <typename SV>
__global__ void __launch_bounds__(kSweepThreads, 1) greedy_persistent_kernel(const __grid_constant__ GreedyParams<SV> prm, int maxRounds)
{
    extern __shared__ __align__(128) int4 shCover[];
    __shared__ unsigned long long shClock[3];      // last stamp, sweep-phase ns, pick-phase ns (CTA 0, thread 0)
    if (blockIdx.x == 0 && threadIdx.x == 0) { shClock[0] = global_ns(); shClock[1] = 0; shClock[2] = 0; }
    for (int r = 0; r < maxRounds; ++r) {
        if (*(volatile int32_t *)&prm.nSweep[3] == 0) break;     // every class is finished
        sweep_step(prm, r, shCover);
        if (!grid_barrier(prm.barrier, (unsigned)(2 * r + 1) * gridDim.x, prm.status)) break;   // gains of round r are in place
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            const unsigned long long t1 = global_ns();
            shClock[1] += t1 - shClock[0];
            shClock[0] = t1;
        }
        for (int l = blockIdx.x; l < prm.L; l += gridDim.x) {
            pick_chain(prm, l, r, shCover, prm.smemBytes);       // the sweep's shared memory is idle in this phase
            __syncthreads();
        }
        if (!grid_barrier(prm.barrier, (unsigned)(2 * r + 2) * gridDim.x, prm.status)) break;   // picks of round r, sweep list of round r+1
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            const unsigned long long t1 = global_ns();
            shClock[2] += t1 - shClock[0];
            shClock[0] = t1;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) { prm.phaseNs[0] = shClock[1]; prm.phaseNs[1] = shClock[2]; }
}

// ---------------------------------------------------------------------------------------------
// The greedy loop without grid-wide phases.  In the kernel above every SM but one per class idles
// while the classes make their picks.  Classes are independent, so here each class cycles on its own
// between "being swept" and "making picks", and the picks of one class overlap the sweeps of the
// others: CTAs [0, nPick) own the classes (class l belongs to CTA l mod nPick) and only make picks,
// the other CTAs only sweep.  The hand-off is the class's ClassSync word:
//   pick CTA   waits until epoch is even and done == nGroups (every row group of the published sweep
//              has written its gains), makes epoch odd, runs the chain of picks (which also fixes
//              the parameters of the class's next sweep), clears done, and makes epoch even again;
//   sweep CTA  looks for a published sweep that still has tickets (the class nearest to the CTA's home
//              position, CTAs being spread evenly over the classes; `asyncGroup` < L serves the sweeps
//              in batches by publication order instead), reads its parameters between two reads of
//              epoch (both must give the same even value: the parameters belong to that sweep), draws
//              one ticket per team from the sweep's own ticket counter, and only then stages the
//              coverage vectors and sweeps.
// Every (class, sweep number) has a ticket counter of its own that starts at zero and is never
// reset, so a CTA that was slow to act on what it read can only draw a ticket beyond the last row
// group and leaves; a valid ticket is only ever drawn while the class waits for its sweep.  While a
// class makes its picks, the CTAs at home there help the neighbouring classes.
// All waits are bounded: a CTA that finds nothing to do for about a second sets the timeout bit, and
// every loop leaves as soon as the status word is non-zero.
constexpr unsigned kIdleLimit = 1u << 20;

__device__ __forceinline__ int4 ld_volatile16(const void *p)
{
    int4 v;
    asm volatile("ld.volatile.global.v4.s32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int32_t ld_volatile32(const int32_t *p) { return *(const volatile int32_t *)p; }
// The second read of a class's epoch (the first one and everything read in between count only if it returns the same
// even value): an acquire load at GPU scope.
__device__ __forceinline__ int32_t ld_acquire32(const int32_t *p)
{
    int32_t v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}


template <typename SV>
__device__ __forceinline__ void async_pick_cta(const GreedyParams<SV> &prm, int4 *scratch)
{
    __shared__ int shEpoch, shFinished;
    const int me = blockIdx.x;
    int mine = 0;                                                   // my classes that are not finished
    for (int l = me; l < prm.L; l += prm.nPick) mine += prm.desc[l].M > 0 ? 1 : 0;
    unsigned idle = 0;
    unsigned long long busy = 0;
    __shared__ int shKeep[2];
    const bool owner = prm.nPick >= prm.L;                          // this CTA serves one class only
    bool kept = false;
    while (mine > 0) {
        bool progressed = false;
        for (int l = me; l < prm.L; l += prm.nPick) {
            if (threadIdx.x == 0) {
                const int4 sy = ld_volatile16(&prm.sync[l]);           // epoch, nGroups, done, seq
                int e = -1;
                if (!(sy.x & 1) && sy.z == sy.y) {
                    e = sy.x;
                    *(volatile int32_t *)&prm.sync[l].epoch = e + 1;    // the class is mine until I publish again
                    if (!owner) __threadfence();                        // (an owner's chain fences after its first loads)
                } else if (!(sy.x & 1) && sy.z > sy.y) {
                    // more row groups reported done than the sweep has: a sweep CTA acted on a torn or stale word
                    atomicOr(prm.status, kDevBadState);
                }
                shEpoch = e;
            }
            __syncthreads();
            const int e = shEpoch;
            if (e < 0) { __syncthreads(); continue; }
            progressed = true;
            unsigned long long t0 = 0;
            if (me == 0 && threadIdx.x == 0) t0 = global_ns();
            pick_chain<SV, true>(prm, l, e >> 1, scratch, prm.smemBytes, owner ? (kept ? 2 : 1) : 0, shKeep);
            kept = true;
            __syncthreads();                                            // all writes of the chain are issued
            if (threadIdx.x == 0) {
                const bool finished = shKeep[0] == 0 || shKeep[1] < 0;
                if (!finished) {
                    prm.sync[l].done = 0;
                    prm.sync[l].seq = ((e >> 1) + 1) * prm.L + l;        // sweep number first: batches follow the classes' progress
                    __threadfence();                                    // parameters, coverage, candidate list before the epoch
                    *(volatile int32_t *)&prm.sync[l].epoch = e + 2;
                }
                shFinished = finished ? 1 : 0;
                if (me == 0) busy += global_ns() - t0;
            }
            __syncthreads();
            if (shFinished) --mine;
        }
        if (progressed) {
            idle = 0;
        } else {
            __nanosleep(200);
            ++idle;
            if ((idle & 255u) == 0) {                                   // uniform: every thread counts alike
                if (threadIdx.x == 0) {
                    int stop = ld_volatile32(prm.status) != 0;
                    if (!stop && idle >= kIdleLimit) { atomicOr(prm.status, kDevTimeout); stop = 1; }
                    shFinished = stop;
                }
                __syncthreads();
                const int stop = shFinished;
                __syncthreads();
                if (stop) break;
            }
        }
    }
    if (me == 0 && threadIdx.x == 0) prm.phaseNs[1] = busy;
}

template <typename SV>
__device__ __forceinline__ void async_sweep_cta(const GreedyParams<SV> &prm, int4 *shCover)
{
    using GV = typename Arith<SV>::GV;
    __shared__ long long shF[kMaxSweepBatch];
    __shared__ int32_t shParts[kSparseMax];
    __shared__ GV shTheta[kLazyBlocks];
    __shared__ int shTicket[kSweepThreads / 32];
    __shared__ GV shPart[kSweepThreads];
    __shared__ unsigned long long shBest;
    __shared__ int shInfo[12];                                      // ok, first ticket, nR, P, CS, mode, nGroups, stop, sweep number, epoch
    const bool clocked = blockIdx.x == prm.nPick;                   // the first sweep CTA keeps the busy clock
    const int home = (int)(((int64_t)(blockIdx.x - prm.nPick) * prm.L) / (gridDim.x - prm.nPick));
    const int helpMin = ((int)(gridDim.x - prm.nPick) >= prm.L) ? prm.helpMin : 1;
    unsigned idle = 0;
    __shared__ unsigned long long shClk[5];                         // busy ns, lull ns, visits, start of the lull, start of the visit (first sweep CTA, thread 0)
    if (threadIdx.x == 0) { shClk[0] = 0; shClk[1] = 0; shClk[2] = 0; shClk[3] = 0; shClk[4] = 0; }
    for (;;) {
        // The sweep to serve: sweeps are served by order number (sweep number first), asyncGroup of them
        // together; inside such a batch a CTA goes to the class nearest to its home position (CTAs spread
        // evenly over the classes), so that a CTA visits few classes per batch.  By default a batch is
        // every class.
        if (threadIdx.x == 0) shBest = ~0ull;
        __syncthreads();
        unsigned long long myKey = ~0ull;
        int4 myA = make_int4(0, 0, 0, 0), myB = make_int4(0, 0, 0, 0);
        for (int l = threadIdx.x; l < prm.L; l += blockDim.x) {
            const int4 a = ld_volatile16(&prm.sync[l]);             // epoch, nGroups, done, seq
            const int4 b = ld_volatile16(&prm.sync[l].pad_[0]);     // -, -, nR, cfg
            const int drawn = (a.x & 1) ? 0 : ld_volatile32(prm.tickets + prm.desc[l].row0 + l + (a.x >> 1));
            if (!(a.x & 1) && drawn < a.y) {
                int dist = l - home;
                if (dist < 0) dist += prm.L;
                // away from home only for a worthwhile number of row groups: the last few of a sweep are mostly
                // gone by the time a helper has drawn its tickets (every class has CTAs at home when helpMin > 1)
                if (dist != 0 && a.y - drawn < helpMin) continue;
                const unsigned long long key = ((unsigned long long)(unsigned)(a.w / prm.asyncGroup) << 40) |
                                               ((unsigned long long)(unsigned)dist << 20) | (unsigned)l;
                if (key < myKey) { myKey = key; myA = a; myB = b; }
            }
        }
        if (myKey != ~0ull) atomicMin(&shBest, myKey);
        __syncthreads();
        const unsigned long long best = shBest;
        if (best == ~0ull) {
            if (threadIdx.x == 0) {
                int stop = (ld_volatile32(&prm.nSweep[3]) == 0 || ld_volatile32(prm.status) != 0) ? 1 : 0;
                if (!stop && ++idle >= kIdleLimit) { atomicOr(prm.status, kDevTimeout); stop = 1; }
                shInfo[7] = stop;
                if (clocked && shClk[3] == 0) shClk[3] = global_ns();
            }
            __syncthreads();
            const int stop = shInfo[7];
            __syncthreads();
            if (stop) break;
            __nanosleep(200);
            continue;
        }
        if (clocked && threadIdx.x == 0 && shClk[3] != 0) {
            shClk[1] += global_ns() - shClk[3];
            shClk[3] = 0;
        }
        const int l = (int)(unsigned)(best & 0xfffffull);
        const ClassDesc c = prm.desc[l];
        const int ld4 = c.ld >> 2;
        const int32_t *parts = prm.sweepParts + (int64_t)l * kSparseMax;
        // Parameters of the sweep, read between two reads of the epoch: the first is the scan's, the second
        // comes after the parameters.  Every load here is volatile (served by L2), and the bulk data of a
        // sweep (coverage, threshold, candidate list) is read with ld.cg, so no stale L1 line can be seen;
        // the barriers keep the groups of loads in order.
        if (myKey == best) {
            shInfo[9] = myA.x;                                      // epoch
            shInfo[6] = myA.y;                                      // row groups
            shInfo[2] = myB.z;                                      // unassigned samples
            shInfo[3] = myB.w & 0xff;                               // blocks
            shInfo[4] = (myB.w >> 8) & 0xff;                        // warps per row group
            shInfo[5] = (myB.w >> 16) & 3;                          // 1 = threshold pass, 2 = one that skips rows
        }
        if (threadIdx.x < kSparseMax) {
            int bp = ld_volatile32(parts + threadIdx.x);
            if (bp < 0 || bp >= prm.W) bp = 0;                      // (beyond the list, or a read that raced with an update)
            shParts[threadIdx.x] = bp;
        } else if (threadIdx.x >= 256 && threadIdx.x < 256 + kLazyBlocks) {
            shTheta[threadIdx.x - 256] = *(const volatile GV *)&prm.sweepTheta[(int64_t)l * kLazyBlocks + (threadIdx.x - 256)];
        }
        if constexpr (Arith<SV>::kInt) {
            if (threadIdx.x >= 128 && threadIdx.x < 128 + kMaxSweepBatch)
                shF[threadIdx.x - 128] = *(const volatile long long *)&prm.sweepF[(int64_t)l * kMaxSweepBatch + (threadIdx.x - 128)];
        }
        __syncthreads();
        // Second read of the epoch, and with it -- before its answer is known -- one ticket per team is
        // drawn and the threshold / coverage vectors are staged.  Should the epoch turn out to have moved,
        // the class had been taken back by its pick CTA, which happens only after every row group of the
        // sweep is done: the tickets drawn were beyond the last row group, and what was staged is dropped.
        const int mode = shInfo[5];
        int P = shInfo[3], CS = shInfo[4];
        if (CS != 1 && CS != 2 && CS != 4 && CS != 8 && CS != 16) CS = 1;
        if (threadIdx.x == 0) {
            const int e1 = shInfo[9];
            const int teams = (kSweepThreads / 32) / (mode ? 1 : CS);
            const int first = atomicAdd(prm.tickets + c.row0 + l + (e1 >> 1), teams);
            const int e2 = ld_acquire32(&prm.sync[l].epoch);
            shInfo[0] = (e1 == e2 && !(e1 & 1) && first < shInfo[6]) ? 1 : 0;
            if (clocked) shClk[2] += 1ull << 32;                   // attempts (high half), visits (low half)
            shInfo[1] = first;
            shInfo[8] = e1 >> 1;
        }
        if (mode) {
            const int4 *thr = reinterpret_cast<const int4 *>(prm.thr + c.vOff / prm.W);
            if ((int64_t)thr_bytes_aligned(c.ld * (int)sizeof(SV)) + kSparseQueueBytes <= prm.smemBytes)
                for (int i = threadIdx.x; i < ld4; i += blockDim.x) shCover[i] = __ldcg(thr + i);
        } else {
            if (P != 1 && P != 2 && P != 4 && P != 8) P = 1;
            const int4 *cov = reinterpret_cast<const int4 *>(prm.cover + c.vOff);
            if ((int64_t)P * c.ld * (int64_t)sizeof(SV) <= prm.smemBytes) {
                for (int i = threadIdx.x; i < P * ld4; i += blockDim.x) {
                    int p = i / ld4, cc = i - p * ld4;
                    shCover[i] = __ldcg(cov + (int64_t)shParts[p] * ld4 + cc);
                }
            }
        }
        __syncthreads();
        if (!shInfo[0]) continue;                                   // another look at the sweeps
        idle = 0;
        if (clocked && threadIdx.x == 0) {
            shClk[4] = global_ns();
            shClk[2] += 1;
        }
        const int nR = shInfo[2], first = shInfo[1];
        int32_t *ticket = prm.tickets + c.row0 + l + shInfo[8];      // the counter of this sweep alone
        int32_t *done = &prm.sync[l].done;
        if (mode) {
            P = shInfo[3];
            if (P < 1 || P > kSparseMax) P = 1;
            uint2 *queue = reinterpret_cast<uint2 *>(reinterpret_cast<char *>(shCover) + thr_bytes_aligned(c.ld * (int)sizeof(SV)) + (threadIdx.x >> 5) * kSparseWarpBytes);
            if (mode == 2) {
                if (P <= 32) sweep_class_lazy<SV, 1>(prm, l, c, nR, P, shCover, shParts, shTheta, queue, ticket, done, first);
                else sweep_class_lazy<SV, 2>(prm, l, c, nR, P, shCover, shParts, shTheta, queue, ticket, done, first);
            } else if (P <= 32) sweep_class_sparse<SV, 1>(prm, l, c, nR, P, shCover, shParts, queue, ticket, done, first);
            else sweep_class_sparse<SV, 2>(prm, l, c, nR, P, shCover, shParts, queue, ticket, done, first);
        } else {
            switch (P) {
            case 1: sweep_class<SV, 1, 8>(prm, l, c, nR, CS, shCover, shF, shParts, shTicket, shPart, ticket, done, first); break;
            case 2: sweep_class<SV, 2, 8>(prm, l, c, nR, CS, shCover, shF, shParts, shTicket, shPart, ticket, done, first); break;
            case 4: sweep_class<SV, 4, 8>(prm, l, c, nR, CS, shCover, shF, shParts, shTicket, shPart, ticket, done, first); break;
            default: sweep_class<SV, 8, 4>(prm, l, c, nR, CS, shCover, shF, shParts, shTicket, shPart, ticket, done, first); break;
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            if (clocked) shClk[0] += global_ns() - shClk[4];
        }
    }
    if (clocked && threadIdx.x == 0) { prm.phaseNs[0] = shClk[0]; prm.phaseNs[6] = shClk[1]; prm.phaseNs[7] = shClk[2]; }
}

template <typename SV>
__global__ void __launch_bounds__(kSweepThreads, 1) greedy_async_kernel(const __grid_constant__ GreedyParams<SV> prm)
{
    extern __shared__ __align__(128) int4 shCover[];
    if ((int)blockIdx.x < prm.nPick) async_pick_cta(prm, shCover);
    else async_sweep_cta(prm, shCover);
}

// ---------------------------------------------------------------------------------------------
// The greedy loop with one CTA per class at a time (many classes: more classes than SMs, or classes too small
// to be worth sharing).  Classes are independent in Algorithm 1, so a CTA draws a class from a counter and runs
// it from its first pick to its last -- sweep with all its warps, then picks until the next sweep is due -- and
// draws the next.  Nothing is shared between CTAs but that counter: no grid barrier, no hand-off, and while one
// SM makes picks (latency-bound) the others stream, so the memory system stays busy without any phase structure.
// Classes are drawn largest first (classOrder), which keeps the last CTAs from finishing long after the rest.
template <typename SV>
__global__ void __launch_bounds__(kSweepThreads, 1) greedy_owner_kernel(const __grid_constant__ GreedyParams<SV> prm)
{
    extern __shared__ __align__(128) int4 shCover[];
    __shared__ SweepShared<SV> shSweep;
    __shared__ int shClass;
    __shared__ int shKeep[2];
    unsigned long long tSweep = 0, tPick = 0, tThreshold = 0;
    for (;;) {
        __syncthreads();
        if (threadIdx.x == 0) {
            const int k = atomicAdd(&prm.nSweep[0], 1);
            shClass = k < prm.L ? prm.classOrder[k] : -1;
        }
        __syncthreads();
        const int l = shClass;
        if (l < 0) break;
        if (prm.desc[l].M == 0) continue;
        for (int round = 0; round <= prm.desc[l].M; ++round) {
            if (*(volatile int32_t *)prm.status != 0) break;
            unsigned long long t0 = 0;
            if (blockIdx.x == 0 && threadIdx.x == 0) t0 = global_ns();
            const bool thresholdPass = prm.sweepN[l] > 0 && prm.sweepMode[l] != 0;
            if (prm.sweepN[l] > 0) sweep_serve_class(prm, l, shCover, shSweep);
            __syncthreads();
            if (blockIdx.x == 0 && threadIdx.x == 0) {
                const unsigned long long t1 = global_ns();
                tSweep += t1 - t0;
                if (thresholdPass) tThreshold += t1 - t0;
                t0 = t1;
            }
            pick_chain<SV, true>(prm, l, round, shCover, prm.smemBytes, 0, shKeep);
            __syncthreads();
            if (blockIdx.x == 0 && threadIdx.x == 0) tPick += global_ns() - t0;
            if (shKeep[0] == 0 || shKeep[1] < 0) break;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) { prm.phaseNs[0] = tSweep; prm.phaseNs[1] = tPick; prm.phaseNs[13] = tThreshold; }
}

// ---------------------------------------------------------------------------------------------
// Launch with programmatic stream serialization: the next kernel's CTAs may be placed while this
// one drains; every kernel starts with cudaGridDependencySynchronize(), so data dependencies hold.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <typename SV>
static rcd_status run_greedy(rcd_ctx *ctx, const Sizes &sz, const Workspace &ws,
                             const std::vector<ClassDesc> &descHost, int32_t *assignment, int32_t *order,
                             cudaStream_t st)
{
    using GV = typename Arith<SV>::GV;
    using FV = typename Arith<SV>::FV;
    GreedyParams<SV> prm;
    prm.desc = ws.desc;
    prm.S = (const SV *)ws.S;
    prm.cover = (SV *)ws.cover;
    prm.gains = (GV *)ws.gains;
    prm.fval = (FV *)ws.fval;
    prm.cnt = ws.cnt;
    prm.quota = ws.quota;
    prm.valid = ws.valid;
    prm.cand = ws.cand;
    prm.pos = ws.pos;
    prm.nR = ws.nR;
    prm.jstar = ws.jstar;
    prm.sweepN = ws.sweepN;
    prm.sweepParts = ws.sweepParts;
    prm.sweepMode = ws.sweepMode;
    prm.thr = (SV *)ws.thr;
    prm.hitCount = ws.hitCount;
    prm.sparseElems = ws.sparseElems;
    prm.sparseFrom = ws.sparseFrom;
    prm.sweepCS = ws.sweepCS;
    prm.rowCtr = ws.rowCtr;
    prm.sweepList = ws.sweepList;
    prm.nSweep = ws.nSweep;
    prm.stepBytes = ws.stepBytes;
    prm.stepOps = ws.stepOps;
    prm.phaseNs = ws.phaseNs;
    prm.barrier = (unsigned *)(ws.phaseNs + 2);
    prm.status = ws.status;
    prm.perm = ws.perm;
    prm.assignment = assignment;
    prm.order = order;
    prm.L = sz.L;
    prm.W = sz.W;
    int batch = ctx->cfg.sweep_batch_max;
    if (batch <= 0) batch = kMaxSweepBatch;
    prm.batchMax = batch;
    prm.sweepWarps = ctx->smCount * (kSweepThreads / 32);
    prm.one = 1u;
    prm.sparseMinMembers = ctx->cfg.sweep_mode == 1 ? -1 : (ctx->cfg.threshold_from > 0 ? ctx->cfg.threshold_from : 8);
    prm.hitShift = ctx->cfg.threshold_hit_shift > 0 ? ctx->cfg.threshold_hit_shift : 5;
    prm.floorv = (FV *)ws.floorv;
    prm.theta = (FV *)ws.theta;
    prm.sweepTheta = (GV *)ws.sweepTheta;
    prm.lazyStat = ws.lazyStat;
    prm.lazyFrom = (ctx->cfg.lazy_mode != 1 || ctx->cfg.sweep_mode == 1) ? -1 : (ctx->cfg.lazy_from > 0 ? ctx->cfg.lazy_from : 8);
    prm.incremental = ctx->cfg.incremental == 1 ? 1 : 0;             // (0 = choose: decided below, once the form of the loop is known)
    prm.deltaMax = ctx->cfg.incremental_max > 0 ? std::min<int>(ctx->cfg.incremental_max, kDeltaMax) : kDeltaMax;
    prm.sync = ws.sync;
    prm.tickets = ws.tickets;
    prm.sweepF = ws.sweepF;
    prm.asyncMode = 0;
    prm.nPick = 0;
    prm.asyncGroup = 1;
    prm.helpMin = 1;
    {
        std::vector<int32_t> sorted;
        sorted.reserve(descHost.size());
        for (const auto &c : descHost) sorted.push_back(c.M);
        std::sort(sorted.begin(), sorted.end());
        prm.sizesSorted = ws.sizesSorted;
        prm.classOrder = ws.classOrder;
        {
            std::vector<int32_t> order(descHost.size());
            for (size_t i = 0; i < order.size(); ++i) order[i] = (int32_t)i;
            std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return descHost[(size_t)a].M > descHost[(size_t)b].M; });
            RCD_CUDA(ctx, cudaMemcpyAsync(ws.classOrder, order.data(), order.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        }
        prm.nonEmpty = 0;
        prm.minM = 0;
        for (int32_t m : sorted) {
            if (m <= 0) continue;
            if (prm.nonEmpty == 0) prm.minM = m;
            ++prm.nonEmpty;
        }
        RCD_CUDA(ctx, cudaMemcpyAsync(ws.sizesSorted, sorted.data(), sorted.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    }
    int maxLd = 0;
    for (const auto &c : descHost) if (c.ld > maxLd) maxLd = c.ld;
    const int64_t smemCap = (int64_t)ctx->maxSmemOptin - 24 * 1024;  // static shared of the kernels + margin
    int64_t smem = (int64_t)batch * maxLd * (int64_t)sizeof(SV);
    if (prm.sparseMinMembers >= 0)                                   // threshold pass: one vector + the warps' rings and queues
        smem = std::max<int64_t>(smem, (int64_t)thr_bytes_aligned(maxLd * (int)sizeof(SV)) + kSparseQueueBytes);
    // room for the rings of the 8-block dense pass behind its coverage vectors, where both fit
    prm.denseRing = 0;
    if (batch == 8 && ctx->cfg.dense_ring != 2) {
        const int64_t withRing = (int64_t)thr_bytes_aligned(8 * maxLd * (int)sizeof(SV)) + dense_ring_bytes(4);
        if (withRing <= smemCap) { smem = std::max<int64_t>(smem, withRing); prm.denseRing = 1; }
    }
    if (smem > smemCap) smem = smemCap;
    if ((int64_t)maxLd * (int64_t)sizeof(SV) > smem)
        return fail(ctx, RCD_ERR_UNSUPPORTED,
                    "class of %d samples: one coverage vector (%lld bytes) exceeds the %lld bytes of shared memory",
                    maxLd, (long long)maxLd * (long long)sizeof(SV), (long long)smem);
    if (smem < 16) smem = 16;
    prm.smemBytes = (int32_t)smem;
    // 32-bit partial sums take terms below 16384*d each, four per chunk iteration
    {
        int64_t bound = 16384LL * sz.d;
        int64_t it = 0xffffffffLL / (4 * bound);
        if (it < 1) return fail(ctx, RCD_ERR_UNSUPPORTED, "feature width %lld too large for 32-bit partial sums", (long long)sz.d);
        if (it > 1 << 20) it = 1 << 20;
        prm.segIters = (int32_t)it;
    }
    RCD_CUDA(ctx, cudaFuncSetAttribute(sweep_kernel<SV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));

    // Which form of the loop: greedy_path 1 = two launches per round, 2 = one launch, rounds with grid
    // barriers, 3 = one launch, asynchronous classes, 0 = choose.  With few classes the pick phases of
    // the round-based kernel leave most SMs idle, and giving every class a pick CTA of its own costs
    // few SMs: the asynchronous kernel is chosen when there are at most a quarter as many classes as SMs.
    const bool perSweep = ctx->cfg.profile >= 2;
    int path = ctx->cfg.greedy_path;
    if (perSweep || !ctx->cooperative) path = 1;
    if (path == 0) path = (sz.L * 4 <= ctx->smCount) ? 3 : 4;
    if (path == 3 && ctx->smCount < 2) path = 2;
    if (path == 4) {
        RCD_CUDA(ctx, cudaFuncSetAttribute(greedy_owner_kernel<SV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        // (in-place correction of stored gains: a class's passes are made by one SM here, so their cost grows with the
        // square of the class size while a correction reads a few dozen rows; measured: it wins on 1300-sample classes
        // with 64 blocks (208 -> 183 ms) and loses on 500-sample classes with 32 (3.9 -> 5.0 ms))
        if (ctx->cfg.incremental == 0) prm.incremental = sz.maxM >= 1024 ? 1 : 0;
        if (ctx->cfg.incremental_max <= 0) prm.deltaMax = 64;
        prm.asyncMode = 2;
        prm.sweepWarps = kSweepThreads / 32;                     // a class is swept by the warps of its own CTA
    }
    if (path == 2 || path == 3) {
        // one cooperative launch needs one CTA per SM resident at once
        RCD_CUDA(ctx, cudaFuncSetAttribute(greedy_persistent_kernel<SV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        RCD_CUDA(ctx, cudaFuncSetAttribute(greedy_async_kernel<SV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        int perSm = 0;
        if (path == 3) RCD_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&perSm, greedy_async_kernel<SV>, kSweepThreads, (size_t)smem));
        else RCD_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&perSm, greedy_persistent_kernel<SV>, kSweepThreads, (size_t)smem));
        if (perSm < 1) path = 1;
    }
    if (path == 3) {
        // (a pass over a class is cheap here, the whole GPU serves it: beyond a few dozen raised columns it is the faster way)
        if (ctx->cfg.incremental_max <= 0) prm.deltaMax = 32;
        // In-place correction of stored gains costs about three dependent trips to memory per pick; a pass refreshes every
        // out-of-date block at once, so its cost per pick falls with the number of blocks.  Measured on CIFAR-10-shaped
        // classes: with 8 blocks the correction wins (99 -> 35 ms), with 16 it wins a little once the picks take their v* from
        // the notes (72.6 -> 70.7 ms); with 32 blocks and small classes it loses.
        if (ctx->cfg.incremental == 0) prm.incremental = sz.W <= 16 ? 1 : 0;
        prm.asyncMode = 1;
        prm.nPick = std::min<int>(sz.L, std::max(1, ctx->smCount / 4));
        prm.sweepWarps = (ctx->smCount - prm.nPick) * (kSweepThreads / 32);
        prm.helpMin = ctx->cfg.async_help_min > 0 ? ctx->cfg.async_help_min : 48;
        prm.asyncGroup = ctx->cfg.async_group > 0 ? ctx->cfg.async_group : std::max<int>(sz.L, 1);
    }

    if (path == 3) RCD_CUDA(ctx, cudaMemsetAsync(ws.tickets, 0, (size_t)(sz.N + sz.L) * sizeof(int32_t), st));
    RCD_CUDA(ctx, cudaMemsetAsync(ws.nSweep, 0, 4 * sizeof(int32_t), st));
    RCD_CUDA(ctx, cudaMemsetAsync(ws.phaseNs, 0, kPhaseWords * sizeof(unsigned long long), st));
    ctx->phaseNsDev = ws.phaseNs;
    RCD_CUDA(ctx, cudaMemsetAsync(ws.stepBytes, 0, (size_t)(sz.maxM + 1) * sizeof(unsigned long long), st));
    RCD_CUDA(ctx, cudaMemsetAsync(ws.stepOps, 0, (size_t)(sz.maxM + 1) * sizeof(unsigned long long), st));
    init_kernel<SV><<<sz.L, kSelectThreads, 0, st>>>(prm);
    ctx->kernelLaunches++;
    RCD_CUDA(ctx, cudaGetLastError());

    ctx->sweepEventsUsed = 0;
    // One cooperative launch for the whole loop when the device can hold one sweep CTA per SM at once;
    // per-sweep event timing (profile 2) needs the sweeps as separate launches.
    const bool persistent = path != 1;
    if (path == 4) {
        // (an ordinary launch: the CTAs never wait for one another)
        greedy_owner_kernel<SV><<<std::min<int>(ctx->smCount, sz.L), kSweepThreads, (size_t)smem, st>>>(prm);
        ctx->kernelLaunches += 1;
    } else if (persistent && path == 3) {
        void *args[] = {(void *)&prm};
        RCD_CUDA(ctx, cudaLaunchCooperativeKernel((const void *)greedy_async_kernel<SV>, dim3(ctx->smCount), dim3(kSweepThreads),
                                                  args, (size_t)smem, st));
        ctx->kernelLaunches += 1;
    } else if (persistent) {
        int steps = (int)sz.maxM;
        void *args[] = {(void *)&prm, (void *)&steps};
        RCD_CUDA(ctx, cudaLaunchCooperativeKernel((const void *)greedy_persistent_kernel<SV>, dim3(ctx->smCount), dim3(kSweepThreads),
                                                  args, (size_t)smem, st));
        ctx->kernelLaunches += 1;
    } else {
        if (perSweep) {
            while ((int64_t)ctx->evSweep.size() < 2 * sz.maxM) {
                cudaEvent_t e;
                RCD_CUDA(ctx, cudaEventCreate(&e));
                ctx->evSweep.push_back(e);
            }
        }
        for (int64_t t = 0; t < sz.maxM; ++t) {
            if (perSweep) RCD_CUDA(ctx, cudaEventRecord(ctx->evSweep[2 * t], st));
            RCD_CUDA(ctx, launch_pdl(sweep_kernel<SV>, dim3(ctx->smCount), dim3(kSweepThreads), (size_t)smem, st, prm, (int)t));
            if (perSweep) RCD_CUDA(ctx, cudaEventRecord(ctx->evSweep[2 * t + 1], st));
            RCD_CUDA(ctx, launch_pdl(chain_kernel<SV>, dim3(sz.L), dim3(kSelectThreads), 0, st, prm, (int)t));
            ctx->kernelLaunches += 2;
        }
    }
    if (perSweep) ctx->sweepEventsUsed = 2 * sz.maxM;
    RCD_CUDA(ctx, cudaGetLastError());
    ctx->steps = sz.maxM;
    ctx->stepBytesDev = ws.stepBytes;
    ctx->stepOpsDev = ws.stepOps;
    return RCD_OK;
}

// One CTA arrives at a barrier that expects two: the bounded wait must run out, set the timeout
// bit and return (used by rcd_selftest_bounded_wait to show that a wait which can never be
// satisfied ends as an error status, not as a hang).
__global__ void bounded_wait_selftest_kernel(unsigned *counter, int32_t *status)
{
    grid_barrier(counter, 2u, status, 1u << 12);
}

rcd_status launch_bounded_wait_selftest(rcd_ctx *ctx, unsigned *counter, int32_t *status, cudaStream_t st)
{
    bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(counter, status);
    ctx->kernelLaunches++;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

rcd_status launch_greedy(rcd_ctx *ctx, rcd_feat_dtype dtype, const Sizes &sz, const Workspace &ws,
                         const std::vector<ClassDesc> &descHost, int32_t *assignment, int32_t *order,
                         cudaStream_t st)
{
    if (sz.L == 0 || sz.maxM == 0) return RCD_OK;
    if (dtype == RCD_FEAT_I8) return run_greedy<int32_t>(ctx, sz, ws, descHost, assignment, order, st);
    return run_greedy<float>(ctx, sz, ws, descHost, assignment, order, st);
}

}  // namespace rcd
