/*
 * rcd.h -- C ABI of the B200 (sm_100a) library for the resource-constrained
 * submodular data partition of RCD-SGD (Algorithm 1, "Ratio-Constrained
 * submodular partitioning", with the facility-location objective of Section 4,
 * item 2).
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers on the context's device; "host"
 *     pointers are ordinary host memory.  The caller owns every buffer,
 *     including the workspace; the library never frees them and reads nothing of them after the
 *     call's last kernel (the device-side status of a call is copied into the context).
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Unless stated otherwise a call only enqueues work on that stream and
 *     returns; outputs are valid once the stream has been synchronised.
 *   - Argument errors are reported synchronously (nothing is launched, nothing is
 *     written).  A CUDA runtime failure returns RCD_ERR_CUDA.  Errors detected on
 *     the device land in a status word and are returned by rcd_sync_status().
 *   - No exception crosses this boundary and there is no CPU fallback: a
 *     configuration the kernels do not cover returns RCD_ERR_UNSUPPORTED.
 *   - Not thread-safe per context: use one context per host thread.
 *
 * Readings of the paper fixed by this library (the paper is silent on each):
 *   f(A) = sum_{i in V_l} max(0, max_{v' in A} S[i][v']),  f(empty) = 0;
 *   argmin over blocks and argmax over samples break ties toward the lowest index;
 *   quotas by largest remainder (rcd_quotas).
 */
#ifndef RCD_H_
#define RCD_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define RCD_API __attribute__((visibility("default")))
#else
#define RCD_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RCD_OK = 0,
    RCD_ERR_INVALID_ARG = 1,
    RCD_ERR_UNSUPPORTED = 2,
    RCD_ERR_WORKSPACE_TOO_SMALL = 3,
    RCD_ERR_CUDA = 4,
    RCD_ERR_TIMEOUT = 5,
    RCD_ERR_INTERNAL = 6
} rcd_status;

/* Feature element type.  It also fixes the arithmetic of everything downstream:
 *   RCD_FEAT_I8   int8 features, S = dot product in int32 (exact), gains and f in int64 (exact);
 *   RCD_FEAT_BF16 bfloat16 features (rows L2-normalised by the caller, so the dot product is the
 *                 cosine), S accumulated and stored in fp32, gains in fp32, f tracked in fp64.  */
typedef enum { RCD_FEAT_I8 = 0, RCD_FEAT_BF16 = 1 } rcd_feat_dtype;

/* Similarity sim(v, v') of Section 4 item 2.
 *   RCD_SIM_DOT       the dot product of the feature vectors (the cosine when rows are normalised);
 *   RCD_SIM_GAUSSIAN  exp(-||v - v'||^2 / (2 sigma^2)) with sigma = the mean of ||v - v'||_2 over all ordered
 *                     pairs of the class (the paper's Gaussian kernel; exponent and the range of the mean are
 *                     readings, the paper gives neither).  S is then fp32 in (0, 1] for either feature type,
 *                     and everything downstream uses the floating-point arithmetic of RCD_FEAT_BF16
 *                     (gains fp32, tracked f and all objective outputs double).  */
typedef enum { RCD_SIM_DOT = 0, RCD_SIM_GAUSSIAN = 1 } rcd_similarity_kind;

/* Submodular function f used by GreedyStep and by the argmin over blocks (Section 4 item 2).
 *   RCD_OBJ_FACILITY   facility location, f(A) = sum_{v in V_l} max_{v' in A} sim(v, v') (clamped at 0);
 *   RCD_OBJ_GRAPH_CUT  graph cut, f(A) = sum_{v in V_l \\ A} sum_{v' in A} sim(v, v').  Needs no pass over S per
 *                      pick (the gain of u is a column sum minus twice its tie to the block); values are
 *                      int64 for int8 features with RCD_SIM_DOT, double otherwise.  Not monotone: gains
 *                      can be negative; Algorithm 1 runs unchanged. */
typedef enum { RCD_OBJ_FACILITY = 0, RCD_OBJ_GRAPH_CUT = 1 } rcd_objective_kind;

typedef struct {
    int32_t sweep_batch_max;   /* blocks whose gains one pass over S may refresh: 1,2,4 or 8; 0 = default (8) */
    int32_t similarity_path;   /* 0 = tensor-core kernel when the shape allows, 2 = always the generic kernel */
    int32_t profile;           /* 0 off; 1 time the phases of rcd_partition; 2 also time every sweep launch */
    int32_t greedy_path;       /* form of the greedy loop.  0 = choose: asynchronous classes (3) when there are at most a quarter
                                  as many classes as SMs, else one CTA per class (4);  1 = two launches per round (always
                                  used with profile 2);  2 = one cooperative launch, rounds of a sweep phase and a pick phase
                                  separated by grid barriers;  3 = one cooperative launch, every class cycles between sweep and
                                  picks on its own: some CTAs only make picks, the others only sweep, so picks overlap other
                                  classes' sweeps;  4 = one launch, every CTA draws a class and runs it from its first pick
                                  to its last (no barrier, no hand-off; picks of one SM overlap sweeps of the others).
                                  All forms make the same picks. */
    int32_t similarity_kind;   /* rcd_similarity_kind used by rcd_partition / rcd_objective (default RCD_SIM_DOT) */
    int32_t objective;         /* rcd_objective_kind used by rcd_partition / rcd_objective (default facility location) */
    int32_t sweep_mode;        /* 0 = threshold passes once the blocks have a few members (up to 64 blocks per pass);
                                  1 = dense passes only (sweep_batch_max blocks per pass) */
    int32_t async_group;       /* greedy_path 3: how many sweeps (ordered by sweep number, then class) the sweep CTAs serve
                                  together, each CTA going to the class nearest its home position; 1 = strictly in
                                  order; 0 = default: all classes together */
    int32_t async_help_min;    /* greedy_path 3: row groups a sweep must have left before a sweep CTA whose home is another
                                  class joins it; 0 = default (48) */
    int32_t threshold_from;    /* members every out-of-date block must have before a class tries threshold passes; 0 = default (8) */
    int32_t threshold_hit_shift; /* a threshold pass that finds more than 1 element in 2^k above the threshold sends the class
                                  back to dense passes until its blocks have twice the members; 0 = default (k = 5) */
    int32_t lazy_mode;         /* exact lazy evaluation of GreedyStep's argmax.  0 = off: every pass visits every unassigned row.
                                  1 = on: a threshold pass skips rows whose stored gains (upper bounds of the current ones, by
                                  diminishing returns) lie below a per-block floor; a pick whose best stored gain is below
                                  its block's floor is not made, the block gets a pass over every row instead.  Same picks
                                  either way; fewer bytes read, but each class waits longer for its short passes. */
    int32_t lazy_from;         /* members every out-of-date block must have before rows are skipped; 0 = default (8) */
    int32_t dense_ring;        /* 0 = 8-block dense passes stream S through per-warp rings of asynchronous copies in shared
                                  memory when the coverage vectors leave room for them; 2 = never (one register buffer ahead) */
    int32_t incremental;       /* in-place correction of stored gains (greedy paths 3 and 4).  When a pick raised its block's coverage
                                  in few columns i, every candidate's gain falls by max(0, S[v][i] - old_i) - max(0, S[v][i] - new_i),
                                  read from row i of S (S is symmetric): the block's stored gains stay exact and it needs no
                                  pass over S.  0 = choose (on for path 3 with at most 16 blocks and for path 4 with classes of 1024 samples or
                                  more: where it was measured faster), 1 = on,
                                  2 = off (every block that received a sample waits for a pass).  Same picks either way. */
    int32_t incremental_max;   /* most columns a pick may raise and still be corrected in place; 0 = default (32 for greedy
                                  path 3, where a pass is served by the whole GPU; 64 for path 4); at most 128 */
} rcd_config;

/* Timings and counters of the last rcd_partition / rcd_partition_host on a context (profile >= 1). */
typedef struct {
    double  total_ms;          /* whole call, first to last kernel, on the call's stream */
    double  group_ms;          /* class split + feature gather */
    double  similarity_ms;     /* similarity kernel(s) */
    double  greedy_ms;         /* all greedy steps */
    double  sweep_ms;          /* profile 2: summed duration of the sweep launches that had work */
    int64_t sweep_launches;    /* profile 2: number of those launches */
    int64_t sweep_bytes;       /* bytes of S and of coverage vectors those launches had to read */
    int64_t sweep_elem_ops;    /* (element of S) x (block refreshed) pairs those launches evaluated */
    int64_t kernel_launches;   /* kernels this library launched during the call */
    int64_t steps;             /* greedy steps executed (= largest class size) */
    int64_t similarity_tc_launches; /* similarity launches of the last call that ran on the tensor cores */
    int64_t persistent_sweep_ns;    /* one-launch greedy loop: time in sweep phases (incl. their barrier); asynchronous
                                       form: time the first sweep CTA spent sweeping (not looking for work) */
    int64_t persistent_pick_ns;     /* one-launch greedy loop: time in pick phases (incl. their barrier); asynchronous
                                       form: time the first pick CTA spent making picks (not waiting for sweeps) */
    int64_t threshold_hits;         /* threshold passes: elements of S above the threshold ... */
    int64_t threshold_elems;        /* ... out of this many elements compared */
    int64_t threshold_max_blocks;   /* most blocks one threshold pass refreshed */
    int64_t async_lull_ns;          /* asynchronous form: time the first sweep CTA found no sweep with tickets left */
    int64_t async_visits;           /* asynchronous form: times the first sweep CTA went to a class and swept there */
    int64_t async_attempts;         /* ... and times it tried (an attempt fails when the tickets run out under way) */
    int64_t lazy_sweeps;            /* threshold passes that skipped rows below the blocks' floors */
    int64_t lazy_misses;            /* picks whose best stored gain lay below its block's floor (answered by a pass over every row) */
    int64_t lazy_rows;              /* rows of S those passes did read */
    int64_t lazy_rows_skipped;      /* rows they did not */
    int64_t incremental_updates;    /* picks after which the block's stored gains were corrected in place (no pass needed) */
    int64_t incremental_rows;       /* rows of S those corrections read (one per column whose coverage rose) */
    int64_t threshold_pass_ns;      /* one CTA per class: time the first CTA spent in threshold passes (part of persistent_sweep_ns) */
    int64_t threshold_pass_bytes;   /* bytes of S and threshold vectors the (row-visiting) threshold passes had to read (part of sweep_bytes) */
    int64_t noted_picks;            /* picks whose v* was noted when the block's stored gains were last corrected (no argmax over stored gains) */
} rcd_profile;

typedef struct rcd_ctx rcd_ctx;

/* ---- context ------------------------------------------------------------------------------ */

/* Creates a context bound to CUDA device `cuda_device` (it owns only a few events, a small pinned
 * staging buffer and a 256-byte device status block).  `cfg_or_null` NULL = defaults.  Fails with RCD_ERR_UNSUPPORTED on a
 * device that is not compute capability 10.x, RCD_ERR_CUDA when no device can be used. */
RCD_API rcd_status rcd_create(rcd_ctx **out, int cuda_device, const rcd_config *cfg_or_null);
RCD_API void rcd_destroy(rcd_ctx *ctx);
/* Text of the last error on this context (owned by the context; "" if none). NULL ctx allowed. */
RCD_API const char *rcd_last_error(const rcd_ctx *ctx);
RCD_API const char *rcd_version(void);

/* Waits for `cuda_stream` and returns the device-side status of the last call on the context. */
RCD_API rcd_status rcd_sync_status(rcd_ctx *ctx, void *cuda_stream);
/* Self-test of the bounded waits the kernels use (grid barrier of the greedy loop, mbarrier waits of the
 * tensor-core kernel): enqueues a one-CTA kernel that arrives at a barrier expecting two arrivals.  The wait
 * gives up after a few thousand polls and records the timeout in the context's status word, so the next
 * rcd_sync_status returns RCD_ERR_TIMEOUT and the context stays usable.  Nothing faults or hangs. */
RCD_API rcd_status rcd_selftest_bounded_wait(rcd_ctx *ctx, void *cuda_stream);
/* Waits for the events of the last profiled call and fills `out`. */
RCD_API rcd_status rcd_get_profile(rcd_ctx *ctx, rcd_profile *out);

/* ---- quotas (Algorithm 1: "Constraint C_{l,j} = |V_l| r_j / sum_j r_j") -------------------- */

/* Host-only.  Integer quotas of one class of M samples over W blocks with capacity ratios
 * `capacities_host[W]` (finite, > 0), by largest remainder in IEEE double: shares
 * q_j = M*r_j/(r_0+r_1+...) are floored and the left-over units go one each to the largest
 * fractional parts, ties to the lowest j.  sum_j quotas[j] == M.  No GPU is touched. */
RCD_API rcd_status rcd_quotas(int64_t M, const double *capacities_host, int32_t W, int32_t *quotas_host_out);

/* ---- similarity (Section 3.1 / Section 4 item 2: sim(v, v') from the feature vectors) ------ */

/* S_b = X_b X_b^T for `batch` classes of equal size.
 *   X_dev  [batch][M][d] row-major, int8 or bf16 (16-byte aligned base)
 *   S_dev  [batch][M][ldS] row-major, int32 (I8) or fp32 (BF16); ldS a multiple of 4 with
 *          M <= ldS <= M rounded up to a multiple of 64 (anything else: RCD_ERR_INVALID_ARG);
 *          columns M..ldS-1 of every row are written as 0.
 * I8 requires 16384*d < 2^31 so that S cannot overflow int32. */
RCD_API rcd_status rcd_similarity(rcd_ctx *ctx, const void *X_dev, rcd_feat_dtype dtype, int64_t M, int64_t d,
                          int64_t batch, void *S_dev, int64_t ldS, void *cuda_stream);

/* Gaussian-kernel similarity of `batch` equal classes (see rcd_similarity_kind), whatever the context's
 * similarity_kind.  S_dev is fp32 [batch][M][ldS] (ldS as for rcd_similarity, pad columns 0);
 * sigma_dev_or_null receives the `batch` bandwidths (fp32).  It first forms the dot products like
 * rcd_similarity, then transforms them in place; the workspace holds row norms and partial sums. */
RCD_API rcd_status rcd_similarity_gaussian_workspace_bytes(rcd_ctx *ctx, int64_t M, int64_t batch, size_t *bytes_out);
RCD_API rcd_status rcd_similarity_gaussian(rcd_ctx *ctx, const void *X_dev, rcd_feat_dtype dtype, int64_t M, int64_t d,
                                   int64_t batch, void *S_dev, int64_t ldS, float *sigma_dev_or_null,
                                   void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/* ---- partition (Algorithm 1 + GreedyStep, facility location) ------------------------------ */

/* Upper bound of the workspace rcd_partition needs for N samples of width d in L classes none
 * larger than M_max, W blocks.  (rcd_partition recomputes the exact need from the label counts
 * and returns RCD_ERR_WORKSPACE_TOO_SMALL if a class was larger than promised.) */
RCD_API rcd_status rcd_partition_workspace_bytes(rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d,
                                         int32_t L, int64_t M_max, int32_t W, size_t *bytes_out);

/* Partitions every class of the dataset into W blocks.
 *   features_dev [N][d] row-major; labels_dev [N], each in [0, L) (classes may be empty and of
 *   unequal size; inside a class samples keep their dataset order, which fixes tie-breaks);
 *   capacities_host [W] the ratios r_j (finite, > 0).
 * Outputs (device):
 *   assignment_dev [N]            block of every sample, in [0, W)
 *   order_dev_or_null [N]         class-major (ascending label); inside a class the dataset
 *                                 indices of its samples in the order they were picked
 *   part_values_dev_or_null [L][W] tracked f(A_j^l): int64 (I8 with RCD_SIM_DOT), else double
 * workspace_dev: 256-byte aligned, at least rcd_partition_workspace_bytes.
 * The call blocks once, briefly, on `cuda_stream` to read the L class sizes back (they fix the
 * launch shapes); everything after that is only enqueued.  Per class and per pick it runs:
 * choose the non-full block of least f; (re)compute the marginal gains
 * sum_i max(0, S[v][i] - cover_p[i]) of every unassigned v for that block, and in the same
 * pass over S for other non-full blocks whose stored gains are out of date (a block's gains
 * only change when the block itself receives a sample); argmax with lowest-index ties;
 * fold row v* into the block's coverage vector and update counts. */
RCD_API rcd_status rcd_partition(rcd_ctx *ctx, const void *features_dev, rcd_feat_dtype dtype, int64_t N, int64_t d,
                         const int32_t *labels_dev, int32_t L, const double *capacities_host, int32_t W,
                         int32_t *assignment_dev, int32_t *order_dev_or_null, void *part_values_dev_or_null,
                         void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/* Same computation with HOST inputs and outputs: copies features and labels to the device
 * (staging areas inside the workspace), runs rcd_partition, copies the results back and
 * synchronises the stream before returning, so the host outputs are valid on return.
 * Pinned host memory makes the copies asynchronous; pageable memory works too. */
RCD_API rcd_status rcd_partition_host_workspace_bytes(rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d,
                                              int32_t L, int64_t M_max, int32_t W, size_t *bytes_out);
RCD_API rcd_status rcd_partition_host(rcd_ctx *ctx, const void *features_host, rcd_feat_dtype dtype, int64_t N,
                              int64_t d, const int32_t *labels_host, int32_t L,
                              const double *capacities_host, int32_t W, int32_t *assignment_host,
                              int32_t *order_host_or_null, void *part_values_host_or_null,
                              void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/* ---- objective (Section 4 item 2: f(A) = sum_{v in V_l} max_{v' in A} sim(v, v')) ---------- */

RCD_API rcd_status rcd_objective_workspace_bytes(rcd_ctx *ctx, rcd_feat_dtype dtype, int64_t N, int64_t d,
                                         int32_t L, int64_t M_max, int32_t W, size_t *bytes_out);

/* Recomputes f(A_j^l) for every class l and block j from the plain definition, given an
 * assignment (values in [0, W); a negative entry means "in no block").  Independent of the
 * greedy state: it rebuilds S and takes, per row i and block j, the maximum over the block's
 * members.
 *   part_values_dev [L][W]  int64 (I8 with RCD_SIM_DOT), else double
 *   total_dev               one value of the same type: the sum over all (l, j)
 * Blocks once on the stream, like rcd_partition, to read the class sizes. */
RCD_API rcd_status rcd_objective(rcd_ctx *ctx, const void *features_dev, rcd_feat_dtype dtype, int64_t N, int64_t d,
                         const int32_t *labels_dev, int32_t L, const int32_t *assignment_dev, int32_t W,
                         void *part_values_dev, void *total_dev, void *workspace_dev,
                         size_t workspace_bytes, void *cuda_stream);

/* ---- per-worker lists and batch sizes (Algorithm 2, initialisation: every worker imports its local subset
 *      from the blocks A_1 .. A_N and runs with a batch size set by its capacity ratio) ------------------------ */

RCD_API rcd_status rcd_worker_lists_workspace_bytes(rcd_ctx *ctx, int64_t N, int32_t W, size_t *bytes_out);

/* Turns an assignment (rcd_partition's output) into one index list per worker.
 *   assignment_dev [N]   block of every sample, each in [0, W) (anything else: RCD_ERR_INVALID_ARG)
 *   offsets_dev    [W+1] out, int64: worker j's list is indices_dev[offsets[j] .. offsets[j+1])
 *   indices_dev    [N]   out: dataset indices, ascending inside every list
 * workspace_dev: 256-byte aligned, rcd_worker_lists_workspace_bytes.  Blocks once on the stream to read the W
 * list sizes back (they fix the offsets); the lists themselves are only enqueued. */
RCD_API rcd_status rcd_worker_lists(rcd_ctx *ctx, const int32_t *assignment_dev, int64_t N, int32_t W, int64_t *offsets_dev,
                            int32_t *indices_dev, void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/* Host-only.  Batch size of every worker for a reference batch size B of worker 1: b_j = B r_j / r_1, rounded
 * half up, at least 1.  (The text below Algorithm 2 makes the batch size proportional to the processing speed;
 * the algorithm's own initialisation line prints the inverse ratio, B r_1 / r_j.  This follows the text: with
 * lists and batches both proportional to r_j every worker needs the same number of steps per epoch.) */
RCD_API rcd_status rcd_batch_sizes(int64_t B, const double *capacities_host, int32_t W, int64_t *batch_sizes_host_out);

/* The same with the reading chosen by the caller.  RCD_BATCH_PROPORTIONAL: b_j = B r_j / r_1 (rcd_batch_sizes: the text
 * below Algorithm 2).  RCD_BATCH_AS_PRINTED: b_j = B r_1 / r_j, the ratio as Algorithm 2's initialisation line prints
 * it (fast workers then get the smallest batches).  Rounded half up, at least 1, either way.  Host-only. */
typedef enum { RCD_BATCH_PROPORTIONAL = 0, RCD_BATCH_AS_PRINTED = 1 } rcd_batch_rule;
RCD_API rcd_status rcd_batch_sizes_rule(int64_t B, const double *capacities_host, int32_t W, rcd_batch_rule rule,
                                int64_t *batch_sizes_host_out);

/* ---- objective of one class without any allocation (no counterpart in the paper) ----------- */

/* The paper has nothing corresponding to this entry point: it exists for callers that cannot
 * allocate device memory (code running inside a fixed, pre-carved memory budget or in a region
 * where touching the CUDA allocator is not allowed) and so cannot supply the workspace that
 * rcd_objective needs.  It computes the facility-location value f(A_j) of the W blocks of ONE
 * class from a similarity matrix the caller already has (for instance from rcd_similarity), using
 * a 1 MiB scratch array that is built into the library instead of a workspace.  A context whose
 * objective is RCD_OBJ_GRAPH_CUT is refused (RCD_ERR_UNSUPPORTED), not silently given other values.
 *   S_dev           [M][ldS] row-major, int32 (RCD_FEAT_I8) or fp32 (RCD_FEAT_BF16), ldS >= M
 *   assignment_dev  [M] block of each sample of the class, in [0, W); negative = in no block
 *   part_values_dev [W] int64 / double;  total_dev one int64 / double (their sum)
 * Limits: W <= 1024 and ceil(M/64) * W * 8 <= 1048576 bytes, otherwise RCD_ERR_UNSUPPORTED with
 * the sizes in rcd_last_error.  The array is held by every GPU that loads the library until the
 * process exits.  All calls on a device share it: calls whose kernels overlap on the GPU race,
 * so keep them on one stream or order them with events.  It keeps the previous call's partial
 * sums; every slot a call reads has been written by that call first, so nothing needs clearing.
 * The first call on each device looks up the array's device address (the lookup is serialised
 * across host threads); make that first call outside any stream capture.  Like every call of this
 * library it leaves the context's device current.  No cudaMalloc/cudaFree or allocating routine
 * is called. */
RCD_API rcd_status rcd_objective_class_static(rcd_ctx *ctx, const void *S_dev, rcd_feat_dtype dtype, int64_t M,
                                      int64_t ldS, const int32_t *assignment_dev, int32_t W,
                                      void *part_values_dev, void *total_dev, void *cuda_stream);

/* ---- yardsticks (measurement only; no counterpart in the paper) ------------------------------ */

/* A read-only sweep with the access pattern of the dense gain sweep (one CTA of 512 threads per SM, 128-bit loads
 * that do not allocate in L1): reads `bytes` bytes at buffer_dev (16-byte aligned, owned by the caller, contents
 * irrelevant) `repeats` times inside ONE launch.  A buffer well below the L2 size with many repeats measures the
 * L2-resident read bandwidth, a buffer of gigabytes with one repeat the HBM read bandwidth: bytes * repeats over
 * the time the caller measures with events on cuda_stream.  Only enqueues. */
RCD_API rcd_status rcd_yardstick_read(rcd_ctx *ctx, const void *buffer_dev, size_t bytes, int32_t repeats, void *cuda_stream);

/* A tensor-core peak loop: one CTA per SM issues `iterations` batches of sixteen 128 x 256 x (32-byte k)
 * tcgen05.mma instructions (RCD_FEAT_I8: s8 x s8 -> s32; RCD_FEAT_BF16: bf16 x bf16 -> f32) on operands that stay in
 * shared memory, accumulators in tensor memory.  *ops_host_out (may be NULL) receives the number of arithmetic
 * operations (2 per multiply-add) the launch performs; divide by the time measured on cuda_stream.  Every wait in
 * the kernel is bounded (RCD_ERR_TIMEOUT from rcd_sync_status otherwise).  Only enqueues. */
RCD_API rcd_status rcd_yardstick_mma(rcd_ctx *ctx, rcd_feat_dtype dtype, int32_t iterations, double *ops_host_out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RCD_H_ */
