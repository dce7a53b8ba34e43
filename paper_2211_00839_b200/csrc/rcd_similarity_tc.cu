// Tensor-core similarity kernel for sm_100a:  S_l = X_l X_l^T  per class (Section 3.1: similarities
// from the feature vectors; int8 -> int32 exact, bf16 -> fp32).
//
// Persistent CTAs (one per SM) walk tiles of 128 rows x 256 columns of every class, those that reach the
// diagonal or lie above it; S is symmetric, so each 128 x 128 block above the diagonal is computed once
// and written twice (itself and its mirror image), which halves the tensor work and the operand traffic
// (a tile whose left half lies below the diagonal computes its right half only).  The tile is twice as wide
// as it is high because the kernel is bound by operand traffic from L2 at 128 x 128 (512 bytes of operands
// per 32 768 multiply-adds and k-step): 128 x 256 moves 768 bytes per 65 536.  Both operands are rows of
// the class-sorted feature matrix (K-major), brought in 128-byte k-slabs by TMA (cp.async.bulk.tensor,
// 128-byte swizzle, out-of-range rows and columns filled with zeros) into a 4-stage shared-memory
// ring; one thread issues tcgen05.mma (kind::i8, or kind::f16 with bf16 inputs) into one of two
// 256-column accumulator buffers in tensor memory, so the next tile's MMAs run while eight warps read the
// previous accumulator back with tcgen05.ld, transpose 32 x 32 blocks through shared memory and
// write S with coalesced 128-bit stores (pad columns as zeros).
//
// Warp roles: 0 = TMA producer, 1 = TMEM allocation + MMA issue, 2..9 = epilogue (two warps per quarter of the
// tensor-memory lanes, one taking the even 32-column blocks of a tile and one the odd ones; the load of a warp's
// next block from tensor memory is in flight while it writes the current one).
// Every wait on an mbarrier is bounded: on expiry the CTA records kDevTimeout in the status
// word, stops issuing work, still waits (bounded) for the copies it has in flight, releases its
// tensor memory and returns.
#include "rcd_internal.h"

#include <cuda.h>

namespace rcd {

namespace {

constexpr int kTileM = 128;
constexpr int kTileN = 256;
constexpr int kSlabBytes = 128;                         // k-slab per stage and operand row
constexpr int kStages = 4;
constexpr int kOperandBytes = kTileM * kSlabBytes;      // 16 KB: 128 rows of one k-slab
constexpr int kStageBytes = 3 * kOperandBytes;          // A (128 rows) + B (256 rows)
constexpr int kEpiWarps = 8;                            // two per quarter of the TMEM lanes
constexpr int kTcThreads = 64 + 32 * kEpiWarps;
constexpr int kTmemCols = 512;                           // two accumulator buffers of 256 columns
constexpr uint32_t kSpinLimit = 1u << 22;               // polls of ~64 ns: a quarter of a second

struct __align__(8) TcShared {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t accFull[2];
    uint64_t accEmpty[2];
    uint32_t tmemBase;
    int32_t abort;
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) when the limit is reached or
// another role has already given up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, TcShared *sh)
{
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        if (mbar_test(bar, parity)) return true;
        if (spin > 64) {
            if (*(volatile int32_t *)&sh->abort) return false;
            __nanosleep(64);
        }
    }
    atomicExch(&sh->abort, 1);
    return false;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(smem_addr(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_addr(bar)) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 bytes apart,
// groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffff) >> 4);             // start address, 16-byte units
    d |= (uint64_t)1 << 16;                             // leading byte offset (unused with 128-byte swizzle, K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset: next 8-row group
    d |= (uint64_t)1 << 46;                             // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                             // layout type: 128-byte swizzle
    return d;
}

template <bool kInt8>
__device__ __forceinline__ void mma_issue(uint32_t tmemD, uint64_t descA, uint64_t descB, uint32_t idesc, uint32_t accumulate)
{
    if constexpr (kInt8) {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                     :: "r"(tmemD), "l"(descA), "l"(descB), "r"(idesc), "r"(accumulate) : "memory");
    } else {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     :: "r"(tmemD), "l"(descA), "l"(descB), "r"(idesc), "r"(accumulate) : "memory");
    }
}

__device__ __forceinline__ void mma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void tmem_load_32cols(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
}
// The registers of an earlier tmem_load_32cols hold their values only after this wait.
__device__ __forceinline__ void tmem_load_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_addr(bar)) : "memory");
}

// Tile idx of the launch -> (class, row block tm of 128 rows, column block sn of 256 columns).  A class lists, row
// block after row block, the tiles with sn >= tm / 2: those that contain a 128 x 128 block on or above the diagonal.
// skip = 128 when the left half of the tile lies below the diagonal (tm odd, sn = tm / 2): that half is the mirror
// image of a block another tile computes, so only the right half is computed.
struct TileCoord { int l, tm, sn, skip, n; };         // n: columns computed, from column sn * 256 + skip on
__device__ __forceinline__ TileCoord decode_tile(const DescSource &src, const int32_t *__restrict__ prefix, int L, int uniTiles, int idx)
{
    TileCoord t;
    int local;
    if (prefix) {
        int lo = 0, hi = L;                              // prefix[lo] <= idx < prefix[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (prefix[mid] <= idx) lo = mid; else hi = mid;
        }
        t.l = lo;
        local = idx - prefix[lo];
    } else {
        t.l = idx / uniTiles;
        local = idx - t.l * uniTiles;
    }
    const ClassDesc c = src.get(t.l);
    const int colBlocks = (c.M + kTileN - 1) / kTileN;
    t.tm = 0;
    for (;;) {
        const int rowLen = colBlocks - t.tm / 2;
        if (local < rowLen) break;
        local -= rowLen;
        ++t.tm;
    }
    t.sn = t.tm / 2 + local;
    t.skip = (2 * t.sn < t.tm) ? kTileM : 0;
    // no further than the rows of S reach, pad columns included (in steps of 32 columns: the epilogue's block, and a
    // legal N of the MMA)
    t.n = min(kTileN - t.skip, (c.ld - (t.sn * kTileN + t.skip) + 31) & ~31);
    return t;
}

template <bool kInt8>
__global__ void __launch_bounds__(kTcThreads, 1) sim_tc_kernel(const __grid_constant__ CUtensorMap map, DescSource src, int32_t L,
                                                              const int32_t *__restrict__ tilePrefix, int32_t uniTiles,
                                                              int32_t totalTiles, int32_t numSlabs, uint32_t *__restrict__ S,
                                                              int32_t *status)
{
    extern __shared__ unsigned char smemRaw[];
    // operand stages need 1024-byte alignment for the 128-byte swizzle pattern
    unsigned char *tiles = reinterpret_cast<unsigned char *>(((uintptr_t)smemRaw + 1023) & ~(uintptr_t)1023);
    __shared__ TcShared sh;
    __shared__ uint32_t stage32[kEpiWarps][32][33];             // per epilogue warp: one 32 x 32 block, padded

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&sh.accFull[b], 1); mbar_init(&sh.accEmpty[b], kEpiWarps); }
        sh.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_addr(&sh.tmemBase)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmemBase = sh.tmemBase;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t it = 0;                             // k-slabs issued so far, over all tiles
            bool ok = true;
            for (int idx = blockIdx.x; idx < totalTiles && ok; idx += gridDim.x) {
                const TileCoord t = decode_tile(src, tilePrefix, L, uniTiles, idx);
                const ClassDesc c = src.get(t.l);
                const int rowA = c.row0 + t.tm * kTileM, rowB = c.row0 + t.sn * kTileN + t.skip;
                const int halves = (t.n + kTileM - 1) / kTileM;         // 128-row pieces of B to bring in: 2, or 1
                for (int kb = 0; kb < numSlabs; ++kb, ++it) {
                    const int s = it % kStages;
                    if (!mbar_wait(&sh.empty[s], ((it / kStages) & 1) ^ 1, &sh)) { ok = false; break; }
                    unsigned char *a = tiles + (size_t)s * kStageBytes;
                    mbar_expect_tx(&sh.full[s], (1 + halves) * kOperandBytes);
                    const int k0 = kb * (kInt8 ? kSlabBytes : kSlabBytes / 2);         // element coordinate
                    tma_load_2d(a, &map, k0, rowA, &sh.full[s]);
                    for (int h = 0; h < halves; ++h) tma_load_2d(a + (1 + h) * kOperandBytes, &map, k0, rowB + h * kTileM, &sh.full[s]);
                }
            }
            // after an abort: let the copies already issued land before the CTA leaves
            if (*(volatile int32_t *)&sh.abort) {
                for (uint32_t k = (it > (uint32_t)kStages ? it - kStages : 0); k < it; ++k) {
                    const int s = k % kStages;
                    for (uint32_t spin = 0; spin < kSpinLimit && !mbar_test(&sh.full[s], (k / kStages) & 1); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            // instruction descriptor: D format, A/B format, K-major operands, N and M of the tile
            const uint32_t idescBase = (kInt8 ? (2u << 4) | (1u << 7) | (1u << 10)   // S32 accumulate, S8 x S8
                                              : (1u << 4) | (1u << 7) | (1u << 10))  // F32 accumulate, BF16 x BF16
                                       | ((uint32_t)(kTileM >> 4) << 24);
            uint32_t it = 0, nt = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < totalTiles && ok; idx += gridDim.x, ++nt) {
                const TileCoord t = decode_tile(src, tilePrefix, L, uniTiles, idx);
                const uint32_t idesc = idescBase | ((uint32_t)(t.n >> 3) << 17);   // N = 256, less for a half tile or at the class's edge
                const uint32_t buf = nt & 1;
                // the epilogue must have drained this accumulator buffer (two tiles ago)
                if (!mbar_wait(&sh.accEmpty[buf], ((nt >> 1) & 1) ^ 1, &sh)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmemD = tmemBase + buf * kTileN;
                for (int kb = 0; kb < numSlabs; ++kb, ++it) {
                    const int s = it % kStages;
                    if (!mbar_wait(&sh.full[s], (it / kStages) & 1, &sh)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t aAddr = smem_addr(tiles + (size_t)s * kStageBytes);
                    const uint64_t descA = make_smem_desc(aAddr);
                    const uint64_t descB = make_smem_desc(aAddr + kOperandBytes);
#pragma unroll
                    for (int k = 0; k < kSlabBytes / 32; ++k)          // one MMA consumes 32 bytes of k per row
                        mma_issue<kInt8>(tmemD, descA + (uint64_t)(2 * k), descB + (uint64_t)(2 * k), idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    mma_commit(&sh.empty[s]);                          // frees the stage when those MMAs retire
                }
                mma_commit(&sh.accFull[buf]);                          // accumulator complete (or abandoned)
            }
        }
    } else {
        // ---------------- epilogue: TMEM -> registers -> shared (transpose) -> global ----------------
        const int q = warp & 3;                                        // TMEM lane quarter this warp may read
        const int ew = warp - 2;
        const int half = ew >> 2;                                      // which column blocks of the tile: even or odd
        uint32_t nt = 0;
        for (int idx = blockIdx.x; idx < totalTiles; idx += gridDim.x, ++nt) {
            const TileCoord t = decode_tile(src, tilePrefix, L, uniTiles, idx);
            const ClassDesc c = src.get(t.l);
            const int rowA = t.tm * kTileM, colB = t.sn * kTileN + t.skip;   // class-local: first row, first column computed
            const uint32_t buf = nt & 1;
            if (!mbar_wait(&sh.accFull[buf], (nt >> 1) & 1, &sh)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (*(volatile int32_t *)&sh.abort) break;
            uint32_t *Sl = S + c.sOff;
            const int cg = (lane & 7) * 4;                             // this lane's 4 columns of a 32-wide block
            const int nCb = t.n / 32;
            const uint32_t tmemRow = tmemBase + buf * kTileN + ((uint32_t)(q * 32) << 16);
            uint32_t v[32];
            if (half < nCb) tmem_load_32cols(tmemRow + (uint32_t)(half * 32), v);
#pragma unroll 1
            for (int cb = half; cb < nCb; cb += kEpiWarps / 4) {
                // the 128 x 128 block this column block belongs to lies on the diagonal (stored once) or above it
                // (stored twice: itself and its mirror image)
                const bool diag = (colB + cb * 32) / kTileM == t.tm;
                tmem_load_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) stage32[ew][lane][j] = v[j];         // lane = row inside the quarter
                __syncwarp();
                // the next block of this warp travels from tensor memory while this one is written out
                if (cb + kEpiWarps / 4 < nCb) tmem_load_32cols(tmemRow + (uint32_t)((cb + kEpiWarps / 4) * 32), v);
                // block rows -> S[rowA + ..][colB + ..]: 8 lanes cover 32 columns with 128-bit stores, 4 rows per pass
                {
                    const int col = colB + cb * 32 + cg;
#pragma unroll
                    for (int pass = 0; pass < 8; ++pass) {
                        const int r = pass * 4 + (lane >> 3);
                        const int row = rowA + q * 32 + r;
                        if (row < c.M && col < c.ld) {
                            uint4 o;
                            o.x = col + 0 < c.M ? stage32[ew][r][cg + 0] : 0u;
                            o.y = col + 1 < c.M ? stage32[ew][r][cg + 1] : 0u;
                            o.z = col + 2 < c.M ? stage32[ew][r][cg + 2] : 0u;
                            o.w = col + 3 < c.M ? stage32[ew][r][cg + 3] : 0u;
                            *reinterpret_cast<uint4 *>(Sl + (int64_t)row * c.ld + col) = o;
                        }
                    }
                }
                // the mirrored block -> S[colB + ..][rowA + ..] (blocks below the diagonal are never computed)
                if (!diag) {
                    const int col = rowA + q * 32 + cg;
#pragma unroll
                    for (int pass = 0; pass < 8; ++pass) {
                        const int jj = pass * 4 + (lane >> 3);
                        const int row = colB + cb * 32 + jj;
                        if (row < c.M && col < c.ld) {
                            uint4 o;
                            o.x = col + 0 < c.M ? stage32[ew][cg + 0][jj] : 0u;
                            o.y = col + 1 < c.M ? stage32[ew][cg + 1][jj] : 0u;
                            o.z = col + 2 < c.M ? stage32[ew][cg + 2][jj] : 0u;
                            o.w = col + 3 < c.M ? stage32[ew][cg + 3][jj] : 0u;
                            *reinterpret_cast<uint4 *>(Sl + (int64_t)row * c.ld + col) = o;
                        }
                    }
                }
                __syncwarp();
            }
            // hand the accumulator buffer back to the MMA warp
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.accEmpty[buf]);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmemBase), "r"(kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && sh.abort && status) atomicOr(status, kDevTimeout);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

rcd_status launch_similarity_tc(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t Ntot, int64_t d,
                                const SimClasses &cls, void *S, cudaStream_t st, bool *handled)
{
    *handled = false;
    const int64_t rowBytes = d * (int64_t)feat_bytes(dtype);
    // TMA needs 16-byte row pitch and base; a row shorter than one 128-byte slab goes to the generic kernel
    if (rowBytes % 16 != 0 || rowBytes < kSlabBytes || ((uintptr_t)Xs) % 16 != 0 || ((uintptr_t)S) % 16 != 0) return RCD_OK;
    if (cls.L == 0 || cls.maxM == 0 || Ntot == 0) { *handled = true; return RCD_OK; }
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return fail(ctx, RCD_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");

    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)Ntot};
    const cuuint64_t strides[1] = {(cuuint64_t)rowBytes};
    const cuuint32_t box[2] = {(cuuint32_t)(dtype == RCD_FEAT_I8 ? kSlabBytes : kSlabBytes / 2), (cuuint32_t)kTileM};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = encode(&map, dtype == RCD_FEAT_I8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                         const_cast<void *>(Xs), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(ctx, RCD_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)cr);

    const int numSlabs = (int)((rowBytes + kSlabBytes - 1) / kSlabBytes);
    const size_t smem = (size_t)kStages * kStageBytes + 1024;
    if (cls.upperTiles <= 0 || cls.upperTiles > 0x7fffffffLL) return RCD_OK;
    const int totalTiles = (int)cls.upperTiles;
    const int grid = totalTiles < ctx->smCount ? totalTiles : ctx->smCount;
    int32_t *status = const_cast<int32_t *>(ctx->statusDev);
    if (dtype == RCD_FEAT_I8) {
        RCD_CUDA(ctx, cudaFuncSetAttribute(sim_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sim_tc_kernel<true><<<grid, kTcThreads, smem, st>>>(map, cls.src, cls.L, cls.tilePrefixDev, cls.uniTiles, totalTiles,
                                                           numSlabs, (uint32_t *)S, status);
    } else {
        RCD_CUDA(ctx, cudaFuncSetAttribute(sim_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sim_tc_kernel<false><<<grid, kTcThreads, smem, st>>>(map, cls.src, cls.L, cls.tilePrefixDev, cls.uniTiles, totalTiles,
                                                            numSlabs, (uint32_t *)S, status);
    }
    ctx->kernelLaunches++;
    ctx->tcLaunches++;
    RCD_CUDA(ctx, cudaGetLastError());
    *handled = true;
    return RCD_OK;
}

}  // namespace rcd
