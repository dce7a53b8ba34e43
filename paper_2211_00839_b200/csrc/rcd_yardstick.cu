// Yardsticks: what the hardware gives to the two access patterns the hot path is made of, measured with
// kernels of this library's own making, so that a roofline fraction has a denominator of the same kind as
// its numerator.  The paper has no counterpart to any of this.
//
//   rcd_yardstick_read  a read-only sweep: persistent CTAs of 512 threads stream a buffer with the same
//                       128-bit non-allocating loads as the dense gain sweep and fold what they read into a
//                       max-plus checksum.  With a buffer well below the L2 size and many repeats inside
//                       one launch this is the L2-resident read bandwidth; with a buffer of gigabytes and
//                       one repeat it is the HBM read bandwidth.
//   rcd_yardstick_mma   a tensor-core peak loop: every CTA keeps two operand tiles in shared memory and
//                       issues tcgen05.mma (kind::i8 or kind::f16 with bf16 inputs) back to back into two
//                       accumulators in tensor memory: no operand traffic, no epilogue.  The rate it
//                       reaches is what the similarity kernel's tensor work is measured against.
// Both only enqueue; the caller times them with events on the stream it passes.
#include "rcd_internal.h"

namespace rcd {

namespace {

constexpr int kYardThreads = 512;

__device__ __forceinline__ int4 ld_stream16(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Every CTA walks the buffer in slabs of (threads x 4 x 16) bytes, four loads in flight per thread.
__global__ void __launch_bounds__(kYardThreads, 1) yardstick_read_kernel(const int4 *__restrict__ buf, long long n16, int repeats,
                                                                        int *__restrict__ sink)
{
    int acc = 0;
    const long long stride = (long long)gridDim.x * kYardThreads;
    for (int r = 0; r < repeats; ++r) {
        long long i = (long long)blockIdx.x * kYardThreads + threadIdx.x;
        for (; i + 3 * stride < n16; i += 4 * stride) {
            const int4 a = ld_stream16(buf + i), b = ld_stream16(buf + i + stride);
            const int4 c = ld_stream16(buf + i + 2 * stride), d = ld_stream16(buf + i + 3 * stride);
            acc += max(max(a.x, a.y), max(a.z, a.w)) + max(max(b.x, b.y), max(b.z, b.w)) +
                   max(max(c.x, c.y), max(c.z, c.w)) + max(max(d.x, d.y), max(d.z, d.w));
        }
        for (; i < n16; i += stride) {
            const int4 a = ld_stream16(buf + i);
            acc += max(max(a.x, a.y), max(a.z, a.w));
        }
    }
    if (acc == 0x7fffffff) *sink = acc;                 // (keeps the loads alive; practically never true)
}

// ---- tensor-core peak loop ------------------------------------------------------------------------------
constexpr int kMmaM = 128, kMmaN = 256;
constexpr int kSlab = 128;                              // bytes of k per operand row and slab
constexpr int kSlabs = 4;                               // k-slabs kept in shared memory
constexpr int kABytes = kMmaM * kSlab, kBBytes = kMmaN * kSlab;
constexpr uint32_t kYardSpin = 1u << 22;

__device__ __forceinline__ uint32_t saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool bar_test(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(saddr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit is reached.
__device__ __forceinline__ bool bar_wait(uint64_t *bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < kYardSpin; ++spin) {
        if (bar_test(bar, parity)) return true;
        if (spin > 64) __nanosleep(64);
    }
    return false;
}

// K-major operand, 128-byte swizzle, rows 128 bytes apart, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t operand_desc(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffff) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

template <bool kInt8>
__global__ void __launch_bounds__(128, 1) yardstick_mma_kernel(int iters, int32_t *status)
{
    extern __shared__ unsigned char raw[];
    unsigned char *tiles = reinterpret_cast<unsigned char *>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar[2];
    __shared__ uint32_t tmemBase;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // operand bytes: any pattern will do (small integers / small bf16 values, nothing that overflows)
    for (int i = threadIdx.x; i < kSlabs * (kABytes + kBBytes) / 4; i += blockDim.x) {
        uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x;
        reinterpret_cast<uint32_t *>(tiles)[i] = kInt8 ? (h & 0x03030303u) : ((h & 0x00030003u) | 0x3c003c00u);
    }
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(saddr(&bar[0])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(saddr(&bar[1])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(saddr(&tmemBase)), "n"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // the generic-proxy stores above, before the tensor pipe reads them
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmemBase;
    bool ok = true;
    if (warp == 0 && lane == 0) {
        const uint32_t idesc = (kInt8 ? (2u << 4) | (1u << 7) | (1u << 10) : (1u << 4) | (1u << 7) | (1u << 10)) |
                               ((uint32_t)(kMmaN >> 3) << 17) | ((uint32_t)(kMmaM >> 4) << 24);
        for (int it = 0; it < iters && ok; ++it) {
            const uint32_t b = it & 1;
            // the batch issued two iterations ago into this accumulator has retired
            if (it >= 2) ok = bar_wait(&bar[b], ((it >> 1) - 1) & 1);
            if (!ok) break;
            const uint32_t d = tmem + b * kMmaN;
#pragma unroll
            for (int s = 0; s < kSlabs; ++s) {
                const uint64_t da = operand_desc(saddr(tiles + (size_t)s * (kABytes + kBBytes)));
                const uint64_t db = operand_desc(saddr(tiles + (size_t)s * (kABytes + kBBytes) + kABytes));
#pragma unroll
                for (int k = 0; k < kSlab / 32; ++k) {
                    const uint32_t accumulate = (s > 0 || k > 0) ? 1u : 0u;
                    if constexpr (kInt8) {
                        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                     "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                                     :: "r"(d), "l"(da + (uint64_t)(2 * k)), "l"(db + (uint64_t)(2 * k)), "r"(idesc), "r"(accumulate) : "memory");
                    } else {
                        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                     :: "r"(d), "l"(da + (uint64_t)(2 * k)), "l"(db + (uint64_t)(2 * k)), "r"(idesc), "r"(accumulate) : "memory");
                    }
                }
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(saddr(&bar[b])) : "memory");
        }
        // drain: the last batch of each accumulator
        if (ok) {
            for (int it = (iters >= 2 ? iters - 2 : 0); it < iters && ok; ++it) ok = bar_wait(&bar[it & 1], (it >> 1) & 1);
        }
        if (!ok && status) atomicOr(status, kDevTimeout);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "n"(512) : "memory");
    }
}

}  // namespace

}  // namespace rcd

using namespace rcd;

extern "C" rcd_status rcd_yardstick_read(rcd_ctx *ctx, const void *buffer_dev, size_t bytes, int32_t repeats, void *cuda_stream)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    if (!buffer_dev || bytes < 16 || repeats < 1 || ((uintptr_t)buffer_dev) % 16) return fail(ctx, RCD_ERR_INVALID_ARG, "buffer null, unaligned or empty, or repeats < 1");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    yardstick_read_kernel<<<ctx->smCount, kYardThreads, 0, st>>>((const int4 *)buffer_dev, (long long)(bytes / 16), repeats,
                                                                (int *)(ctx->statusOwn + 16));
    ctx->kernelLaunches = 1;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}

extern "C" rcd_status rcd_yardstick_mma(rcd_ctx *ctx, rcd_feat_dtype dtype, int32_t iterations, double *ops_out, void *cuda_stream)
{
    if (!ctx) return RCD_ERR_INVALID_ARG;
    if ((dtype != RCD_FEAT_I8 && dtype != RCD_FEAT_BF16) || iterations < 1) return fail(ctx, RCD_ERR_INVALID_ARG, "unknown dtype or iterations < 1");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    RCD_CUDA(ctx, cudaSetDevice(ctx->device));
    RCD_CUDA(ctx, cudaMemsetAsync(ctx->statusOwn, 0, sizeof(int32_t), st));
    ctx->statusDev = ctx->statusOwn;
    const size_t smem = (size_t)kSlabs * (kABytes + kBBytes) + 1024;
    // one instruction: 128 x 256 outputs x 32 bytes of k (32 int8 or 16 bf16 products each)
    const double perMma = 2.0 * kMmaM * kMmaN * (dtype == RCD_FEAT_I8 ? 32.0 : 16.0);
    if (ops_out) *ops_out = perMma * (kSlab / 32) * kSlabs * (double)iterations * (double)ctx->smCount;
    if (dtype == RCD_FEAT_I8) {
        RCD_CUDA(ctx, cudaFuncSetAttribute(yardstick_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        yardstick_mma_kernel<true><<<ctx->smCount, 128, smem, st>>>(iterations, ctx->statusOwn);
    } else {
        RCD_CUDA(ctx, cudaFuncSetAttribute(yardstick_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        yardstick_mma_kernel<false><<<ctx->smCount, 128, smem, st>>>(iterations, ctx->statusOwn);
    }
    ctx->kernelLaunches = 1;
    RCD_CUDA(ctx, cudaGetLastError());
    return RCD_OK;
}
