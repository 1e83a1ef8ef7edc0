// Tensor-pipe issue-peak microbenchmark: back-to-back tcgen05.mma on operands that stay
// resident in shared memory (no loads, no unpack, no epilogue), one CTA per SM.  It
// gives the roof the GEMM kernels are measured against on the box they run on:
// multiply-accumulates per clock per SM for kind::i8 (u8 x u8 -> s32), and for
// kind::f16 (bf16) / kind::f8f6f4 (e4m3) as cross-checks against the measured bf16
// library figure.
#include <cuda.h>

#include "q4_common.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {
namespace peak {

constexpr int ROWS_A = 128, ROWS_B = 256, UROW = 128;
constexpr int OFF_A = 0, OFF_B = ROWS_A * UROW, OFF_BAR = OFF_B + ROWS_B * UROW;
constexpr int SMEM = OFF_BAR + 64 + 1024;

// kind: 0 = i8 (u8 x u8 -> s32), 1 = f16 (bf16 x bf16 -> f32), 2 = f8f6f4 (e4m3 -> f32)
__device__ __forceinline__ void mma_kind(int kind, uint32_t d, uint64_t a, uint64_t b, uint32_t idesc,
                                         uint32_t acc)
{
    if (kind == 0) {
        tc_mma_i8(d, a, b, idesc, acc);
    } else if (kind == 1) {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
    } else {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
    }
}

__global__ void __launch_bounds__(128, 1)
peak_kernel(int kind, int n, int iters, unsigned long long* cycles, unsigned* status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar = sbase + OFF_BAR, slot = sbase + OFF_BAR + 16, abort_flag = sbase + OFF_BAR + 20;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // operands: all zero (valid in every format)
    for (uint32_t o = threadIdx.x * 16u; o < (uint32_t)OFF_BAR; o += blockDim.x * 16u)
        sts128(sbase + o, make_uint4(0, 0, 0, 0));
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        sts32(abort_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_async_smem();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(slot), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = (uint32_t)lds32(slot);

    if (warp == 0 && lane == 0) {
        // c_format: s32 for i8, f32 otherwise; a/b format: u8 / bf16 / e4m3
        const uint32_t cfmt = kind == 0 ? 2u : 1u;
        const uint32_t abfmt = kind == 1 ? 1u : 0u;
        const uint32_t idesc = (cfmt << 4) | (abfmt << 7) | (abfmt << 10) |
                               ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint64_t adesc = make_kmajor_sw128_desc(sbase + OFF_A);
        const uint64_t bdesc = make_kmajor_sw128_desc(sbase + OFF_B);
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it)
#pragma unroll
            for (int i = 0; i < 4; ++i)      // four 32-byte depth steps of one 128-byte row
                mma_kind(kind, tmem_base, adesc + (uint64_t)(2 * i), bdesc + (uint64_t)(2 * i), idesc,
                         (it | i) ? 1u : 0u);
        tc_commit(bar);
        mbar_wait(bar, 0, abort_flag, status);
        const long long t1 = clock64();
        cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"(256u) : "memory");
    }
}


// The same for CTA pairs: tcgen05.mma.cta_group::2, 256 x n per instruction (128 rows of A
// and n/2 rows of B resident in each CTA), issued by the leader CTA.
__global__ void __launch_bounds__(128, 1)
peak_pair_kernel(int n, int iters, unsigned long long* cycles, unsigned* status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar = sbase + OFF_BAR, slot = sbase + OFF_BAR + 16, abort_flag = sbase + OFF_BAR + 20;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();

    for (uint32_t o = threadIdx.x * 16u; o < (uint32_t)OFF_BAR; o += blockDim.x * 16u)
        sts128(sbase + o, make_uint4(0, 0, 0, 0));
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        sts32(abort_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_async_smem();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(slot), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = (uint32_t)lds32(slot);

    if (warp == 0 && lane == 0 && rank == 0) {
        const uint32_t idesc = (2u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
        const uint64_t adesc = make_kmajor_sw128_desc(sbase + OFF_A);
        const uint64_t bdesc = make_kmajor_sw128_desc(sbase + OFF_B);
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                tc_mma_i8_pair(tmem_base, adesc + (uint64_t)(2 * i), bdesc + (uint64_t)(2 * i), idesc,
                               (it | i) ? 1u : 0u);
        tc_commit_pair(bar, 1);
        mbar_wait(bar, 0, abort_flag, status);
        const long long t1 = clock64();
        cycles[blockIdx.x >> 1] = (unsigned long long)(t1 - t0);
    }
    tc_fence_before();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"(256u) : "memory");
    }
}

}  // namespace peak

unsigned* device_status_ptr();

}  // namespace q4

extern "C" q4_status q4_measure_mma_peak(int kind, int n, int iters, unsigned long long* cycles_dev,
                                         int num_ctas, void* stream)
{
    using namespace q4;
    if (kind == 3) {
        // CTA pairs, kind::i8: num_ctas must be even, n a multiple of 32; cycles_dev gets
        // one entry per pair
        if (n < 32 || n > 256 || (n % 32) || iters < 1 || iters > (1 << 20) || !cycles_dev ||
            num_ctas < 2 || (num_ctas & 1))
            return Q4_ERR_INVALID_ARG;
        unsigned* st = q4::device_status_ptr();
        if (!st) return Q4_ERR_CUDA;
        static bool attr2 = false;
        if (!attr2) {
            if (cudaFuncSetAttribute(q4::peak::peak_pair_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     q4::peak::SMEM) != cudaSuccess) return Q4_ERR_CUDA;
            attr2 = true;
        }
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3((unsigned)num_ctas);
        cfg.blockDim = dim3(128);
        cfg.dynamicSmemBytes = q4::peak::SMEM;
        cfg.stream = static_cast<cudaStream_t>(stream);
        cfg.attrs = at;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, q4::peak::peak_pair_kernel, n, iters, cycles_dev, st);
        q4::count_launch();
        return e == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
    }
    if (kind < 0 || kind > 2 || n < 16 || n > 256 || (n % 16) || iters < 1 || iters > (1 << 20) ||
        !cycles_dev || num_ctas < 1)
        return Q4_ERR_INVALID_ARG;
    unsigned* status = device_status_ptr();
    if (!status) return Q4_ERR_CUDA;
    static bool attr = false;
    if (!attr) {
        if (cudaFuncSetAttribute(peak::peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 peak::SMEM) != cudaSuccess) return Q4_ERR_CUDA;
        attr = true;
    }
    peak::peak_kernel<<<num_ctas, 128, peak::SMEM, static_cast<cudaStream_t>(stream)>>>(
        kind, n, iters, cycles_dev, status);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}
