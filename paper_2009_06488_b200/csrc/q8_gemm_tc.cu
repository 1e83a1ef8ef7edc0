// 8-bit quantized GEMM for sm_100a: the comparison system of the paper's experiments
// (Section II-B: 8-bit values in 0..255, 32-bit accumulators; Section IV: the 4-bit product
// is measured against it).  Same Eq. 2, same four terms, but the operands are already one
// byte per value, so the tiles that TMA brings in are what the tensor core reads: there is
// no unpack stage.
//
//   warp 0        TMA producer   128 x 128-byte tile of A and BN x 128-byte tile of Bt per
//                                stage, 128-byte swizzle (the K-major layout the MMA reads)
//   warp 1        MMA issuer     tcgen05.mma kind::i8 (u8 x u8 -> s32), 128 x BN x 32 per
//                                instruction, two accumulators in tensor memory
//   warps 2..5    epilogue       tcgen05.ld, zero-point correction of Eq. 2, int32 stores
//
// The depth sums of Eq. 2's second and third terms come from the caller or from a
// bandwidth-bound pre-pass (byte_sums_kernel).  Every mbarrier wait is bounded.
#include <cuda.h>

#include "q4_common.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {

bool make_byte_map(CUtensorMap* tm, const uint8_t* base, int64_t ld, int rows, int kbytes, int box_rows);

namespace u8 {

constexpr int TM = 128;            // rows of A per tile (UMMA M)
constexpr int ROWB = 128;          // bytes (= depth values) per row per stage: one swizzle row
constexpr int NTHREADS = 6 * 32;

// Instruction descriptor: D = s32, A = B = unsigned 8-bit, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t idesc_u8(int n)
{
    return (2u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}

template <int BN> struct Cfg {
    static constexpr int STAGE = (TM + BN) * ROWB;
    static constexpr int STAGES = (BN == 256) ? 4 : 6;
    static constexpr int TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;
    static constexpr int OFF_COLTERM = STAGES * STAGE;
    static constexpr int OFF_BAR = OFF_COLTERM + BN * 4;
    static constexpr int NBAR = 2 * STAGES + 4;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
    static constexpr int SMEM = OFF_MISC + 16 + 1024;          // + slack to align the base
};

struct Params {
    GemmParams g;                  // A, Bt: one byte per value; rowsum_a, colsum_b always set
    int32_t tiles_m, tiles_n, nslab;
    int32_t c_vec;                 // int32 rows may be stored with 16-byte vectors
};

template <int BN>
__global__ void __launch_bounds__(NTHREADS, 1)
gemm_u8_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const Params p)
{
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t colterm_s = sbase + C::OFF_COLTERM;    // int32 [BN]
    const uint32_t bar0 = sbase + C::OFF_BAR;
    auto bar_full   = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto bar_empty  = [&](int s) { return bar0 + 8u * (uint32_t)(C::STAGES + s); };
    auto bar_tfull  = [&](int a) { return bar0 + 8u * (uint32_t)(2 * C::STAGES + a); };
    auto bar_tempty = [&](int a) { return bar0 + 8u * (uint32_t)(2 * C::STAGES + 2 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_MISC);
    const uint32_t abort_flag = sbase + C::OFF_MISC + 4;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const GemmParams& g = p.g;
    const int ntiles = p.tiles_m * p.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);
            mbar_init(bar_tempty(a), 128);
        }
        sts32(abort_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)C::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
                const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    mbar_wait(bar_empty(st), ph ^ 1u, abort_flag, g.status);
                    mbar_expect_tx(bar_full(st), (uint32_t)C::STAGE);
                    const uint32_t dst = sbase + st * C::STAGE;
                    tma_load_2d(dst, &tmA, s * ROWB, tm * TM, bar_full(st));
                    tma_load_2d(dst + TM * ROWB, &tmB, s * ROWB, tn * BN, bar_full(st));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_u8(BN);
            uint32_t it = 0, lt = 0;
            for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++lt) {
                const int acc = lt & 1;
                const uint32_t aph = (lt >> 1) & 1u;
                mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    mbar_wait(bar_full(st), ph, abort_flag, g.status);
                    tc_fence_after();
                    const uint32_t ua = sbase + st * C::STAGE;
                    const uint64_t adesc = make_kmajor_sw128_desc(ua);
                    const uint64_t bdesc = make_kmajor_sw128_desc(ua + TM * ROWB);
                    const int rem = g.K - s * ROWB;
                    const int ksteps = rem >= ROWB ? 4 : (rem + 31) / 32;
                    for (int i = 0; i < ksteps; ++i)
                        tc_mma_i8(d_tmem, adesc + (uint64_t)(2 * i), bdesc + (uint64_t)(2 * i), idesc,
                                  (s > 0 || i > 0) ? 1u : 0u);
                    tc_commit(bar_empty(st));
                }
                tc_commit(bar_tfull(acc));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int lg = warp & 3;                 // TMEM lane group this warp may read
        const int row = lg * 32 + lane;          // row of the tile held by this thread
        const int et = threadIdx.x - 64;         // 0..127
        const int kzz = g.K * g.za * g.zb;
        uint32_t lt = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++lt) {
            const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
            const int acc = lt & 1;
            const uint32_t aph = (lt >> 1) & 1u;
            const int m = tm * TM + row;
            const int n0 = tn * BN;
            // per-column term of Eq. 2: -za * colsum + K za zb
            for (int j = et; j < BN; j += 128) {
                const int n = n0 + j;
                const int cb = n < g.N ? g.colsum_b[n] : 0;
                sts32(colterm_s + 4 * j, (int)((uint32_t)kzz - (uint32_t)(g.za * cb)));
            }
            const int ra = m < g.M ? g.rowsum_a[m] : 0;
            const uint32_t rowterm = (uint32_t)0 - (uint32_t)(g.zb * ra);
            asm volatile("bar.sync 1, 128;" ::: "memory");

            mbar_wait(bar_tfull(acc), aph, abort_flag, g.status);
            tc_fence_after();
            const uint32_t taddr0 = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
            for (int ch = 0; ch < BN / 32; ++ch) {
                const int nc = n0 + ch * 32;
                if (nc >= g.N) break;             // warp-uniform
                uint32_t r[32];
                tc_ld32(taddr0 + (uint32_t)(ch * 32), r);
                tc_wait_ld();
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const uint4 ct = lds128(colterm_s + 4 * (ch * 32 + 4 * q));
                    r[4 * q + 0] += rowterm + ct.x;
                    r[4 * q + 1] += rowterm + ct.y;
                    r[4 * q + 2] += rowterm + ct.z;
                    r[4 * q + 3] += rowterm + ct.w;
                }
                if (m < g.M) {
                    int32_t* dst = g.C + (int64_t)m * g.ldc + nc;
                    if (nc + 32 <= g.N && p.c_vec) {
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            *reinterpret_cast<uint4*>(dst + 4 * q) =
                                make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nc + j < g.N) dst[j] = (int32_t)r[j];
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar_tempty(acc));
            asm volatile("bar.sync 1, 128;" ::: "memory");   // colterm_s is rewritten next tile
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
    }
}

// sums[r] = sum of the K bytes of row r: a warp per row, 16-byte loads, bytes past K masked.
__global__ void __launch_bounds__(256)
byte_sums_kernel(const uint8_t* __restrict__ P, int64_t ld, int32_t rows, int32_t K, int32_t* __restrict__ sums)
{
    const int lane = threadIdx.x & 31;
    const int chunks = (K + 15) / 16;
    for (int64_t r = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); r < rows;
         r += (int64_t)gridDim.x * (blockDim.x >> 5)) {
        const uint4* row = reinterpret_cast<const uint4*>(P + r * ld);
        int s = 0;
        for (int c = lane; c < chunks; c += 32) {
            uint4 v = row[c];
            const int valid = K - 16 * c;              // bytes of this chunk inside the row
            if (valid < 16) {
                uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int vb = valid - 4 * e;      // valid bytes of word e
                    if (vb <= 0) w[e] = 0;
                    else if (vb < 4) w[e] &= (1u << (8 * vb)) - 1u;
                }
                v = make_uint4(w[0], w[1], w[2], w[3]);
            }
            s = dp4a_u8(v.x, 0x01010101u, s);
            s = dp4a_u8(v.y, 0x01010101u, s);
            s = dp4a_u8(v.z, 0x01010101u, s);
            s = dp4a_u8(v.w, 0x01010101u, s);
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        if (lane == 0) sums[r] = s;
    }
}

}  // namespace u8

static int sm_count_u8()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        n = 148;
    return n;
}

cudaError_t launch_byte_sums(const uint8_t* P, int64_t ld, int32_t rows, int32_t K, int32_t* sums,
                             cudaStream_t st)
{
    if (rows == 0) return cudaSuccess;
    int blocks = (rows + 7) / 8;
    if (blocks > 148 * 8) blocks = 148 * 8;
    u8::byte_sums_kernel<<<blocks, 256, 0, st>>>(P, ld, rows, K, sums);
    count_launch();
    return cudaGetLastError();
}

template <int BN>
static q4_status launch_u8_bn(const GemmParams& g, cudaStream_t st)
{
    using C = u8::Cfg<BN>;
    u8::Params p;
    p.g = g;
    p.tiles_m = (g.M + u8::TM - 1) / u8::TM;
    p.tiles_n = (g.N + BN - 1) / BN;
    p.nslab = (g.K + u8::ROWB - 1) / u8::ROWB;
    p.c_vec = (((uintptr_t)g.C % 16 == 0) && (g.ldc % 4 == 0)) ? 1 : 0;

    CUtensorMap tmA, tmB;
    if (!make_byte_map(&tmA, g.A, g.lda, g.M, g.K, u8::TM)) return Q4_ERR_CUDA;
    if (!make_byte_map(&tmB, g.Bt, g.ldb, g.N, g.K, BN)) return Q4_ERR_CUDA;

    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    const int sms = sm_count_u8();
    const int grid = (int)(tiles < sms ? tiles : sms);
    if (cudaFuncSetAttribute(u8::gemm_u8_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM) != cudaSuccess)
        return Q4_ERR_CUDA;
    u8::gemm_u8_kernel<BN><<<grid, u8::NTHREADS, C::SMEM, st>>>(tmA, tmB, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status launch_gemm_u8(const GemmParams& g, cudaStream_t st)
{
    if (g.N > 128) return launch_u8_bn<256>(g, st);
    if (g.N > 64)  return launch_u8_bn<128>(g, st);
    return launch_u8_bn<64>(g, st);
}

}  // namespace q4
