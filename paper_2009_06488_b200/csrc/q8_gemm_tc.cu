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

// sums[r] = sum of the K bytes of row r, for the rows of A and then those of Bt in one launch:
// a warp per row, 16-byte loads, four of them in flight per lane, bytes past K masked.
__device__ __forceinline__ int masked_chunk_sum(uint4 v, int valid, int s)
{
    if (valid < 16) {
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int vb = valid - 4 * e;              // valid bytes of word e
            if (vb <= 0) w[e] = 0;
            else if (vb < 4) w[e] &= (1u << (8 * vb)) - 1u;
        }
        v = make_uint4(w[0], w[1], w[2], w[3]);
    }
    s = dp4a_u8(v.x, 0x01010101u, s);
    s = dp4a_u8(v.y, 0x01010101u, s);
    s = dp4a_u8(v.z, 0x01010101u, s);
    return dp4a_u8(v.w, 0x01010101u, s);
}

__global__ void __launch_bounds__(256)
byte_sums_kernel(const uint8_t* __restrict__ A, int64_t lda, int32_t rows_a, int32_t* __restrict__ sums_a,
                 const uint8_t* __restrict__ B, int64_t ldb, int32_t rows_b, int32_t* __restrict__ sums_b,
                 int32_t K)
{
    const int lane = threadIdx.x & 31;
    const int chunks = (K + 15) / 16;
    const int64_t total = (int64_t)rows_a + rows_b;
    for (int64_t r = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); r < total;
         r += (int64_t)gridDim.x * (blockDim.x >> 5)) {
        const bool second = r >= rows_a;
        const int64_t rr = second ? r - rows_a : r;
        const uint4* row = reinterpret_cast<const uint4*>(second ? B + rr * ldb : A + rr * lda);
        int s = 0;
        int c = lane;
        for (; c + 96 < chunks; c += 128) {            // four loads in flight
            const uint4 v0 = row[c], v1 = row[c + 32], v2 = row[c + 64], v3 = row[c + 96];
            s = masked_chunk_sum(v0, K - 16 * c, s);
            s = masked_chunk_sum(v1, K - 16 * (c + 32), s);
            s = masked_chunk_sum(v2, K - 16 * (c + 64), s);
            s = masked_chunk_sum(v3, K - 16 * (c + 96), s);
        }
        for (; c < chunks; c += 32) s = masked_chunk_sum(row[c], K - 16 * c, s);
#pragma unroll
        for (int off = 16; off; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        if (lane == 0) (second ? sums_b : sums_a)[rr] = s;
    }
}

}  // namespace u8

// ---------------------------------------------------------------------------------------
// CTA pairs (clusters of two, tcgen05.mma.cta_group::2): 256 x 256 output tiles, each CTA
// staging its own 128 rows of A and its own 128 rows of Bt, so a byte of an operand tile is
// brought from L2 once per pair instead of once per CTA.  Both CTAs' TMA loads report to
// the LEADER's "stage landed" barrier (cta_group::2 loads, no multicast; each CTA also
// announces its byte count there), so the leader's MMA thread waits on one local barrier
// and no relay is needed; its commits arrive on both CTAs' "stage free" and "accumulator
// full" barriers.  The peer's epilogue warps report "accumulator drained" directly to the
// leader.  int32 tiles leave through a swizzled staging tile and TMA stores.
// ---------------------------------------------------------------------------------------
namespace u8p {

constexpr int TMC = 128;             // rows of A per CTA
constexpr int BNC = 256;             // columns of the pair tile
constexpr int BH = BNC / 2;          // rows of Bt staged per CTA
constexpr int ROWB = 128;            // bytes (= depth values) per row per stage
constexpr int STAGES = 6;
constexpr int STAGE = (TMC + BH) * ROWB;          // 32 KB per CTA
constexpr int NTHREADS = 6 * 32;
constexpr int TMEM_COLS = 512;       // two accumulators of 256 columns
constexpr int OFF_STG = STAGES * STAGE;           // int32 epilogue staging: 4 warps x 32 rows x 128 B
constexpr int STG_BYTES = 4 * 32 * 128;
constexpr int OFF_COLTERM = OFF_STG + STG_BYTES;
constexpr int OFF_BAR = OFF_COLTERM + BNC * 4;
constexpr int NBAR = 2 * STAGES + 4;
constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
constexpr int SMEM = OFF_MISC + 16 + 1024;
static_assert(STAGE % 1024 == 0 && OFF_STG % 1024 == 0, "stage and staging alignment");

// D = s32, A = B = unsigned 8-bit, K-major, M = 256 (pair), N = BNC.
constexpr uint32_t kIdesc = (2u << 4) | ((uint32_t)(BNC >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

struct Params {
    GemmParams g;
    int32_t tiles_m, tiles_n, nslab;
    int32_t c_tma;                   // int32 output goes out through TMA stores (tmC is valid)
};

__global__ void __launch_bounds__(NTHREADS, 1)
gemm_u8_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    // the same offset in both CTAs: dynamic shared memory starts at the same address
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t colterm_s = sbase + OFF_COLTERM;  // int32 [BNC]
    const uint32_t bar0 = sbase + OFF_BAR;
    auto bar_full   = [&](int s) { return bar0 + 8u * (uint32_t)s; };                  // used in the leader
    auto bar_empty  = [&](int s) { return bar0 + 8u * (uint32_t)(STAGES + s); };
    auto bar_tfull  = [&](int a) { return bar0 + 8u * (uint32_t)(2 * STAGES + a); };
    auto bar_tempty = [&](int a) { return bar0 + 8u * (uint32_t)(2 * STAGES + 2 + a); };  // used in the leader
    const uint32_t tmem_slot = sbase + OFF_MISC;
    const uint32_t abort_flag = sbase + OFF_MISC + 4;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;
    const GemmParams& g = p.g;
    const int ntiles = p.tiles_m * p.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full(s), 2);       // one announcement per CTA's producer
            mbar_init(bar_empty(s), 1);      // the leader's commit
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);
            mbar_init(bar_tempty(a), 8);     // four epilogue warps of each CTA
        }
        sts32(abort_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(tmem_slot), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();              // barriers of both CTAs are initialised past this point
    tc_fence_after();
    const uint32_t tmem_base = (uint32_t)lds32(tmem_slot);

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t full_leader = map_to_cta(bar_full(0), 0);
            uint32_t it = 0;
            for (int tile = cluster_id; tile < ntiles; tile += nclusters) {
                const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
                const int arow = tm * 256 + (int)rank * TMC;
                const int brow = tn * BNC + (int)rank * BH;
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    mbar_wait(bar_empty(st), ph ^ 1u, abort_flag, g.status);
                    const uint32_t full = full_leader + 8u * (uint32_t)st;
                    mbar_expect_tx_cluster(full, (uint32_t)STAGE);
                    const uint32_t dst = sbase + st * STAGE;
                    tma_load_2d_pair(dst, &tmA, s * ROWB, arow, full);
                    tma_load_2d_pair(dst + TMC * ROWB, &tmB, s * ROWB, brow, full);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ pair MMA issuer (leader)
        if (rank == 0 && lane == 0) {
            uint32_t it = 0, lt = 0;
            for (int tile = cluster_id; tile < ntiles; tile += nclusters, ++lt) {
                const int acc = lt & 1;
                const uint32_t aph = (lt >> 1) & 1u;
                mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BNC);
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    mbar_wait(bar_full(st), ph, abort_flag, g.status);
                    tc_fence_after();
                    const uint32_t ua = sbase + st * STAGE;
                    const uint64_t adesc = make_kmajor_sw128_desc(ua);
                    const uint64_t bdesc = make_kmajor_sw128_desc(ua + TMC * ROWB);
                    const int rem = g.K - s * ROWB;
                    const int ksteps = rem >= ROWB ? 4 : (rem + 31) / 32;
                    for (int i = 0; i < ksteps; ++i)
                        tc_mma_i8_pair(d_tmem, adesc + (uint64_t)(2 * i), bdesc + (uint64_t)(2 * i), kIdesc,
                                       (s > 0 || i > 0) ? 1u : 0u);
                    tc_commit_pair(bar_empty(st), 3);
                }
                tc_commit_pair(bar_tfull(acc), 3);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const int et = threadIdx.x - 64;
        const int kzz = g.K * g.za * g.zb;
        const uint32_t tempty_leader = map_to_cta(bar_tempty(0), 0);
        uint32_t lt = 0;
        for (int tile = cluster_id; tile < ntiles; tile += nclusters, ++lt) {
            const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
            const int acc = lt & 1;
            const uint32_t aph = (lt >> 1) & 1u;
            const int m = tm * 256 + (int)rank * TMC + row;
            const int n0 = tn * BNC;
            for (int j = et; j < BNC; j += 128) {
                const int n = n0 + j;
                const int cb = n < g.N ? g.colsum_b[n] : 0;
                sts32(colterm_s + 4 * j, (int)((uint32_t)kzz - (uint32_t)(g.za * cb)));
            }
            const int ra = m < g.M ? g.rowsum_a[m] : 0;
            const uint32_t rowterm = (uint32_t)0 - (uint32_t)(g.zb * ra);
            asm volatile("bar.sync 1, 128;" ::: "memory");

            mbar_wait(bar_tfull(acc), aph, abort_flag, g.status);
            tc_fence_after();
            const uint32_t taddr0 = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(acc * BNC);
#pragma unroll 1
            for (int ch = 0; ch < BNC / 32; ++ch) {
                const int nc = n0 + ch * 32;
                if (nc >= g.N) break;             // warp-uniform
                uint32_t r[32];
                tc_ld32(taddr0 + (uint32_t)(ch * 32), r);
                tc_wait_ld();
#pragma unroll
                for (int qd = 0; qd < 8; ++qd) {
                    const uint4 ct = lds128(colterm_s + 4 * (ch * 32 + 4 * qd));
                    r[4 * qd + 0] += rowterm + ct.x;
                    r[4 * qd + 1] += rowterm + ct.y;
                    r[4 * qd + 2] += rowterm + ct.z;
                    r[4 * qd + 3] += rowterm + ct.w;
                }
                if (p.c_tma) {
                    // my row's 128 bytes go to the swizzled staging slice of my warp; rows and
                    // columns past M / N are clipped by the tensor map
                    const uint32_t slice = sbase + OFF_STG + (uint32_t)(lg * 4096);
                    if (lane == 0) bulk_wait_read();       // the previous store has read the slice
                    __syncwarp();
#pragma unroll
                    for (int qd = 0; qd < 8; ++qd)
                        sts128(slice + (uint32_t)(lane * 128 + ((qd ^ (lane & 7)) << 4)),
                               make_uint4(r[4 * qd], r[4 * qd + 1], r[4 * qd + 2], r[4 * qd + 3]));
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmC, slice, nc, tm * 256 + (int)rank * TMC + lg * 32);
                        bulk_commit();
                    }
                } else if (m < g.M) {
                    int32_t* dst = g.C + (int64_t)m * g.ldc + nc;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (nc + j < g.N) dst[j] = (int32_t)r[j];
                }
            }
            tc_fence_before();
            __syncwarp();                          // every lane's tensor-memory loads are done
            if (lane == 0) mbar_arrive_cluster(tempty_leader + 8u * (uint32_t)acc);
            asm volatile("bar.sync 1, 128;" ::: "memory");   // colterm_s is rewritten next tile
        }
        if (p.c_tma && lane == 0) bulk_wait_read();  // my TMA stores have read their slices; their writes complete with the grid
    }

    tc_fence_before();
    cluster_sync_all();          // no CTA leaves (or frees TMEM) while its peer may still use it
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

}  // namespace u8p

static int sm_count_u8()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        n = 148;
    return n;
}

cudaError_t launch_byte_sums(const uint8_t* A, int64_t lda, int32_t rows_a, int32_t* sums_a,
                             const uint8_t* B, int64_t ldb, int32_t rows_b, int32_t* sums_b, int32_t K,
                             cudaStream_t st)
{
    const int64_t rows = (int64_t)rows_a + rows_b;
    if (rows == 0) return cudaSuccess;
    int64_t blocks = (rows + 7) / 8;
    if (blocks > 148 * 8) blocks = 148 * 8;
    u8::byte_sums_kernel<<<(int)blocks, 256, 0, st>>>(A, lda, rows_a, sums_a, B, ldb, rows_b, sums_b, K);
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

bool make_c32_map(CUtensorMap* tm, int32_t* base, int64_t ldc, int rows, int cols);

static q4_status launch_u8_pair(const GemmParams& g, cudaStream_t st)
{
    u8p::Params p;
    p.g = g;
    p.tiles_m = (g.M + 255) / 256;
    p.tiles_n = (g.N + u8p::BNC - 1) / u8p::BNC;
    p.nslab = (g.K + u8p::ROWB - 1) / u8p::ROWB;
    CUtensorMap tmA, tmB, tmC{};
    if (!make_byte_map(&tmA, g.A, g.lda, g.M, g.K, u8p::TMC)) return Q4_ERR_CUDA;
    if (!make_byte_map(&tmB, g.Bt, g.ldb, g.N, g.K, u8p::BH)) return Q4_ERR_CUDA;
    p.c_tma = 0;
    if ((uintptr_t)g.C % 16 == 0 && g.ldc % 4 == 0) {
        if (!make_c32_map(&tmC, g.C, g.ldc, g.M, g.N)) return Q4_ERR_CUDA;
        p.c_tma = 1;
    }
    if (cudaFuncSetAttribute(u8p::gemm_u8_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             u8p::SMEM) != cudaSuccess)
        return Q4_ERR_CUDA;
    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    const int max_clusters = sm_count_u8() / 2;
    const long long clusters = tiles < max_clusters ? tiles : max_clusters;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    cfg.blockDim = dim3(u8p::NTHREADS);
    cfg.dynamicSmemBytes = u8p::SMEM;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, u8p::gemm_u8_pair_kernel, tmA, tmB, tmC, p);
    count_launch();
    return e == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status launch_gemm_u8(const GemmParams& g, cudaStream_t st)
{
    // large problems: CTA pairs on 256 x 256 tiles (at least one tile per pair of SMs)
    if (g.M >= 256 && g.N >= 256 &&
        (long long)((g.M + 255) / 256) * ((g.N + 255) / 256) >= sm_count_u8() / 2) {
        log_choice("q4_gemm_u8", "CTA-pair tcgen05 kernel");
        return launch_u8_pair(g, st);
    }
    log_choice("q4_gemm_u8", "single-CTA tcgen05 kernel");
    if (g.N > 128) return launch_u8_bn<256>(g, st);
    if (g.N > 64)  return launch_u8_bn<128>(g, st);
    return launch_u8_bn<64>(g, st);
}

}  // namespace q4
