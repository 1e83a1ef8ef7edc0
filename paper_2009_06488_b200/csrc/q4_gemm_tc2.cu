// Tensor-core 4-bit quantized GEMM for large problems: CTA pairs (thread-block clusters
// of two) computing 256 x 256 output tiles with tcgen05.mma.cta_group::2 (Eq. 2 of the
// paper, all four terms).
//
// Each CTA of a pair owns 128 rows of A and 128 of the tile's 256 rows of Bt; the pair
// MMA reads A from both CTAs and shares the two halves of Bt between them, so every
// CTA stages and unpacks only half of the Bt tile -- the step that bounds the
// single-CTA kernel (the unpack is a shared-memory-bandwidth problem).  The
// accumulator (256 x 256 int32) lives in the two CTAs' tensor memory, 128 rows each,
// double-buffered, so each CTA's epilogue of tile t overlaps the main loop of t+1.
//
// Roles per CTA (14 warps): warp 0 TMA producer (its own rows of A and Bt, no
// multicast); warps 2..9 unpack nibbles to bytes in the K-major 128-byte-swizzled
// layout and take the depth sums; warp 1 of the leader CTA issues the pair MMAs and
// commits to the barriers of both CTAs; warp 1 of the peer CTA relays "my operands are
// ready" / "my accumulator is drained" to the leader with one remote arrive each;
// warps 10..13 epilogue.  Column sums of the two Bt halves are exchanged through
// distributed shared memory.
//
// Every mbarrier wait is bounded (see q4_tc_ptx.cuh); the only unbounded waits are the
// two cluster barriers at entry and exit, which every thread reaches unconditionally.
#include <cuda.h>

#include "q4_common.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {
namespace pair {

constexpr int TMC = 128;             // rows of A per CTA
constexpr int BNC = 256;             // columns of the pair tile
constexpr int BH = BNC / 2;          // rows of Bt staged per CTA
constexpr int ROWS = TMC + BH;       // rows unpacked per CTA per stage
constexpr int PROW = 64, UROW = 128, SLAB = 128;
constexpr int PSTAGE = ROWS * PROW;  // 16 KB
constexpr int USTAGE = ROWS * UROW;  // 32 KB
constexpr int STAGES = 4;
constexpr int UW = 8, UT = UW * 32;
constexpr int NT = ROWS * 4 / UT;    // unpack tasks per thread per stage
constexpr int NTHREADS = (2 + UW + 4) * 32;
constexpr int TMEM_COLS = 512;
constexpr int SUMS_N = TMC + BNC;    // per buffer: 128 row sums, 256 column sums

constexpr int OFF_U = 0;
constexpr int OFF_P = OFF_U + STAGES * USTAGE;
constexpr int OFF_SUMS = OFF_P + STAGES * PSTAGE;
constexpr int OFF_COLTERM = OFF_SUMS + 2 * SUMS_N * 4;
constexpr int OFF_BAR = OFF_COLTERM + BNC * 4;
constexpr int NBAR = 5 * STAGES + 10;
constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
constexpr int SMEM = OFF_MISC + 16 + 1024;

static_assert(ROWS * 4 % UT == 0, "unpack tasks must divide evenly");

// D = s32, A = B = unsigned 8-bit, K-major, M = 256 (pair), N = 256.
constexpr uint32_t kIdesc = (2u << 4) | ((uint32_t)(BNC >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

struct Params {
    GemmParams g;
    int32_t tiles_m, tiles_n, nslab;
    int32_t c_vec, cq_vec;
};

template <bool REQUANT>
__global__ void __launch_bounds__(NTHREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    // the same offset in both CTAs: dynamic shared memory starts at the same address
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;

    const uint32_t sums_s = sbase + OFF_SUMS;        // int32 [2][SUMS_N]
    const uint32_t colterm_s = sbase + OFF_COLTERM;  // int32 [BNC]
    const uint32_t bar0 = sbase + OFF_BAR;
    auto bar_full_p    = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto bar_empty_p   = [&](int s) { return bar0 + 8u * (uint32_t)(STAGES + s); };
    auto bar_full_u    = [&](int s) { return bar0 + 8u * (uint32_t)(2 * STAGES + s); };
    auto bar_empty_u   = [&](int s) { return bar0 + 8u * (uint32_t)(3 * STAGES + s); };
    auto bar_peer_full = [&](int s) { return bar0 + 8u * (uint32_t)(4 * STAGES + s); };
    auto bar_tfull     = [&](int a) { return bar0 + 8u * (uint32_t)(5 * STAGES + a); };
    auto bar_tempty    = [&](int a) { return bar0 + 8u * (uint32_t)(5 * STAGES + 2 + a); };
    auto bar_peer_tempty = [&](int a) { return bar0 + 8u * (uint32_t)(5 * STAGES + 4 + a); };
    auto bar_sums      = [&](int a) { return bar0 + 8u * (uint32_t)(5 * STAGES + 6 + a); };
    auto bar_tstart    = [&](int a) { return bar0 + 8u * (uint32_t)(5 * STAGES + 8 + a); };
    const uint32_t tmem_slot = sbase + OFF_MISC;
    const uint32_t abort_flag = sbase + OFF_MISC + 4;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t peer = rank ^ 1u;
    const int cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;
    const GemmParams& g = p.g;
    const bool need_ra = (g.rowsum_a == nullptr);
    const bool need_cb = (g.colsum_b == nullptr);
    const bool need_sums = need_ra || need_cb;
    const int ntiles = p.tiles_m * p.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full_p(s), 1);
            mbar_init(bar_empty_p(s), UW);   // one arrive per unpack warp
            mbar_init(bar_full_u(s), UW);
            mbar_init(bar_empty_u(s), 1);
            mbar_init(bar_peer_full(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);
            mbar_init(bar_tempty(a), 128);
            mbar_init(bar_peer_tempty(a), 1);
            mbar_init(bar_sums(a), 2 * UW);       // one arrive per unpack warp of each CTA
            mbar_init(bar_tstart(a), 1);
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
            uint32_t it = 0;
            for (int tile = cluster_id; tile < ntiles; tile += nclusters) {
                const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
                const int arow = tm * 256 + (int)rank * TMC;
                const int brow = tn * BNC + (int)rank * BH;
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    mbar_wait_cl(bar_empty_p(st), ph ^ 1u, abort_flag, g.status);
                    mbar_expect_tx(bar_full_p(st), (uint32_t)PSTAGE);
                    const uint32_t dst = sbase + OFF_P + st * PSTAGE;
                    tma_load_2d(dst, &tmA, s * PROW, arow, bar_full_p(st));
                    tma_load_2d(dst + TMC * PROW, &tmB, s * PROW, brow, bar_full_p(st));
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------- pair MMA issuer
            uint32_t it = 0, lt = 0;
            for (int tile = cluster_id; tile < ntiles; tile += nclusters, ++lt) {
                const int acc = lt & 1;
                const uint32_t aph = (lt >> 1) & 1u;
                mbar_wait_cl(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
                if (lt >= 2) mbar_wait_cl(bar_peer_tempty(acc), aph ^ 1u, abort_flag, g.status);
                tc_fence_after();
                // both epilogues are done with buffer `acc`: tell the unpack warps of both CTAs
                tc_commit_pair(bar_tstart(acc), 3);
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BNC);
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    mbar_wait_cl(bar_full_u(st), ph, abort_flag, g.status);
                    mbar_wait_cl(bar_peer_full(st), ph, abort_flag, g.status);
                    tc_fence_after();
                    const uint32_t ua = sbase + OFF_U + st * USTAGE;
                    const uint64_t adesc = make_kmajor_sw128_desc(ua);
                    const uint64_t bdesc = make_kmajor_sw128_desc(ua + TMC * UROW);
                    const int rem = g.K - s * SLAB;
                    const int ksteps = rem >= SLAB ? 4 : (rem + 31) / 32;
                    for (int i = 0; i < ksteps; ++i)
                        tc_mma_i8_pair(d_tmem, adesc + (uint64_t)(2 * i), bdesc + (uint64_t)(2 * i),
                                       kIdesc, (s > 0 || i > 0) ? 1u : 0u);
                    tc_commit_pair(bar_empty_u(st), 3);
                }
                tc_commit_pair(bar_tfull(acc), 3);
            }
        } else if (lane == 0) {
            // -------------------------------------------------------- peer relay
            uint32_t it = 0, lt = 0;
            for (int tile = cluster_id; tile < ntiles; tile += nclusters, ++lt) {
                const int acc = lt & 1;
                const uint32_t aph = (lt >> 1) & 1u;
                if (lt >= 2) {
                    mbar_wait_cl(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
                    mbar_arrive_cluster(map_to_cta(bar_peer_tempty(acc), 0));
                }
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    mbar_wait_cl(bar_full_u(st), ph, abort_flag, g.status);
                    mbar_arrive_cluster(map_to_cta(bar_peer_full(st), 0));
                }
            }
        }
    } else if (warp < 2 + UW) {
        // ------------------------------------------------------------ unpack warps
        const int ut = threadIdx.x - 64;
        uint32_t it = 0, lt = 0;
        for (int tile = cluster_id; tile < ntiles; tile += nclusters, ++lt) {
            int psum[NT];
#pragma unroll
            for (int j = 0; j < NT; ++j) psum[j] = 0;
            for (int s = 0; s < p.nslab; ++s, ++it) {
                const int st = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1u;
                const int rem = g.K - s * SLAB;
                const int ksteps = rem >= SLAB ? 4 : (rem + 31) / 32;
                mbar_wait_cl(bar_full_p(st), ph, abort_flag, g.status);
                mbar_wait_cl(bar_empty_u(st), ph ^ 1u, abort_flag, g.status);
                tc_fence_after();
                const uint32_t ps = sbase + OFF_P + st * PSTAGE;
                const uint32_t us = sbase + OFF_U + st * USTAGE;
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const int id = ut + j * UT;
                    const int r = id >> 2, c = id & 3;
                    if (c < ksteps) {
                        const uint4 w = lds128(ps + r * PROW + c * 16);
                        uint4 lo, hi;
                        lo.x = w.x & 0x0F0F0F0Fu; hi.x = (w.x >> 4) & 0x0F0F0F0Fu;
                        lo.y = w.y & 0x0F0F0F0Fu; hi.y = (w.y >> 4) & 0x0F0F0F0Fu;
                        lo.z = w.z & 0x0F0F0F0Fu; hi.z = (w.z >> 4) & 0x0F0F0F0Fu;
                        lo.w = w.w & 0x0F0F0F0Fu; hi.w = (w.w >> 4) & 0x0F0F0F0Fu;
                        const uint32_t row = us + r * UROW;
                        const int sw = r & 7;
                        sts128(row + (((2 * c) ^ sw) << 4), lo);
                        sts128(row + (((2 * c + 1) ^ sw) << 4), hi);
                        if (need_sums) {
                            int t = psum[j];
                            t = dp4a_u8(lo.x + hi.x, 0x01010101u, t);
                            t = dp4a_u8(lo.y + hi.y, 0x01010101u, t);
                            t = dp4a_u8(lo.z + hi.z, 0x01010101u, t);
                            t = dp4a_u8(lo.w + hi.w, 0x01010101u, t);
                            psum[j] = t;
                        }
                    }
                }
                // every lane publishes its own writes to the async proxy; one lane per warp
                // then arrives (256 arrives on one barrier word serialise badly)
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar_full_u(st));
                    mbar_arrive(bar_empty_p(st));
                }
            }
            if (need_sums) {
                const int acc = lt & 1;
                const uint32_t aph = (lt >> 1) & 1u;
                // both CTAs' epilogues two tiles back are done with this sums buffer
                mbar_wait_cl(bar_tstart(acc), aph, abort_flag, g.status);
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    int t = psum[j];
                    t += __shfl_xor_sync(0xFFFFFFFFu, t, 1);
                    t += __shfl_xor_sync(0xFFFFFFFFu, t, 2);
                    const int id = ut + j * UT;
                    if ((id & 3) == 0) {
                        const int r = id >> 2;
                        if (r < TMC) {
                            sts32(sums_s + 4 * (acc * SUMS_N + r), t);         // row sum: local
                        } else {
                            // column sum of my half of Bt: both CTAs need it
                            const uint32_t a = sums_s + 4 * (acc * SUMS_N + TMC + (int)rank * BH + (r - TMC));
                            sts32(a, t);
                            sts32_cluster(map_to_cta(a, peer), t);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive_cluster(map_to_cta(bar_sums(acc), rank));
                    mbar_arrive_cluster(map_to_cta(bar_sums(acc), peer));
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const int et = threadIdx.x - (2 + UW) * 32;
        const int kzz = g.K * g.za * g.zb;
        uint32_t lt = 0;
        for (int tile = cluster_id; tile < ntiles; tile += nclusters, ++lt) {
            const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
            const int acc = lt & 1;
            const uint32_t aph = (lt >> 1) & 1u;
            const int m = tm * 256 + (int)rank * TMC + row;
            const int n0 = tn * BNC;
            if (need_sums) mbar_wait_cl(bar_sums(acc), aph, abort_flag, g.status);
            for (int j = et; j < BNC; j += 128) {
                const int n = n0 + j;
                int cb = 0, bias = 0;
                if (n < g.N) {
                    cb = need_cb ? lds32(sums_s + 4 * (acc * SUMS_N + TMC + j)) : g.colsum_b[n];
                    if (REQUANT && g.bias) bias = g.bias[n];
                }
                sts32(colterm_s + 4 * j, (int)((uint32_t)kzz - (uint32_t)(g.za * cb) + (uint32_t)bias));
            }
            int ra = 0;
            if (need_ra) ra = lds32(sums_s + 4 * (acc * SUMS_N + row));
            else if (m < g.M) ra = g.rowsum_a[m];
            const uint32_t rowterm = (uint32_t)0 - (uint32_t)(g.zb * ra);
            asm volatile("bar.sync 1, 128;" ::: "memory");

            mbar_wait_cl(bar_tfull(acc), aph, abort_flag, g.status);
            tc_fence_after();
            const uint32_t taddr0 = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(acc * BNC);
#pragma unroll 1
            for (int ch = 0; ch < BNC / 32; ++ch) {
                const int nc = n0 + ch * 32;
                if (nc >= g.N) break;
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
                    const bool full = (nc + 32 <= g.N);
                    if (!REQUANT) {
                        int32_t* dst = g.C + (int64_t)m * g.ldc + nc;
                        if (full && p.c_vec) {
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                *reinterpret_cast<uint4*>(dst + 4 * q) =
                                    make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (nc + j < g.N) dst[j] = (int32_t)r[j];
                        }
                    } else {
                        uint32_t o[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint32_t wv = 0;
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                wv |= requant((int32_t)r[8 * q + e], g.rq) << (4 * e);
                            o[q] = wv;
                        }
                        uint8_t* dst = g.Cq + (int64_t)m * g.ldcq + (nc >> 1);
                        if (full && p.cq_vec) {
                            *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
                        } else {
#pragma unroll
                            for (int b = 0; b < 16; ++b)
                                if (nc + 2 * b < g.N) dst[b] = (uint8_t)(o[b >> 2] >> (8 * (b & 3)));
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar_tempty(acc));
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
    }

    tc_fence_before();
    cluster_sync_all();          // no CTA leaves (or frees TMEM) while its peer may still use it
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

}  // namespace pair

// ---- host side ------------------------------------------------------------------------
bool make_packed_map(CUtensorMap* tm, const uint8_t* base, int64_t ld, int rows, int kbytes,
                     int box_rows);

bool gemm_tc_pair_supported(const GemmParams& p)
{
    return gemm_tc_supported(p) && p.M >= 256 && p.N >= 256;
}

template <bool RQ>
static q4_status launch_pair_t(const pair::Params& p, const CUtensorMap& tmA, const CUtensorMap& tmB,
                               long long tiles, cudaStream_t st)
{
    static int max_clusters = 0;
    auto kernel = pair::gemm_tc_pair_kernel<RQ>;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(pair::NTHREADS);
    cfg.dynamicSmemBytes = pair::SMEM;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (!max_clusters) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, pair::SMEM) !=
            cudaSuccess) return Q4_ERR_CUDA;
        int dev = 0, sms = 148, n = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cfg.gridDim = dim3((unsigned)(sms / 2 * 2));
        if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = sms / 2;
        }
        max_clusters = n < sms / 2 ? n : sms / 2;
    }
    const long long clusters = tiles < max_clusters ? tiles : max_clusters;
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, p);
    count_launch();
    return e == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status launch_gemm_tc_pair(const GemmParams& g, bool rq, cudaStream_t st)
{
    pair::Params p;
    p.g = g;
    p.tiles_m = (g.M + 255) / 256;
    p.tiles_n = (g.N + pair::BNC - 1) / pair::BNC;
    const int kbytes = (g.K + 1) / 2;
    p.nslab = (kbytes + pair::PROW - 1) / pair::PROW;
    p.c_vec = (!rq && ((uintptr_t)g.C % 16 == 0) && (g.ldc % 4 == 0)) ? 1 : 0;
    p.cq_vec = (rq && ((uintptr_t)g.Cq % 16 == 0) && (g.ldcq % 16 == 0)) ? 1 : 0;
    CUtensorMap tmA, tmB;
    if (!make_packed_map(&tmA, g.A, g.lda, g.M, kbytes, pair::TMC)) return Q4_ERR_CUDA;
    if (!make_packed_map(&tmB, g.Bt, g.ldb, g.N, kbytes, pair::BH)) return Q4_ERR_CUDA;
    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    return rq ? launch_pair_t<true>(p, tmA, tmB, tiles, st) : launch_pair_t<false>(p, tmA, tmB, tiles, st);
}

}  // namespace q4
