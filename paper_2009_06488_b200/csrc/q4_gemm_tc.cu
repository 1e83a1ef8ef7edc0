// Tensor-core 4-bit quantized GEMM for sm_100a (Eq. 2 of the paper, all four terms).
//
// One persistent, warp-specialised kernel:
//
//   warp 0      TMA producer   packed-nibble tiles of A (128 rows) and Bt (BN rows),
//                              64 bytes = 128 depth values per row per stage
//   warps 2..   unpack         nibbles -> one byte per value, written in the K-major
//                              128-byte-swizzled layout the MMA reads; the depth sums
//                              of Eq. 2's second and third terms ride along (dp4a)
//   warp 1      MMA issuer     tcgen05.mma kind::i8 (u8 x u8 -> s32), 128 x BN x 32
//                              per instruction, accumulators in tensor memory
//                              (two buffers, so the epilogue of tile t overlaps the
//                              main loop of tile t+1)
//   last 4 warps epilogue      tcgen05.ld, zero-point correction, then either the
//                              int32 store or bias + re-quantization + nibble packing
//
// The sum over the depth commutes, so the unpack stores the even nibbles of each
// 16-byte packed chunk as one 16-byte group and the odd nibbles as the next one
// (three integer ops per eight values, no byte shuffles); A and Bt use the same
// order, so the product is unchanged.
//
// Every mbarrier wait is bounded by a clock limit.  A wait that expires raises the
// kernel's abort flag and the device status word; every role then finishes its current
// tile with short waits, takes no further tile and leaves through the common exit (TMEM
// is freed).
#include <cuda.h>

#include <mutex>

#include "q4_common.cuh"
#include "q4_requant8.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {

constexpr int TM = 128;            // rows of A per tile (UMMA M)
constexpr int PROW = 64;           // packed bytes per row per stage
constexpr int UROW = 128;          // unpacked bytes per row per stage (one swizzle row)
constexpr int UW = 8;              // unpack warps
constexpr int UT = UW * 32;        // unpack threads
constexpr int NTHREADS = (2 + UW + 4) * 32;

template <int BN> struct Cfg {
    // The unpack warps work as two groups of four that take the stages in turn, so that one
    // group's loads, fences and hand-over hide behind the other's work (256 columns: one group,
    // shared memory has no room for a second set of partial sums).
    static constexpr int UG = BN == 256 ? 1 : 2;
    static constexpr int GT = UT / UG;                         // threads per group
    static constexpr int ROWS = TM + BN;
    static constexpr int PSTAGE = ROWS * PROW;
    static constexpr int USTAGE = ROWS * UROW;
    static constexpr int STAGES = (BN == 256) ? 3 : 4;
    static constexpr int NT = (ROWS * 4 + GT - 1) / GT;        // unpack tasks (16-byte packed chunks) per thread and stage
    static constexpr int NBATCH = (NT + 5) / 6;                // ... taken in batches of at most six (registers)
    static constexpr int NTB = (NT + NBATCH - 1) / NBATCH;
    static constexpr int TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;
    // layout: [U stages][P stages][sums 2*ROWS int32][colterm BN int32][barriers][misc]
    static constexpr int OFF_U = 0;
    static constexpr int OFF_P = OFF_U + STAGES * USTAGE;
    static constexpr int OFF_SUMS = OFF_P + STAGES * PSTAGE;
    static constexpr int OFF_COLTERM = OFF_SUMS + 2 * UG * ROWS * 4;   // sums: int32 [2 accumulators][UG groups][ROWS]
    static constexpr int OFF_PC = OFF_COLTERM + BN * 4;        // per-channel: int32 [4][BN]
    static constexpr int OFF_BAR = OFF_PC + 4 * BN * 4;
    static constexpr int NBAR = 4 * STAGES + 6;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
    static constexpr int SMEM = OFF_MISC + 16 + 1024;          // + slack to align the base
    static_assert(SMEM <= 227 * 1024, "shared memory budget");
};

// Instruction descriptor: D = s32, A = B = unsigned 8-bit, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t make_idesc_u8(int n)
{
    return (2u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}

struct TcParams {
    GemmParams g;
    int32_t tiles_m, tiles_n, nslab;
    int32_t c_vec;      // int32 rows may be stored with 16-byte vectors
    int32_t cq_vec;     // packed rows may be stored with 16-byte vectors
};

template <int BN, bool REQUANT>
__global__ void __launch_bounds__(NTHREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const TcParams p)
{
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);

    const uint32_t sums_s = sbase + C::OFF_SUMS;          // int32 [2][UG][ROWS]
    const uint32_t colterm_s = sbase + C::OFF_COLTERM;    // int32 [BN]
    const uint32_t pc_s = sbase + C::OFF_PC;              // int32 [4][BN]: zero point, multiplier, rounding, shift
    const uint32_t bar0 = sbase + C::OFF_BAR;
    auto bar_full_p  = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto bar_empty_p = [&](int s) { return bar0 + 8u * (uint32_t)(C::STAGES + s); };
    auto bar_full_u  = [&](int s) { return bar0 + 8u * (uint32_t)(2 * C::STAGES + s); };
    auto bar_empty_u = [&](int s) { return bar0 + 8u * (uint32_t)(3 * C::STAGES + s); };
    auto bar_tfull   = [&](int a) { return bar0 + 8u * (uint32_t)(4 * C::STAGES + a); };
    auto bar_tempty  = [&](int a) { return bar0 + 8u * (uint32_t)(4 * C::STAGES + 2 + a); };
    auto bar_sums    = [&](int a) { return bar0 + 8u * (uint32_t)(4 * C::STAGES + 4 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_MISC);
    const uint32_t abort_flag = sbase + C::OFF_MISC + 4;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const GemmParams& g = p.g;
    const bool need_ra = (g.rowsum_a == nullptr);
    const bool need_cb = (g.colsum_b == nullptr);
    const bool need_sums = need_ra || need_cb;
    const int ntiles = p.tiles_m * p.tiles_n;
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(bar_full_p(s), 1);
            mbar_init(bar_empty_p(s), UW / C::UG);   // one arrive per warp of the group that took the stage
            mbar_init(bar_full_u(s), UW / C::UG);
            mbar_init(bar_empty_u(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);
            mbar_init(bar_tempty(a), 128);
            mbar_init(bar_sums(a), UT);
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
    // Launched with programmatic stream serialization: everything above may overlap the end
    // of the previous kernel of the stream; no operand is read and nothing is written before
    // that kernel has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // per-channel re-quantization: the 32-bit rounding form needs every shift in 2..27
    const bool pc = REQUANT && g.mult_ch != nullptr;
    int pc_fast = 1;
    if (pc) {
        int ok = 1;
        for (int n = threadIdx.x; n < g.N; n += NTHREADS) {
            const int sh = g.shift_ch[n];
            ok = ok && sh >= 2 && sh <= 27;
        }
        pc_fast = __syncthreads_and(ok);
    }

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < ntiles && !lds32(abort_flag); tile += gridDim.x) {
                const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    mbar_wait(bar_empty_p(st), ph ^ 1u, abort_flag, g.status);
                    mbar_expect_tx(bar_full_p(st), (uint32_t)C::PSTAGE);
                    const uint32_t dst = sbase + C::OFF_P + st * C::PSTAGE;
                    tma_load_2d(dst, &tmA, s * PROW, tm * TM, bar_full_p(st));
                    tma_load_2d(dst + TM * PROW, &tmB, s * PROW, tn * BN, bar_full_p(st));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_u8(BN);
            uint32_t it = 0, lt = 0;
            for (int tile = blockIdx.x; tile < ntiles && !lds32(abort_flag); tile += gridDim.x, ++lt) {
                const int acc = lt & 1;
                const uint32_t aph = (lt >> 1) & 1u;
                mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    mbar_wait(bar_full_u(st), ph, abort_flag, g.status);
                    tc_fence_after();
                    const uint32_t ua = sbase + C::OFF_U + st * C::USTAGE;
                    const uint64_t adesc = make_kmajor_sw128_desc(ua);
                    const uint64_t bdesc = make_kmajor_sw128_desc(ua + TM * UROW);
                    // all four 32-deep steps, always: past the end of a ragged depth the TMA
                    // loads filled both operands with zeros
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        tc_mma_i8(d_tmem, adesc + (uint64_t)(2 * i), bdesc + (uint64_t)(2 * i), idesc,
                                  (s > 0 || i > 0) ? 1u : 0u);
                    tc_commit(bar_empty_u(st));
                }
                tc_commit(bar_tfull(acc));
            }
        }
    } else if (warp < 2 + UW) {
        // ------------------------------------------------------------ unpack warps
        constexpr int UG = C::UG, GT = C::GT;
        const int grp = (warp - 2) / (UW / UG);          // takes the stages with it % UG == grp
        const int gt = threadIdx.x - 64 - grp * GT;      // 0 .. GT-1 inside the group
        uint32_t it = (uint32_t)grp, lt = 0;
        for (int tile = blockIdx.x; tile < ntiles && !lds32(abort_flag); tile += gridDim.x, ++lt) {
            int psum[C::NT];
#pragma unroll
            for (int j = 0; j < C::NT; ++j) psum[j] = 0;
            // stages are numbered across tiles: stage s of my lt-th tile is lt * nslab + s
            const uint32_t it_end = (lt + 1) * (uint32_t)p.nslab;
            for (; it < it_end; it += UG) {
                const int st = it % C::STAGES;
                const uint32_t ph = (it / C::STAGES) & 1u;
                mbar_wait(bar_full_p(st), ph, abort_flag, g.status);
                const uint32_t ps = sbase + C::OFF_P + st * C::PSTAGE;
                const uint32_t us = sbase + C::OFF_U + st * C::USTAGE;
#pragma unroll
                for (int b = 0; b < C::NBATCH; ++b) {
                    // a batch's loads first (their latencies overlap), then -- before the first
                    // store -- the wait for the unpacked slot
                    uint4 wv[C::NTB];
#pragma unroll
                    for (int jj = 0; jj < C::NTB; ++jj) {
                        const int j = b * C::NTB + jj;
                        const int id = gt + j * GT;
                        if (j < C::NT && id < C::ROWS * 4) wv[jj] = lds128(ps + (id >> 2) * PROW + (id & 3) * 16);
                    }
                    if (b == 0) {
                        mbar_wait(bar_empty_u(st), ph ^ 1u, abort_flag, g.status);
                        tc_fence_after();
                    }
#pragma unroll
                    for (int jj = 0; jj < C::NTB; ++jj) {
                        const int j = b * C::NTB + jj;
                        const int id = gt + j * GT;
                        const int r = id >> 2, c = id & 3;
                        if (j < C::NT && id < C::ROWS * 4) {
                            const uint4 w = wv[jj];
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
                }
                // every lane publishes its own writes to the async proxy; one lane per warp
                // then arrives (many arrives on one barrier word serialise badly)
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
                // the epilogue two tiles back must be done with this sums buffer
                mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
#pragma unroll
                for (int j = 0; j < C::NT; ++j) {
                    int t = psum[j];
                    t += __shfl_xor_sync(0xFFFFFFFFu, t, 1);
                    t += __shfl_xor_sync(0xFFFFFFFFu, t, 2);
                    const int id = gt + j * GT;
                    if (id < C::ROWS * 4 && (id & 3) == 0)
                        sts32(sums_s + 4 * ((acc * UG + grp) * C::ROWS + (id >> 2)), t);
                }
                mbar_arrive(bar_sums(acc));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int lg = warp & 3;                 // TMEM lane group this warp may read
        const int row = lg * 32 + lane;          // row of the tile held by this thread
        const int et = threadIdx.x - (2 + UW) * 32;   // 0..127
        uint32_t lt = 0;
        for (int tile = blockIdx.x; tile < ntiles && !lds32(abort_flag); tile += gridDim.x, ++lt) {
            const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
            const int acc = lt & 1;
            const uint32_t aph = (lt >> 1) & 1u;
            const int m = tm * TM + row;
            const int n0 = tn * BN;
            if (need_sums) mbar_wait(bar_sums(acc), aph, abort_flag, g.status);
            // per-column term of Eq. 2: -za * colsum + K za zb (+ bias)
            for (int j = et; j < BN; j += 128) {
                const int n = n0 + j;
                int cb = 0, bias = 0, zbn = pc ? 0 : g.zb;
                if (n < g.N) {
                    if (need_cb) {
#pragma unroll
                        for (int gi = 0; gi < C::UG; ++gi) cb += lds32(sums_s + 4 * ((acc * C::UG + gi) * C::ROWS + TM + j));
                    } else {
                        cb = g.colsum_b[n];
                    }
                    if (REQUANT && g.bias) bias = g.bias[n];
                    if (pc && g.zb_ch) zbn = g.zb_ch[n];
                }
                sts32(colterm_s + 4 * j,
                      (int)((uint32_t)(g.K * g.za * zbn) - (uint32_t)(g.za * cb) + (uint32_t)bias));
                if (pc) {
                    const int mult = n < g.N ? g.mult_ch[n] : (1 << 30);
                    const int sh = n < g.N ? g.shift_ch[n] : 2;
                    const int s = pc_fast ? sh - 1 : sh;
                    sts32(pc_s + 4 * j, zbn);
                    sts32(pc_s + 4 * (BN + j), mult);
                    sts32(pc_s + 4 * (2 * BN + j), pc_fast ? (1 << (s - 1)) + (g.rq.zo - g.rq.lo) * (1 << s) : 0);
                    sts32(pc_s + 4 * (3 * BN + j), s);
                }
            }
            int ra = 0;
            if (need_ra) {
#pragma unroll
                for (int gi = 0; gi < C::UG; ++gi) ra += lds32(sums_s + 4 * ((acc * C::UG + gi) * C::ROWS + row));
            }
            else if (m < g.M) ra = g.rowsum_a[m];
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
                if (pc) {
                    // the column's own zero point in Eq. 2's row-sum term
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const uint4 ct = lds128(colterm_s + 4 * (ch * 32 + 4 * q));
                        const uint4 zz = lds128(pc_s + 4 * (ch * 32 + 4 * q));
                        r[4 * q + 0] += ct.x - (uint32_t)ra * zz.x;
                        r[4 * q + 1] += ct.y - (uint32_t)ra * zz.y;
                        r[4 * q + 2] += ct.z - (uint32_t)ra * zz.z;
                        r[4 * q + 3] += ct.w - (uint32_t)ra * zz.w;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const uint4 ct = lds128(colterm_s + 4 * (ch * 32 + 4 * q));
                        r[4 * q + 0] += rowterm + ct.x;
                        r[4 * q + 1] += rowterm + ct.y;
                        r[4 * q + 2] += rowterm + ct.z;
                        r[4 * q + 3] += rowterm + ct.w;
                    }
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
                        if (pc) {
                            // eight values at a time (channels i and i + 4 share a packed pair); each
                            // word holds value - lo per nibble
                            const uint32_t hml2 = (uint32_t)(g.rq.hi - g.rq.lo) * 0x00010001u;
                            const uint32_t lofill = (uint32_t)g.rq.lo * 0x11111111u;
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                o[q] = requant8_channels<true>(r + 8 * q, g.rq, pc_s + 4 * BN, BN, ch * 32 + 8 * q,
                                                               pc_fast != 0, hml2) + lofill;
                        } else {
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                uint32_t wv = 0;
#pragma unroll
                                for (int e = 0; e < 8; ++e)
                                    wv |= requant((int32_t)r[8 * q + e], g.rq) << (4 * e);
                                o[q] = wv;
                            }
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

// ---- host side ------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

// Packed matrix [rows x kbytes] with pitch ld, box = 64 bytes x box_rows; out-of-range
// rows and bytes are filled with zeros (zero nibbles add nothing to any term of Eq. 2).
// swizzle64: the 16-byte chunks of each 64-byte row are XOR-permuted by (row / 2) % 4 in
// shared memory, which makes one-row-per-lane reads bank-conflict free.
bool make_packed_map(CUtensorMap* tm, const uint8_t* base, int64_t ld, int rows, int kbytes,
                     int box_rows, bool swizzle64)
{
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kbytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {(cuuint32_t)PROW, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides,
               box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// One-byte-per-value matrix [rows x kbytes] with pitch ld, box = 128 bytes x box_rows with
// the 128-byte swizzle: the tile lands in the K-major layout the MMA descriptors describe.
// Out-of-range rows and bytes are filled with zeros.
bool make_byte_map(CUtensorMap* tm, const uint8_t* base, int64_t ld, int rows, int kbytes, int box_rows)
{
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kbytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides,
               box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool gemm_tc_supported(const GemmParams& p)
{
    return ((uintptr_t)p.A % 16 == 0) && ((uintptr_t)p.Bt % 16 == 0) && (p.lda % 16 == 0) &&
           (p.ldb % 16 == 0) && p.M > 0 && p.N > 0;
}

static int sm_count()
{
    static int per_dev[64] = {};           // SM count of each device, looked up with it current
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int& n = per_dev[dev];
    if (!n) {
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

template <int BN>
static q4_status launch_bn(const GemmParams& g, bool rq, cudaStream_t st)
{
    using C = Cfg<BN>;
    TcParams p;
    p.g = g;
    p.tiles_m = (g.M + TM - 1) / TM;
    p.tiles_n = (g.N + BN - 1) / BN;
    const int kbytes = (g.K + 1) / 2;
    p.nslab = (kbytes + PROW - 1) / PROW;
    p.c_vec = (!rq && ((uintptr_t)g.C % 16 == 0) && (g.ldc % 4 == 0)) ? 1 : 0;
    p.cq_vec = (rq && ((uintptr_t)g.Cq % 16 == 0) && (g.ldcq % 16 == 0)) ? 1 : 0;

    CUtensorMap tmA, tmB;
    if (!make_packed_map(&tmA, g.A, g.lda, g.M, kbytes, TM, false)) return Q4_ERR_CUDA;
    if (!make_packed_map(&tmB, g.Bt, g.ldb, g.N, kbytes, BN, false)) return Q4_ERR_CUDA;

    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
    cudaError_t e;
    // the attribute is per kernel and per device: set on every call, it is cheap
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel waits before it touches memory
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = C::SMEM;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (rq) {
        e = cudaFuncSetAttribute(gemm_tc_kernel<BN, true>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
        if (e != cudaSuccess) return Q4_ERR_CUDA;
        e = cudaLaunchKernelEx(&cfg, gemm_tc_kernel<BN, true>, tmA, tmB, p);
    } else {
        e = cudaFuncSetAttribute(gemm_tc_kernel<BN, false>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
        if (e != cudaSuccess) return Q4_ERR_CUDA;
        e = cudaLaunchKernelEx(&cfg, gemm_tc_kernel<BN, false>, tmA, tmB, p);
    }
    count_launch();
    return e == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status launch_gemm_tc(const GemmParams& g, bool rq, cudaStream_t st)
{
    int bn = g.N > 128 ? 256 : g.N > 64 ? 128 : g.N > 32 ? 64 : 32;
    // a grid that would leave more than a quarter of the SMs idle: narrower tiles, more CTAs
    const long long rows = (g.M + TM - 1) / TM;
    while (bn > 32 && rows * ((g.N + bn - 1) / bn) * 4 < 3LL * sm_count()) bn >>= 1;
    if (bn == 256) return launch_bn<256>(g, rq, st);
    if (bn == 128) return launch_bn<128>(g, rq, st);
    if (bn == 64)  return launch_bn<64>(g, rq, st);
    return launch_bn<32>(g, rq, st);
}

}  // namespace q4
