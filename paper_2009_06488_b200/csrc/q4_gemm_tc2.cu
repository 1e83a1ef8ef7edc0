// Tensor-core 4-bit quantized GEMM for large problems (Eq. 2 of the paper, all four
// terms): CTA pairs computing 256 x 192 or 256 x 256 output tiles with
// tcgen05.mma.cta_group::2, the A operand fed from tensor memory.
//
// Why this shape.  The unpack (nibbles -> bytes) costs shared-memory traffic -- every
// packed byte is read once and every unpacked byte written once before the MMA can read
// it, through a 128 B/clk pipe -- and instructions of the unpack warps, which is what
// bound the kernel in the end.  Two things cut the traffic:
//   * a CTA pair shares the Bt tile, so each CTA stages and unpacks only half of it;
//   * the unpacked A rows never touch shared memory: each unpack thread owns one row,
//     expands its 64 packed bytes in registers and writes them to tensor memory
//     (tcgen05.st), from where the MMA reads A directly.
// Per 128-deep stage a CTA then moves 8 KB (A, loads only) + 6 KB + 12 KB (Bt, loads and
// stores; 8 + 16 KB with 256-column tiles) through the load/store pipe -- about half of
// what the MMAs' 400 to 530 clocks allow.
//
// Tensor memory (512 columns), 192-column tiles: two accumulators (the epilogue of tile t
// overlaps the main loop of t+1) and four A stages of 32 columns (128 depth bytes); the
// unpacked Bt stages live in a deeper shared-memory ring (eight), so only the short
// tensor-memory store of A sits between "stage free" and "operands ready".  256-column
// tiles: three half accumulators of 128 columns in rotation, four A and four Bt stages
// (see Cfg).
//
// Roles per CTA (18 warps): warp 0 TMA producer (its own 128 rows of A, 64-byte-swizzled
// so that row-per-lane reads are conflict-free, and its own half of the tile's rows of Bt;
// no multicast); warps 2..13 unpack, as three groups of four that take stages in turn so
// one group's waits and fences hide behind the others' work, and arrive -- from both
// CTAs -- on the leader CTA's "operands ready" barrier; warp 1 of the leader CTA issues
// the pair MMAs and commits to both CTAs' barriers; warp 1 of the peer CTA relays
// "accumulator drained" to the leader; the last four warps are the epilogue.  Column sums
// of the two CTAs' Bt rows are exchanged through distributed shared memory.
//
// The depth order inside each 32-value group (even nibbles, then odd) is the same for A
// and Bt, so the product is unchanged.  Every mbarrier wait is bounded; the only
// unbounded waits are the cluster barriers at entry and exit, which every thread
// reaches unconditionally.  A wait that runs out raises the CTA's abort flag: every role
// then finishes its current tile with short waits and takes no further tile.  The waits
// acquire at CTA scope -- what they order is asynchronous-proxy traffic (TMA, tcgen05)
// fenced explicitly -- except the wait on the depth-sum exchange, the one place where data
// written by the peer CTA's threads with ordinary stores is read afterwards: a
// cluster-scope acquire costs an L1 invalidate per try (8192^3: 367 -> 359 us without).
#include <cuda.h>

#include "q4_common.cuh"
#include "q4_requant8.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {
namespace pair {

constexpr int TMC = 128;             // rows of A per CTA
constexpr int PROW = 64, UROW = 128;
constexpr int PA = TMC * PROW;       // packed A bytes per stage
#ifndef Q4_PAIR_GROUPS
#define Q4_PAIR_GROUPS 3
#endif
constexpr int G = Q4_PAIR_GROUPS, WPG = 4, GT = WPG * 32;   // unpack groups, warps / threads per group
constexpr int UW = G * WPG;
constexpr int NTHREADS = (2 + UW + 4) * 32;
constexpr int TMEM_COLS = 512;
constexpr int STG_SET = 4 * 32 * 128;      // int32 epilogue staging: 4 warps x 32 rows x 128 B

// Two tile widths, chosen per problem by the launcher.  Tensor memory holds NACC
// accumulators of BNC columns and US A stages of 32 columns.
// 192 columns: two accumulators (the epilogue of a tile overlaps the next tile's main
// loop), four A stages, eight Bt stages.
// 256 columns: a third more work per unpacked row of A, but two whole accumulators would
// leave no room for A.  The accumulator is therefore two halves of 128 columns out of three
// half-buffers (ROT): every tile's upper half (columns 128..255) lives in the middle buffer,
// the lower halves alternate between the outer two, and each depth step is two MMAs of 128
// columns (the same tensor time as one of 256).  The epilogue drains the upper half first;
// the next tile's lower-half MMAs start at once on the free outer buffer and only its
// upper-half MMAs wait for that half drain; a tile's last upper-half MMAs are issued before
// its last lower-half ones, so that the drain starts early.  About a third of the epilogue is
// exposed instead of all of it.  Four A and four Bt stages.  It wins where its tile count fits the
// 74 CTA pairs better or the depth is long, and loses e.g. at 4096^3 (four waves against
// five of 192-column tiles with fully overlapped epilogues).
// NSTG: staging slices per epilogue warp.  With two, a TMA store reads one while the next is
// filled.  The 192-column form has room for two; in the 256-column form a second set would
// cost a packed stage, which long problems miss (8192^3: 297 -> 302 us), and short ones no
// longer need it since the unpack warps help to drain a CTA pair's last tile.
template <int BNC_, int NSTG_>
struct Cfg {
    static constexpr int BNC = BNC_;             // columns of the pair tile
    static constexpr int NSTG = NSTG_;
    static constexpr int STG_BYTES = NSTG * STG_SET;
    static constexpr int BH = BNC / 2;           // rows of Bt staged per CTA
    static constexpr bool ROT = BNC == 256;      // rotating half accumulators
    static constexpr int NACC = ROT ? 1 : 2;     // whole accumulators / depth-sum buffers in flight
    static constexpr int US = 4;                 // A operand stages in tensor memory
    static constexpr int BS = ROT ? 4 : 8;       // Bt operand stages in shared memory (BH * 128 B each)
    static constexpr int WALK = BS;              // stages per block of the MMA loop: a multiple of both ring depths
    static constexpr int BBOX = ROT ? BH / 2 : BH;   // rows per TMA box of Bt
    static constexpr int PS = ROT ? 8 : 6;       // packed stages (A 8 KB + Bt BH * 64 B)
    static constexpr int PSTAGE = PA + BH * PROW;
    static constexpr int BSTAGE = BH * UROW;     // unpacked Bt bytes per stage
    static constexpr int NTB = BH * 4 / GT;      // Bt tasks (16-byte packed chunks) per thread per stage
    static constexpr int ACOL0 = ROT ? 384 : NACC * BNC;     // first TMEM column of the A stages
    static constexpr int SUMS_N = TMC + BNC;     // per buffer and group: 128 row sums, BNC column sums

    static constexpr int OFF_B = 0;
    static constexpr int OFF_P = OFF_B + BS * BSTAGE;
    static constexpr int OFF_STG = OFF_P + PS * PSTAGE;
    static constexpr int OFF_SUMS = OFF_STG + STG_BYTES;
    static constexpr int OFF_COLTERM = OFF_SUMS + 2 * G * SUMS_N * 4;
    static constexpr int OFF_PC = OFF_COLTERM + BNC * 4;       // per-channel: int32 [4][BNC] zero point, multiplier, rounding, shift
    static constexpr int OFF_BAR = OFF_PC + 4 * BNC * 4;
    static constexpr int NBAR = 2 * PS + 2 * US + BS + 13;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
    static constexpr int SMEM = OFF_MISC + 16 + 1024;

    static_assert(BH * 4 % GT == 0, "Bt tasks must divide evenly");
    static_assert(ACOL0 + US * 32 <= TMEM_COLS, "tensor memory budget");
    static_assert(WALK % BS == 0 && WALK % US == 0, "the MMA loop walks blocks of WALK stages and derives both ring slots from the position in the block");
    static_assert(BSTAGE % 1024 == 0 && PSTAGE % 1024 == 0, "stage alignment");
    static_assert(OFF_STG % 1024 == 0, "staging tile alignment (128-byte swizzle atoms)");
    static_assert(SMEM <= 227 * 1024, "shared memory budget");
    static_assert(!ROT || NSTG == 1, "the 256-column form has room for one set of staging slices");
    static_assert(G <= PS, "a group's packed-ring slot advances by G per stage and wraps at most once");
    static_assert(((BNC / 32 - 1) / 2) * WPG * 2 * 4096 <= PS * PSTAGE && G + 1 >= (BNC / 32 + 1) / 2,
                  "last tile: the helping unpack warps stage two chunks each in the packed ring, and with the epilogue warps they cover every chunk");

    // D = s32, A = B = unsigned 8-bit, K-major, M = 256 (pair), N = BNC (ROT: BNC / 2 per MMA).
    static constexpr uint32_t kIdesc = (2u << 4) | ((uint32_t)((ROT ? BNC / 2 : BNC) >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
};

struct Params {
    GemmParams g;
    int32_t tiles_m, tiles_n, nslab;
    int32_t c_vec, cq_vec;
    int32_t c_tma;      // int32 output goes out through TMA stores (tmC is valid)
};

__device__ __forceinline__ void unpack16(const uint4& w, uint4& lo, uint4& hi)
{
    lo.x = w.x & 0x0F0F0F0Fu; hi.x = (w.x >> 4) & 0x0F0F0F0Fu;
    lo.y = w.y & 0x0F0F0F0Fu; hi.y = (w.y >> 4) & 0x0F0F0F0Fu;
    lo.z = w.z & 0x0F0F0F0Fu; hi.z = (w.z >> 4) & 0x0F0F0F0Fu;
    lo.w = w.w & 0x0F0F0F0Fu; hi.w = (w.w >> 4) & 0x0F0F0F0Fu;
}
// Sum of the 32 values of one unpacked chunk (bytes of the word sum stay <= 120).
__device__ __forceinline__ int chunk_sum(const uint4& lo, const uint4& hi, int acc)
{
    const uint32_t t = (lo.x + hi.x) + (lo.y + hi.y) + (lo.z + hi.z) + (lo.w + hi.w);
    return dp4a_u8(t, 0x01010101u, acc);
}

template <int BNC, int NSTG, bool REQUANT>
__global__ void __launch_bounds__(NTHREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, const Params p)
{
    using C = Cfg<BNC, NSTG>;
    constexpr int BH = C::BH, NACC = C::NACC, US = C::US, BS = C::BS, PSTAGE = C::PSTAGE, BSTAGE = C::BSTAGE,
                  NTB = C::NTB, ACOL0 = C::ACOL0, SUMS_N = C::SUMS_N, OFF_B = C::OFF_B, OFF_P = C::OFF_P,
                  OFF_STG = C::OFF_STG, OFF_SUMS = C::OFF_SUMS, OFF_COLTERM = C::OFF_COLTERM, OFF_PC = C::OFF_PC,
                  OFF_BAR = C::OFF_BAR, OFF_MISC = C::OFF_MISC;
    constexpr uint32_t kIdesc = C::kIdesc;
    constexpr bool ROT = C::ROT;
    constexpr int PS = C::PS, WALK = C::WALK;
    extern __shared__ uint8_t smem_raw[];
    // the same offset in both CTAs: dynamic shared memory starts at the same address
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;

    const uint32_t sums_s = sbase + OFF_SUMS;        // int32 [2 buffers][G][SUMS_N]
    const uint32_t colterm_s = sbase + OFF_COLTERM;  // int32 [BNC]
    const uint32_t pc_s = sbase + OFF_PC;            // int32 [4][BNC]
    const uint32_t bar0 = sbase + OFF_BAR;
    auto bar_full_p    = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto bar_empty_p   = [&](int s) { return bar0 + 8u * (uint32_t)(PS + s); };
    auto bar_full_u    = [&](int s) { return bar0 + 8u * (uint32_t)(2 * PS + s); };
    auto bar_empty_b   = [&](int s) { return bar0 + 8u * (uint32_t)(2 * PS + 2 * US + s); };
    const uint32_t barT = bar0 + 8u * (uint32_t)(2 * PS + 2 * US + BS);
    // accumulator buffers: two whole ones, or (ROT) 0 / 1 = the outer half-buffers of even /
    // odd tiles, 2 = the middle one
    auto bar_tfull       = [&](int a) { return barT + 8u * (uint32_t)a; };
    auto bar_tempty      = [&](int a) { return barT + 8u * (uint32_t)(2 + a); };
    auto bar_peer_tempty = [&](int a) { return barT + 8u * (uint32_t)(5 + a); };
    auto bar_sums        = [&](int a) { return barT + 8u * (uint32_t)(8 + a); };
    auto bar_tstart      = [&](int a) { return barT + 8u * (uint32_t)(10 + a); };
    const uint32_t bar_final = barT + 8u * 12u;      // the last tile's column terms are in shared memory
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
        for (int s = 0; s < PS; ++s) {
            mbar_init(bar_full_p(s), 1);
            mbar_init(bar_empty_p(s), WPG);      // one arrive per warp of the group that took it
        }
        for (int s = 0; s < US; ++s)
            mbar_init(bar_full_u(s), 2 * WPG);   // used in the leader: a group's warps of both CTAs
        for (int s = 0; s < BS; ++s)
            mbar_init(bar_empty_b(s), 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);
            // one arrive per unpack warp: of both CTAs where column sums are exchanged, else of this one
            mbar_init(bar_sums(a), need_cb ? 2 * UW : UW);
            mbar_init(bar_tstart(a), 1);
        }
        for (int a = 0; a < 3; ++a) {
            mbar_init(bar_tempty(a), 128);
            mbar_init(bar_peer_tempty(a), 1);
        }
        mbar_init(bar_final, 128);
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

    // One 32-column chunk of an accumulator: tensor memory -> Eq. 2's remaining terms -> the
    // output (int32 through a staging slice and a TMA store, or re-quantized and packed).
    // taddr: the chunk in tensor memory (my lane quarter lg); ch, nc: its first column in the
    // tile / in C; m, ra, rowterm: my row, its depth sum and Eq. 2's row term; slice: my
    // 4 KB staging slice and how to wait for it (0: it is free, 1: my stores have all read
    // their slices, 2: all but the latest); release_mid: hand the middle half-buffer back
    // once the chunk is in registers.
    auto drain_chunk = [&](uint32_t taddr, int ch, int nc, int lg, int tm, int m, int ra, uint32_t rowterm,
                           uint32_t slice, int slice_wait, bool release_mid) {
        uint32_t r[32];
        tc_ld32(taddr, r);
        tc_wait_ld();
        if (ROT && release_mid) {
            // the middle buffer is in registers: the next tile's upper-half MMAs may start
            tc_fence_before();
            mbar_arrive(bar_tempty(2));
        }
        if (pc) {
            // the column's own zero point in Eq. 2's row-sum term
#pragma unroll
            for (int qd = 0; qd < 8; ++qd) {
                const uint4 ct = lds128(colterm_s + 4 * (ch * 32 + 4 * qd));
                const uint4 zz = lds128(pc_s + 4 * (ch * 32 + 4 * qd));
                r[4 * qd + 0] += ct.x - (uint32_t)ra * zz.x;
                r[4 * qd + 1] += ct.y - (uint32_t)ra * zz.y;
                r[4 * qd + 2] += ct.z - (uint32_t)ra * zz.z;
                r[4 * qd + 3] += ct.w - (uint32_t)ra * zz.w;
            }
        } else {
#pragma unroll
            for (int qd = 0; qd < 8; ++qd) {
                const uint4 ct = lds128(colterm_s + 4 * (ch * 32 + 4 * qd));
                r[4 * qd + 0] += rowterm + ct.x;
                r[4 * qd + 1] += rowterm + ct.y;
                r[4 * qd + 2] += rowterm + ct.z;
                r[4 * qd + 3] += rowterm + ct.w;
            }
        }
        if (!REQUANT && p.c_tma) {
            // int32 tile out through shared memory and one TMA store per warp: my
            // row's 128 bytes go to the swizzled staging slice of my warp; rows and
            // columns past M / N are clipped by the tensor map
            if (lane == 0) {                       // the store that last used this slice has read it
                if (slice_wait == 2) bulk_wait_read_but_one(); else if (slice_wait == 1) bulk_wait_read();
            }
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
            const bool full = (nc + 32 <= g.N);
            if (!REQUANT) {
                int32_t* dst = g.C + (int64_t)m * g.ldc + nc;
                if (full && p.c_vec) {
#pragma unroll
                    for (int qd = 0; qd < 8; ++qd)
                        *reinterpret_cast<uint4*>(dst + 4 * qd) =
                            make_uint4(r[4 * qd], r[4 * qd + 1], r[4 * qd + 2], r[4 * qd + 3]);
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
                    for (int qd = 0; qd < 4; ++qd)
                        o[qd] = requant8_channels<true>(r + 8 * qd, g.rq, pc_s + 4 * BNC, BNC, ch * 32 + 8 * qd,
                                                        pc_fast != 0, hml2) + lofill;
                } else {
#pragma unroll
                    for (int qd = 0; qd < 4; ++qd) {
                        uint32_t wv = 0;
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            wv |= requant((int32_t)r[8 * qd + e], g.rq) << (4 * e);
                        o[qd] = wv;
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
    };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = cluster_id; tile < ntiles && !lds32(abort_flag); tile += nclusters) {
                const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
                const int arow = tm * 256 + (int)rank * TMC;
                // ROT: my Bt rows are two runs of 64, one from each half of the tile's columns
                const int brow = tn * BNC + (int)rank * C::BBOX;
                for (int s = 0; s < p.nslab; ++s, ++it) {
                    const int st = it % PS;
                    const uint32_t ph = (it / PS) & 1u;
                    mbar_wait(bar_empty_p(st), ph ^ 1u, abort_flag, g.status);
                    mbar_expect_tx(bar_full_p(st), (uint32_t)PSTAGE);
                    const uint32_t dst = sbase + OFF_P + st * PSTAGE;
                    tma_load_2d(dst, &tmA, s * PROW, arow, bar_full_p(st));
                    tma_load_2d(dst + PA, &tmB, s * PROW, brow, bar_full_p(st));
                    if (ROT) tma_load_2d(dst + PA + C::BBOX * PROW, &tmB, s * PROW, brow + BH, bar_full_p(st));
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // -------------------------------------------------------- pair MMA issuer
            // The whole warp runs the loop (uniform control flow and addresses); one
            // elected lane issues the MMAs and commits.
            const uint32_t a_tmem0 = tmem_base + (uint32_t)ACOL0;
            const uint64_t bdesc0 = make_kmajor_sw128_desc(sbase + OFF_B);
            constexpr uint32_t kUpper = (uint32_t)(BH / 2 * UROW >> 4);   // ROT: descriptor offset of Bt rows 64..127
            uint32_t lt = 0;
            for (int tile = cluster_id; tile < ntiles && !lds32(abort_flag); tile += nclusters, ++lt) {
                const int acc = (int)(lt % NACC);
                const uint32_t aph = (lt / NACC) & 1u;
                // Stages are numbered across tiles (stage s of my lt-th tile is lt*nslab + s).
                const uint32_t it_begin = lt * (uint32_t)p.nslab, it_end = it_begin + (uint32_t)p.nslab;
                uint32_t d_tmem, d_up = 0, it_main = it_begin, it_tail = it_end;
                if (!ROT) {
                    mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
                    if (lt >= (uint32_t)NACC) mbar_wait(bar_peer_tempty(acc), aph ^ 1u, abort_flag, g.status);
                    tc_fence_after();
                    // both epilogues are done with buffer `acc`: tell the unpack warps of both CTAs
                    if (elect_one()) tc_commit_pair(bar_tstart(acc), 3);
                    __syncwarp();
                    d_tmem = tmem_base + (uint32_t)(acc * BNC);
                } else {
                    // Lower half: the outer buffer of this tile's parity, drained two tiles ago.
                    const int lo = (int)(lt & 1u);
                    const uint32_t lph = ((lt >> 1) & 1u) ^ 1u, mph = (lt & 1u) ^ 1u;
                    mbar_wait(bar_tempty(lo), lph, abort_flag, g.status);
                    if (lt >= 2u) mbar_wait(bar_peer_tempty(lo), lph, abort_flag, g.status);
                    tc_fence_after();
                    d_tmem = tmem_base + (lo ? 256u : 0u);
                    d_up = tmem_base + 128u;
                    // The lower-half MMAs of the first stages run while the previous tile's upper
                    // half is still being drained from the middle buffer ...
                    const uint32_t la = (uint32_t)p.nslab < (uint32_t)US ? (uint32_t)p.nslab : (uint32_t)US;
                    for (uint32_t k = 0; k < la; ++k) {
                        const uint32_t it = it_begin + k;
                        mbar_wait(bar_full_u((int)(it % US)), (it / US) & 1u, abort_flag, g.status);
                        tc_fence_after();
                        const uint32_t a_tmem = a_tmem0 + (it % US) * 32u;
                        const uint64_t bdesc = bdesc0 + (uint64_t)((it % BS) * (uint32_t)(BSTAGE >> 4));
                        if (elect_one()) {
#pragma unroll
                            for (uint32_t i = 0; i < 4; ++i)
                                tc_mma_i8_pair_ts(d_tmem, a_tmem + 8u * i, bdesc + 2u * i, kIdesc, (k | i) ? 1u : 0u);
                        }
                        __syncwarp();
                    }
                    // ... then the upper halves of the same stages, once it is free
                    mbar_wait(bar_tempty(2), mph, abort_flag, g.status);
                    if (lt >= 1u) mbar_wait(bar_peer_tempty(2), mph, abort_flag, g.status);
                    tc_fence_after();
                    // both epilogues have also read the previous tile's depth sums by now
                    if (elect_one()) tc_commit_pair(bar_tstart(acc), 3);
                    __syncwarp();
                    for (uint32_t k = 0; k < la; ++k) {
                        const uint32_t it = it_begin + k;
                        const uint32_t a_tmem = a_tmem0 + (it % US) * 32u;
                        const uint64_t bdesc = bdesc0 + (uint64_t)((it % BS) * (uint32_t)(BSTAGE >> 4) + kUpper);
                        if (elect_one()) {
#pragma unroll
                            for (uint32_t i = 0; i < 4; ++i)
                                tc_mma_i8_pair_ts(d_up, a_tmem + 8u * i, bdesc + 2u * i, kIdesc, (k | i) ? 1u : 0u);
                            tc_commit_pair(bar_empty_b((int)(it % BS)), 3);
                        }
                        __syncwarp();
                    }
                    it_main = it_begin + la;
                    // the stages of the tail (see below): up to US of those left
                    const uint32_t left = (uint32_t)p.nslab - la;
                    it_tail = it_end - (left < (uint32_t)US ? left : (uint32_t)US);
                    if (it_tail == it_end && elect_one()) tc_commit_pair(bar_tfull(1), 3);   // no tail: the upper half is complete
                    __syncwarp();
                }
                // The loop walks the stages in aligned blocks of WALK (a multiple of both ring depths)
                // so that ring slots, tensor-memory columns, descriptors and barrier addresses are
                // compile-time offsets.
                for (uint32_t blk = it_main - it_main % WALK; blk < it_tail; blk += WALK) {
                    const uint32_t bph = (blk / US) & 1u;     // phase of A slot 0 in this block
#pragma unroll
                    for (int j = 0; j < WALK; ++j) {
                        const uint32_t it = blk + (uint32_t)j;
                        if (it < it_main || it >= it_tail) continue;        // warp-uniform
                        // A ring slot j % US: its phase is (it / US) & 1, blk being a multiple of US
                        mbar_wait(bar_full_u(j % US), (bph + (uint32_t)(j / US)) & 1u, abort_flag, g.status);
                        tc_fence_after();
                        const uint32_t a_tmem = a_tmem0 + (uint32_t)((j % US) * 32);
                        const uint64_t bdesc = bdesc0 + (uint64_t)((j % BS) * (BSTAGE >> 4));
                        if (elect_one()) {
                            // a ragged last stage is multiplied whole: its missing depth is zeros
                            tc_mma_i8_pair_ts(d_tmem, a_tmem, bdesc, kIdesc, it > it_begin ? 1u : 0u);
                            tc_mma_i8_pair_ts(d_tmem, a_tmem + 8u, bdesc + 2u, kIdesc, 1u);
                            tc_mma_i8_pair_ts(d_tmem, a_tmem + 16u, bdesc + 4u, kIdesc, 1u);
                            tc_mma_i8_pair_ts(d_tmem, a_tmem + 24u, bdesc + 6u, kIdesc, 1u);
                            if (ROT) {
#pragma unroll
                                for (uint32_t i = 0; i < 4; ++i)
                                    tc_mma_i8_pair_ts(d_up, a_tmem + 8u * i, bdesc + kUpper + 2u * i, kIdesc, 1u);
                            }
                            // one commit frees this stage's Bt slot and, through the same
                            // barrier, its A slot (see the unpack warps' wait)
                            tc_commit_pair(bar_empty_b(j % BS), 3);
                        }
                        __syncwarp();
                    }
                    (void)bph;
                }
                if (ROT && it_tail < it_end) {
                    // Tail: the last stages' upper-half MMAs first, so that the epilogue can start on
                    // the middle buffer -- which the next tile needs first -- while their lower-half
                    // MMAs and the next tile's first lower-half MMAs still run.
                    for (uint32_t it = it_tail; it < it_end; ++it) {
                        mbar_wait(bar_full_u((int)(it % US)), (it / US) & 1u, abort_flag, g.status);
                        tc_fence_after();
                        const uint32_t a_tmem = a_tmem0 + (it % US) * 32u;
                        const uint64_t bdesc = bdesc0 + (uint64_t)((it % BS) * (uint32_t)(BSTAGE >> 4) + kUpper);
                        if (elect_one()) {
#pragma unroll
                            for (uint32_t i = 0; i < 4; ++i)
                                tc_mma_i8_pair_ts(d_up, a_tmem + 8u * i, bdesc + 2u * i, kIdesc, 1u);
                        }
                        __syncwarp();
                    }
                    if (elect_one()) tc_commit_pair(bar_tfull(1), 3);      // the upper half is complete
                    __syncwarp();
                    for (uint32_t it = it_tail; it < it_end; ++it) {
                        const uint32_t a_tmem = a_tmem0 + (it % US) * 32u;
                        const uint64_t bdesc = bdesc0 + (uint64_t)((it % BS) * (uint32_t)(BSTAGE >> 4));
                        if (elect_one()) {
#pragma unroll
                            for (uint32_t i = 0; i < 4; ++i)
                                tc_mma_i8_pair_ts(d_tmem, a_tmem + 8u * i, bdesc + 2u * i, kIdesc, 1u);
                            tc_commit_pair(bar_empty_b((int)(it % BS)), 3);
                        }
                        __syncwarp();
                    }
                }
                if (elect_one()) tc_commit_pair(bar_tfull(acc), 3);
                __syncwarp();
            }
        } else if (lane == 0) {
            // -------------------------------------------------------- peer relay (per tile)
            // forwards "my epilogue has drained the buffer" to the leader, which issues the MMAs.
            // The arrives carry no release: what they order is the epilogue's tensor-memory
            // loads, which were complete (tcgen05.wait::ld) and fenced before the epilogue
            // threads arrived on the barrier this thread has just seen complete; the releasing
            // form took the relay 1100 clk per arrive, on the path of the next tile's MMAs.
            uint32_t lt = 0;
            for (int tile = cluster_id; tile < ntiles && !lds32(abort_flag); tile += nclusters, ++lt) {
                if (!ROT) {
                    const int acc = (int)(lt % NACC);
                    const uint32_t aph = (lt / NACC) & 1u;
                    if (lt >= (uint32_t)NACC) {
                        mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, g.status);
                        mbar_arrive_cluster_relaxed(map_to_cta(bar_peer_tempty(acc), 0));
                    }
                } else {
                    const int lo = (int)(lt & 1u);
                    if (lt >= 2u) {
                        mbar_wait(bar_tempty(lo), ((lt >> 1) & 1u) ^ 1u, abort_flag, g.status);
                        mbar_arrive_cluster_relaxed(map_to_cta(bar_peer_tempty(lo), 0));
                    }
                    if (lt >= 1u) {
                        mbar_wait(bar_tempty(2), (lt & 1u) ^ 1u, abort_flag, g.status);
                        mbar_arrive_cluster_relaxed(map_to_cta(bar_peer_tempty(2), 0));
                    }
                }
            }
        }
    } else if (warp < 2 + UW) {
        // ------------------------------------------------------------ unpack warps
        const int grp = (warp - 2) / WPG;               // takes the stages with it % G == grp
        const int gt = threadIdx.x - 64 - grp * GT;     // 0..127 inside the group
        const int q = warp & 3;                         // TMEM lane quarter of this warp
        const int arow = q * 32 + lane;                 // row of A owned by this thread
        const uint32_t a_sw = (uint32_t)((arow >> 1) & 3);            // 64-byte TMA swizzle
        const uint32_t a_off = (uint32_t)(arow * PROW);
        const uint32_t a_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)ACOL0;
        const uint32_t full_u_leader = map_to_cta(bar_full_u(0), 0);  // barrier in the leader CTA
        // per-thread, stage-independent offsets: my four packed chunks of A (swizzled), my
        // packed chunks of Bt and where their two unpacked halves go
        uint32_t a_ld[4], b_ld[NTB], b_lo[NTB], b_hi[NTB];
#pragma unroll
        for (int c = 0; c < 4; ++c) a_ld[c] = a_off + (((uint32_t)c ^ a_sw) << 4);
#pragma unroll
        for (int j = 0; j < NTB; ++j) {
            const int id = gt + j * GT;
            const int r = id >> 2, c = id & 3, sw = r & 7;
            b_ld[j] = (uint32_t)(PA + r * PROW + c * 16);
            b_lo[j] = (uint32_t)(r * UROW + (((2 * c) ^ sw) << 4));
            b_hi[j] = (uint32_t)(r * UROW + (((2 * c + 1) ^ sw) << 4));
        }
        // Stages are numbered across tiles (every tile has nslab of them, so stage s of my
        // lt-th tile is number lt * nslab + s); this group takes the numbers congruent to grp
        // mod G, and carries its packed-ring slot and phase from one stage to the next.
        int psum_a = 0;
        int psum_b[NTB];
        // One stage.  All four 32-deep steps are always expanded and multiplied: past the end
        // of a ragged depth the TMA loads filled both operands with zeros, which add nothing
        // to the products or to the depth sums.
        auto unpack_stage = [&](uint32_t it, int pst, uint32_t pph) {
            const int ust = (int)(it % US);
            mbar_wait(bar_full_p(pst), pph, abort_flag, g.status);
            const uint32_t ps = sbase + OFF_P + pst * PSTAGE;
            // all shared-memory loads first, so their latencies overlap
            uint4 wa[4], wb[NTB];
#pragma unroll
            for (int c = 0; c < 4; ++c)
                wa[c] = lds128(ps + a_ld[c]);
#pragma unroll
            for (int j = 0; j < NTB; ++j)
                wb[j] = lds128(ps + b_ld[j]);
            // Bt first: with 192 columns its shared-memory ring is twice as deep as the
            // tensor-memory ring of A, so this wait is normally over and the work hides behind
            // the MMAs
            {
                const int bst = (int)(it % BS);
                mbar_wait(bar_empty_b(bst), ((it / BS) & 1u) ^ 1u, abort_flag, g.status);
                const uint32_t us = sbase + OFF_B + bst * BSTAGE;
#pragma unroll
                for (int j = 0; j < NTB; ++j) {
                    uint4 lo, hi;
                    unpack16(wb[j], lo, hi);
                    if (need_cb) psum_b[j] = chunk_sum(lo, hi, psum_b[j]);
                    sts128(us + b_lo[j], lo);
                    sts128(us + b_hi[j], hi);
                }
            }
            // A: expand my row in registers, then wait for its tensor-memory stage
            uint4 alo[4], ahi[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                unpack16(wa[c], alo[c], ahi[c]);
                if (need_ra) psum_a = chunk_sum(alo[c], ahi[c], psum_a);
            }
            // my A slot was last used by stage it - US, whose MMAs' commit arrived on the
            // Bt ring's barrier of that stage
            if (it >= (uint32_t)US)
                mbar_wait(bar_empty_b((it - US) % BS), ((it - US) / BS) & 1u, abort_flag, g.status);
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t r8[8] = {alo[c].x, alo[c].y, alo[c].z, alo[c].w,
                                        ahi[c].x, ahi[c].y, ahi[c].z, ahi[c].w};
                tc_st8(a_taddr + (uint32_t)(ust * 32 + 8 * c), r8);
            }
            tc_wait_st();                 // my tensor-memory stores are complete
            fence_async_smem();           // my shared-memory stores are visible to the MMA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_cluster_relaxed(full_u_leader + 8u * (uint32_t)ust);
                mbar_arrive_relaxed(bar_empty_p(pst));
            }
        };
        uint32_t lt = 0, it = (uint32_t)grp, pph = 0;
        int pst = grp % PS;
        for (int tile = cluster_id; tile < ntiles && !lds32(abort_flag); tile += nclusters, ++lt) {
            psum_a = 0;
#pragma unroll
            for (int j = 0; j < NTB; ++j) psum_b[j] = 0;
            const uint32_t it_end = (lt + 1) * (uint32_t)p.nslab;
            for (; it < it_end; it += G) {
                unpack_stage(it, pst, pph);
                pst += G;
                if (pst >= PS) { pst -= PS; pph ^= 1u; }
            }
            if (need_sums) {
                const int acc = (int)(lt % NACC);
                const uint32_t aph = (lt / NACC) & 1u;
                // both CTAs' epilogues NACC tiles back are done with this sums buffer
                mbar_wait(bar_tstart(acc), aph, abort_flag, g.status);
                const uint32_t mine = sums_s + 4 * ((acc * G + grp) * SUMS_N);
                sts32(mine + 4 * arow, psum_a);
#pragma unroll
                for (int j = 0; j < NTB; ++j) {
                    int t = psum_b[j];
                    t += __shfl_xor_sync(0xFFFFFFFFu, t, 1);
                    t += __shfl_xor_sync(0xFFFFFFFFu, t, 2);
                    const int id = gt + j * GT;
                    if ((id & 3) == 0) {
                        // column sum of one of my rows of Bt: both CTAs need it.  Tile column
                        // of my row r: my run of BH rows, or (ROT) one of my two runs of 64
                        const int r = id >> 2;
                        const int col = !ROT ? (int)rank * BH + r
                                             : (r < C::BBOX ? (int)rank * C::BBOX + r : BH + (int)rank * C::BBOX + r - C::BBOX);
                        const uint32_t a = mine + 4 * (TMC + col);
                        sts32(a, t);
                        sts32_cluster(map_to_cta(a, peer), t);
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    if (need_cb) {
                        mbar_arrive_cluster(map_to_cta(bar_sums(acc), rank));
                        mbar_arrive_cluster(map_to_cta(bar_sums(acc), peer));
                    } else {
                        mbar_arrive(bar_sums(acc));       // row sums stay in this CTA
                    }
                }
            }
        }
        // The last tile of this CTA pair has no next tile to hide its epilogue behind, and the
        // unpack warps are idle from its last stages on: each of them drains two of the tile's
        // chunks in its own lane quarter (the epilogue warp of the quarter takes the first
        // two).  Staging slices: the packed ring, which nothing reads or fills any more once an
        // accumulator (half) is complete -- every stage of the tile has been expanded by then.
        if (lt > 0 && !lds32(abort_flag)) {
            const uint32_t ltf = lt - 1;
            const int tile = cluster_id + (int)ltf * nclusters;
            const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
            const int acc = (int)(ltf % NACC);
            const uint32_t aph = (ltf / NACC) & 1u;
            const int m = tm * 256 + (int)rank * TMC + arow;
            const int n0 = tn * BNC;
            mbar_wait(bar_final, 0, abort_flag, g.status);
            int ra = 0;
            if (need_ra) {
                const uint32_t s0 = sums_s + 4 * (acc * G * SUMS_N);
#pragma unroll
                for (int gi = 0; gi < G; ++gi) ra += lds32(s0 + 4 * (gi * SUMS_N + arow));
            } else if (m < g.M) {
                ra = g.rowsum_a[m];
            }
            const uint32_t rowterm = (uint32_t)0 - (uint32_t)(g.zb * ra);
            const uint32_t taddr0 = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ROT ? 0 : acc * BNC);
#pragma unroll 1
            for (int k = 0; k < 2; ++k) {
                const int ci = 2 * (grp + 1) + k;              // in the epilogue's drain order
                if (ci >= BNC / 32) break;
                const int ch = ROT ? ((ci + BNC / 64) & (BNC / 32 - 1)) : ci;
                const int nc = n0 + ch * 32;
                const uint32_t tcol = (ROT && ch < BNC / 64 && (ltf & 1u)) ? 256u + (uint32_t)(ch * 32) : (uint32_t)(ch * 32);
                mbar_wait(bar_tfull(ROT ? (ci < BNC / 64 ? 1 : 0) : acc), aph, abort_flag, g.status);
                tc_fence_after();
                if (nc < g.N)              // warp-uniform
                    drain_chunk(taddr0 + tcol, ch, nc, q, tm, m, ra, rowterm,
                                sbase + OFF_P + (uint32_t)((2 * (warp - 2) + k) * 4096), 0, false);
            }
            tc_fence_before();
            if (!REQUANT && p.c_tma && lane == 0) bulk_wait_read();  // my TMA stores have read their slices; their writes complete with the grid
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const int et = threadIdx.x - (2 + UW) * 32;
        uint32_t lt = 0, nstore = 0;            // tiles taken, chunks drained by my warp
        for (int tile = cluster_id; tile < ntiles && !lds32(abort_flag); tile += nclusters, ++lt) {
            const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
            const int acc = (int)(lt % NACC);
            const uint32_t aph = (lt / NACC) & 1u;
            const int m = tm * 256 + (int)rank * TMC + row;
            const int n0 = tn * BNC;
            if (need_cb) mbar_wait_cl(bar_sums(acc), aph, abort_flag, g.status);      // the peer's stores are read below
            else if (need_ra) mbar_wait(bar_sums(acc), aph, abort_flag, g.status);
            const uint32_t s0 = sums_s + 4 * (acc * G * SUMS_N);
            for (int j = et; j < BNC; j += 128) {
                const int n = n0 + j;
                int cb = 0, bias = 0, zbn = pc ? 0 : g.zb;
                if (n < g.N) {
                    if (need_cb) {
#pragma unroll
                        for (int gi = 0; gi < G; ++gi) cb += lds32(s0 + 4 * (gi * SUMS_N + TMC + j));
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
                    sts32(pc_s + 4 * (BNC + j), mult);
                    sts32(pc_s + 4 * (2 * BNC + j), pc_fast ? (1 << (s - 1)) + (g.rq.zo - g.rq.lo) * (1 << s) : 0);
                    sts32(pc_s + 4 * (3 * BNC + j), s);
                }
            }
            int ra = 0;
            if (need_ra) {
#pragma unroll
                for (int gi = 0; gi < G; ++gi) ra += lds32(s0 + 4 * (gi * SUMS_N + row));
            } else if (m < g.M) {
                ra = g.rowsum_a[m];
            }
            const uint32_t rowterm = (uint32_t)0 - (uint32_t)(g.zb * ra);
            asm volatile("bar.sync 1, 128;" ::: "memory");
            // My CTA pair's last tile: the unpack warps have nothing left to expand and drain
            // all chunks but the first two of every lane quarter (see the end of their branch).
            const bool last_tile = tile + nclusters >= ntiles;
            if (last_tile) mbar_arrive(bar_final);

            // ROT: barrier 1 = this tile's upper half is complete, barrier 0 = all of it
            mbar_wait(bar_tfull(ROT ? 1 : acc), aph, abort_flag, g.status);
            tc_fence_after();
            const uint32_t taddr0 = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(ROT ? 0 : acc * BNC);
#pragma unroll 1
            for (int ci = 0; ci < (last_tile ? 2 : BNC / 32); ++ci) {
                // ROT: the upper half (the middle buffer, which the next tile needs first), then
                // the lower half in this tile's outer buffer
                const int ch = ROT ? ((ci + BNC / 64) & (BNC / 32 - 1)) : ci;
                const int nc = n0 + ch * 32;
                const uint32_t tcol = (ROT && ch < BNC / 64 && (lt & 1u)) ? 256u + (uint32_t)(ch * 32) : (uint32_t)(ch * 32);
                if (ROT && ci == BNC / 64 - 1) {
                    // Last chunk of the upper half.  The whole tile must be seen complete before
                    // the middle buffer is handed back: once it is, the next tile may complete too
                    // (a short depth), and a wait for this tile's parity would then miss it.  The
                    // tile's last MMAs ended long ago (they ran while the first chunks were drained).
                    mbar_wait(bar_tfull(0), aph, abort_flag, g.status);
                    tc_fence_after();
                    if (nc >= g.N) {       // a chunk past the last column: nothing to read
                        tc_fence_before();
                        mbar_arrive(bar_tempty(2));
                    }
                }
                if (nc < g.N) {            // warp-uniform
                    // Two staging slices alternate by the count of chunks drained, not by the
                    // chunk's position: a tile whose last columns lie past N drains an odd number
                    // of chunks, and "all but the latest store have read their slice" protects a
                    // slice only if the latest store used the other one.
                    drain_chunk(taddr0 + tcol, ch, nc, lg, tm, m, ra, rowterm,
                                sbase + OFF_STG + (uint32_t)(((NSTG > 1 ? (nstore & 1u) : 0u) * 4 + (uint32_t)lg) * 4096),
                                NSTG > 1 ? 2 : 1, ci == BNC / 64 - 1);
                    ++nstore;
                }
            }
            tc_fence_before();
            mbar_arrive(bar_tempty(ROT ? (int)(lt & 1u) : acc));
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        if (!REQUANT && p.c_tma && lane == 0) bulk_wait_read();  // my TMA stores have read their slices; their writes complete with the grid
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
                     int box_rows, bool swizzle64);

bool gemm_tc_pair_supported(const GemmParams& p)
{
    return gemm_tc_supported(p) && p.M >= 256 && p.N >= 192;
}

template <int BNC, int NSTG, bool RQ>
static q4_status launch_pair_t(const pair::Params& p, const CUtensorMap& tmA, const CUtensorMap& tmB,
                               const CUtensorMap& tmC, long long tiles, cudaStream_t st)
{
    static int max_clusters_dev[64] = {};     // per device (and per instance of this template)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return Q4_ERR_CUDA;
    int& max_clusters = max_clusters_dev[dev];
    auto kernel = pair::gemm_tc_pair_kernel<BNC, NSTG, RQ>;
    constexpr int SMEM = pair::Cfg<BNC, NSTG>::SMEM;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel waits before it touches memory
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(pair::NTHREADS);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (!max_clusters) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) !=
            cudaSuccess) return Q4_ERR_CUDA;
        int sms = 148, n = 0;
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC, p);
    count_launch();
    return e == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                             CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                             CUtensorMapFloatOOBfill);
static EncodeFn encode_fn()
{
    static EncodeFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) !=
                cudaSuccess || qres != cudaDriverEntryPointSuccess) return nullptr;
        fn = reinterpret_cast<EncodeFn>(sym);
    }
    return fn;
}

// int32 C [M x N], pitch ldc elements: box = 32 columns (128 bytes) x 32 rows, read from a
// 128-byte-swizzled shared-memory tile.
static bool make_c_map(CUtensorMap* tm, int32_t* base, int64_t ldc, int rows, int cols)
{
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ldc * 4};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, base, dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same map for other translation units.
bool make_c32_map(CUtensorMap* tm, int32_t* base, int64_t ldc, int rows, int cols)
{
    return make_c_map(tm, base, ldc, rows, cols);
}

// Tile width for a problem: estimated clocks of the busiest CTA pair with either width, from
// measured stage and epilogue times (192 columns: 520 clk per 128-deep stage, epilogues
// overlapped but the last; 256 columns: 540 clk per stage, 4200 clk per tile of exposed
// half drain and pipeline restart, 2500 clk for the last tile's drain).  Checked against forced
// widths at 1536^3, 2048^3, 3072^3, 4096^3, 4096 x 11008 x 4096, 6144^3, 8192^3.
int gemm_tc_pair_width(const GemmParams& g)
{
    const long long nslab = ((g.K + 1) / 2 + pair::PROW - 1) / pair::PROW;
    const long long tm = ((long long)g.M + 255) / 256;
    const long long t192 = tm * (((long long)g.N + 191) / 192), t256 = tm * (((long long)g.N + 255) / 256);
    const long long pairs = 74;
    const long long c192 = (t192 + pairs - 1) / pairs * nslab * 520 + 5000;
    const long long c256 = (t256 + pairs - 1) / pairs * (nslab * 540 + 4200) + 2500;
    return c256 < c192 ? 256 : 192;
}

template <int BNC, int NSTG>
static q4_status launch_pair_w(const GemmParams& g, bool rq, cudaStream_t st)
{
    using C = pair::Cfg<BNC, NSTG>;
    pair::Params p;
    p.g = g;
    p.tiles_m = (g.M + 255) / 256;
    p.tiles_n = (g.N + BNC - 1) / BNC;
    const int kbytes = (g.K + 1) / 2;
    p.nslab = (kbytes + pair::PROW - 1) / pair::PROW;
    p.c_vec = (!rq && ((uintptr_t)g.C % 16 == 0) && (g.ldc % 4 == 0)) ? 1 : 0;
    p.cq_vec = (rq && ((uintptr_t)g.Cq % 16 == 0) && (g.ldcq % 16 == 0)) ? 1 : 0;
    CUtensorMap tmA, tmB, tmC;
    if (!make_packed_map(&tmA, g.A, g.lda, g.M, kbytes, pair::TMC, true)) return Q4_ERR_CUDA;
    p.c_tma = 0;
    tmC = CUtensorMap{};
    if (p.c_vec) {
        if (!make_c_map(&tmC, g.C, g.ldc, g.M, g.N)) return Q4_ERR_CUDA;
        p.c_tma = 1;
    }
    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    if (!make_packed_map(&tmB, g.Bt, g.ldb, g.N, kbytes, C::BBOX, false)) return Q4_ERR_CUDA;
    return rq ? launch_pair_t<BNC, NSTG, true>(p, tmA, tmB, tmC, tiles, st)
              : launch_pair_t<BNC, NSTG, false>(p, tmA, tmB, tmC, tiles, st);
}

q4_status launch_gemm_tc_pair(const GemmParams& g, bool rq, cudaStream_t st, int width)
{
    if (width != 192 && width != 256) width = gemm_tc_pair_width(g);
    if (width == 192) return launch_pair_w<192, 2>(g, rq, st);
    return launch_pair_w<256, 1>(g, rq, st);
}

}  // namespace q4
