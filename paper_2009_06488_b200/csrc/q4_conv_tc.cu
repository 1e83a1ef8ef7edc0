// Fused quantized convolution layer on the tensor-memory path: GEMM-based convolution
// (Section I; depth D = kh*kw*c, Section III-A) as an implicit GEMM on tcgen05.mma
// kind::i8, the unrolled matrix never written to memory.
//
// One GEMM row covers P horizontally adjacent output pixels.  Its depth is the union
// of their receptive fields -- KH window rows of ((P-1)*sw + KW) input pixels -- and its
// P*OC columns are (pixel, output channel) pairs; the weight matrix B holds w - zb where
// a window column is one of the pixel's taps and 0 elsewhere.  On this machine one
// tcgen05.mma of 128 rows costs the same 64 clocks for any width up to 128 columns, so
// the structural zeros are free, while the rows to build, the pixels to decode and the
// MMAs to issue per output pixel all shrink by about P.
//
// Zero points.  B holds signed bytes w - zb (the MMA takes a signed 8-bit B operand), so the
// product is sum a*(w - zb) = sum a*w - zb*sum a: Eq. 2's row-sum term is absorbed and
// never formed.  What is left of Eq. 3 is one constant per output channel,
// K*za*zb - za*sum w + bias, which the accumulator columns are preloaded with.
//
// Roles (one persistent CTA per SM):
//   warps 0..3    producers (tiles in turn): copy the input rows a tile touches into a ring
//                 of shared-memory buffers -- dense rows, one bulk copy per image and tile --
//                 and fill the rows above / below the image with the input zero point
//   warp 4        MMA issuer: KS instructions of 128 x N x 32 per tile, A from tensor
//                 memory, B from shared memory
//   4*G workers   G groups of four warps (one warp per tensor-memory lane quarter), each
//                 taking every G-th tile from its staged copy to its packed output: a thread
//                 owns one GEMM row; it reads its window rows with the widest aligned
//                 loads, replaces the words left or right of the image by the zero point,
//                 splits the nibbles into bytes (even nibbles, then odd ones, of each 32-bit
//                 word -- B uses the same depth order), writes them to tensor memory
//                 (tcgen05.st), preloads its accumulator columns with the per-channel
//                 constants, hands the tile to the MMA warp, and when the product is there
//                 reads it back (tcgen05.ld), re-quantizes, packs and stores 16 bytes per 32
//                 values (a row's P*OC/2 output bytes are contiguous).
// A group works through its tiles one after the other; the groups overlap one another, so
// while one waits for its product the others keep the issue slots busy.
//
// Every mbarrier wait is bounded; a role whose wait runs out leaves its loop, the others
// follow with short waits, and all meet at the common exit where tensor memory is freed.
#include <cuda.h>

#include "q4_common.cuh"
#include "q4_conv_stage.cuh"
#include "q4_requant8.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {

unsigned* device_status_ptr();     // the device status word (q4_api.cu)

namespace convtc {

using fused::Params;

constexpr int NBMAX = 8;           // staged input buffers: at most this many, at least 3
#ifndef Q4_CTC_SUSPEND
#define Q4_CTC_SUSPEND 1
#endif
#ifndef Q4_CTC_PWN
#define Q4_CTC_PWN 3
#endif
constexpr int PWN = Q4_CTC_PWN;     // producer warps
constexpr int ROWS = 128;          // GEMM rows per tile (UMMA M)
constexpr int SMEM_LIMIT = 200 * 1024;
constexpr int SMEM_LIMIT_WIDE = 224 * 1024;

__host__ __device__ constexpr int pow2_at_least(int v) { int r = 32; while (r < v) r *= 2; return r; }

// CW: 32-bit words per input pixel (C / 8), 0 = single-channel input (pixels are nibbles).
// PH: position (in words, mod 4) of a row's first window word in its 16-byte line -- the
// same for every row because P*sw*unit is a multiple of 16 bytes --, which fixes where
// 16- and 8-byte loads apply.
template <int CW_, int SW_, int KW_, int KH_, int P_, int OC_, int PH_>
struct Shape {
    static constexpr int CW = CW_, SW = SW_, KW = KW_, KH = KH_, P = P_, OC = OC_, PH = PH_;
    static constexpr bool NIB = (CW == 0);
    static constexpr int C = NIB ? 1 : 8 * CW;
    static constexpr int COLS = (P - 1) * SW + KW;            // input columns of a row's window
    static constexpr int WW = NIB ? (COLS + 7) / 8 : COLS * CW;   // packed words per window row
    static constexpr int NW = KH * WW;                        // packed words per GEMM row
    // 32-byte depth steps.  The words past NW carry the per-channel constants of Eq. 3 into
    // the product (their A bytes are the same for every row: 1, then 255s; their B bytes the
    // constant's digits d0 + 255 * (d1 + d2 + ...), signed bytes): a layer whose depth fills
    // its last step gets one step more.
    static constexpr int KS = NW / 4 + 1;
    static constexpr int SPARE = KS * 4 - NW;                 // 1..4 words = 8 * SPARE bytes
    static constexpr int QMAX = (8 * SPARE - 1) * 127;        // largest |d1 + d2 + ...|
    static constexpr int N = P * OC;
    static constexpr int ACCW = N < 32 ? 32 : N;
    static constexpr int ACOLS = KS * 8;                      // tensor-memory columns of one A tile
    static constexpr int NKB = (KS + 3) / 4;                  // 128-byte depth blocks of B
    static constexpr int B_BYTES = NKB * N * 128;
    static constexpr int TILE = ROWS * P;                     // output pixels per tile
    static_assert(N % 32 == 0 && N <= 256, "UMMA N, and the epilogue reads 32 columns at a time");
    static_assert((N * 128) % 1024 == 0, "depth blocks of B start on swizzle-atom boundaries");
};

constexpr int GMAX = 6;             // worker groups
constexpr int NBAR = 2 * NBMAX + 2 * GMAX + 2;      // (an even count keeps what follows 16-byte aligned)
template <class S> struct Layout {
    static constexpr int OFF_B = 0;
    static constexpr int OFF_CT = OFF_B + S::B_BYTES;         // int32 [N] per-column constants
    static constexpr int OFF_PC = OFF_CT + S::N * 4;          // int32 [3][N] per-column multiplier, rounding, shift
    static constexpr int OFF_GEO = OFF_PC + 3 * S::N * 4;     // int4 [NBMAX]
    static constexpr int OFF_BAR = OFF_GEO + NBMAX * 16;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;       // tensor-memory base, abort flag
    static constexpr int OFF_BUF = OFF_MISC + 16;
    static constexpr int FIXED = OFF_BUF + 1024;              // + slack to align the base
};

__device__ __forceinline__ uint2 lds64(uint32_t a)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}

// Words I .. WW-1 of a window row whose word 0 sits at shared address `addr`, PH words
// into its 16-byte line: 16-byte loads where a group of four is aligned, 8-byte loads
// where a pair is, single words elsewhere.
template <int I, int WW, int PH>
__device__ __forceinline__ void load_row(uint32_t addr, uint32_t* w)
{
    if constexpr (I < WW) {
        constexpr int pos = PH < 0 ? 1 : PH + I;
        if constexpr (PH >= 0 && pos % 4 == 0 && I + 4 <= WW) {
            const uint4 v = lds128(addr + 4 * I);
            w[I] = v.x; w[I + 1] = v.y; w[I + 2] = v.z; w[I + 3] = v.w;
            load_row<I + 4, WW, PH>(addr, w);
        } else if constexpr (PH >= 0 && pos % 2 == 0 && I + 2 <= WW) {
            const uint2 v = lds64(addr + 4 * I);
            w[I] = v.x; w[I + 1] = v.y;
            load_row<I + 2, WW, PH>(addr, w);
        } else {
            w[I] = (uint32_t)lds32(addr + 4 * I);
            load_row<I + 1, WW, PH>(addr, w);
        }
    }
}

// Development aid (-DQ4_CTC_TRACE): clock stamps of the first tiles of CTA 0, per role.
#ifdef Q4_CTC_TRACE
__device__ long long* g_trace = nullptr;
#define TR(role, k, slot) \
    do { if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && (k) < 24 && g_trace) \
             g_trace[(((role) * 24 + (k)) << 3) + (slot)] = clock64(); } while (0)
#else
#define TR(role, k, slot) do { } while (0)
#endif

// A wait of a warp that has nothing else to do until the barrier completes.
__device__ __forceinline__ bool wait_idle(uint32_t bar, uint32_t parity, uint32_t abort_flag, unsigned* status)
{
#if Q4_CTC_SUSPEND
    return mbar_wait_suspend(bar, parity, abort_flag, status);
#else
    return mbar_wait(bar, parity, abort_flag, status);
#endif
}

__device__ __forceinline__ void cp_async8(uint32_t dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4s(uint32_t dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

// One image's share ("segment") of a tile's staged rows: staged rows [ss, ss + cnt) hold
// input rows ih0 .. ih0 + cnt - 1 of image n; [lo, hi) of them lie inside the image.
struct Segment {
    int ss, cnt, lo, hi;
    int64_t row0;                                      // n * H + ih0 (meaningful where inside the image)
};
__device__ __forceinline__ Segment tile_segment(const Params& p, const fused::Geo& g, int seg)
{
    Segment t;
    int ih0;
    if (seg == 0) {
        t.ss = 0;
        t.cnt = g.s0;
        ih0 = g.oh_first * p.sh - p.ph;
    } else {
        t.ss = g.s0 + (seg - 1) * p.sfull;
        t.cnt = g.nslots - t.ss < p.sfull ? g.nslots - t.ss : p.sfull;
        ih0 = -p.ph;
    }
    t.lo = ih0 < 0 ? -ih0 : 0;
    t.hi = p.H - ih0 < t.cnt ? p.H - ih0 : t.cnt;
    if (t.lo > t.cnt) t.lo = t.cnt;
    if (t.hi < t.lo) t.hi = t.lo;
    t.row0 = (int64_t)(g.n_first + seg) * p.H + ih0;
    return t;
}

// A producer warp's loop.  Tile j lives in buffer j % nb; producer warp i stages the tiles
// j = i, i + PWN, ...  The staged rows are dense (one image row after the other, no halo
// columns: the workers replace the few window words that fall left or right of the image),
// so the input rows of one image that a tile touches are one contiguous run in memory and
// in the buffer: ONE bulk copy per image and tile where rows are whole 16-byte pieces (a
// bulk copy costs its issuing warp about a hundred clocks, whatever its size), else a run of
// 8- or 4-byte asynchronous copies.  Staged rows above or below the image are filled with
// the zero point by ordinary stores.  A buffer is refilled once the worker group that had
// it has reported (on its "read" mbarrier) that it is done with the tile that was there.
// A tile is announced on the buffer's "landed" mbarrier by the bulk copies themselves, or
// by lane 0 once this warp's asynchronous copies of it have landed, which is checked after
// the warp's next tile has been issued so that copies stay in flight.  The tile's geometry
// is written before the arrive that publishes it.
__device__ __forceinline__ void producer(const Params& p, int mytiles, int nb, int pwi, uint8_t* buf0,
                                         int4* geo_s, uint32_t full0, uint32_t empty0, uint32_t abort_flag,
                                         int lane, int64_t tile0, int64_t tstride, int npw = PWN)
{
    const bool bulk = p.vec16;
    const uint32_t zfill = (uint32_t)p.za * 0x11111111u;
    const int rowwords = p.rowbytes >> 2;
    int b = pwi, prev_b = -1;                          // j % nb (nb > npw), buffer of my previous tile
    uint32_t round = 0;                                // j / nb
    for (int j = pwi; j < mytiles; j += npw) {
        TR(0, j, 0);
        if (round > 0 && !wait_idle(empty0 + 8 * b, (round - 1) & 1, abort_flag, p.status)) return;
        TR(0, j, 1);
        const fused::Geo gn = fused::tile_geometry(p, tile0 + (int64_t)j * tstride);      // my j-th tile
        if (lane == 0) geo_s[b] = make_int4(gn.n_first, gn.oh_first, gn.s0, gn.nslots);
        const int nseg = gn.nslots <= gn.s0
            ? 1 : 1 + (int)fdiv((uint32_t)(gn.nslots - gn.s0 + p.sfull - 1), p.div_sfull);
        uint8_t* rows = buf0 + b * p.bufbytes + 16;
        if (bulk) {
            // ordinary accesses to this buffer (earlier border rows, the workers' reads)
            // come before the copy engine's writes
            fence_async_smem();
            uint32_t bytes = 0;
            for (int seg = lane; seg < nseg; seg += 32) {
                const Segment t = tile_segment(p, gn, seg);
                bytes += (uint32_t)(t.hi - t.lo) * (uint32_t)p.rowbytes;
                for (int r = 0; r < t.cnt; ++r) {
                    if (r == t.lo) { r = t.hi; if (r >= t.cnt) break; }
                    uint4* dst = reinterpret_cast<uint4*>(rows + (t.ss + r) * p.rowbytes);
                    for (int c = 0; c < p.rowbytes / 16; ++c) dst[c] = make_uint4(zfill, zfill, zfill, zfill);
                }
            }
            bytes = __reduce_add_sync(0xFFFFFFFFu, bytes);     // also orders the fills before lane 0's arrive
            if (lane == 0) mbar_expect_tx(full0 + 8 * b, bytes);
            __syncwarp();
            for (int seg = lane; seg < nseg; seg += 32) {
                const Segment t = tile_segment(p, gn, seg);
                if (t.hi > t.lo)
                    fused::bulk_load_row(smem_u32(rows + (t.ss + t.lo) * p.rowbytes),
                                         p.X + (t.row0 + t.lo) * p.rowbytes,
                                         (uint32_t)(t.hi - t.lo) * (uint32_t)p.rowbytes, full0 + 8 * b);
            }
        } else {
            for (int seg = 0; seg < nseg; ++seg) {
                const Segment t = tile_segment(p, gn, seg);
                uint32_t* top = reinterpret_cast<uint32_t*>(rows + t.ss * p.rowbytes);
                for (int i = lane; i < t.lo * rowwords; i += 32) top[i] = zfill;
                uint32_t* bot = reinterpret_cast<uint32_t*>(rows + (t.ss + t.hi) * p.rowbytes);
                for (int i = lane; i < (t.cnt - t.hi) * rowwords; i += 32) bot[i] = zfill;
                const uint32_t dst = smem_u32(rows + (t.ss + t.lo) * p.rowbytes);
                const uint8_t* src = p.X + (t.row0 + t.lo) * p.rowbytes;
                const int runbytes = (t.hi - t.lo) * p.rowbytes;
                if (p.cpr == 8) {
                    for (int o = 8 * lane; o < runbytes; o += 256) cp_async8(dst + o, src + o);
                } else {
                    for (int o = 4 * lane; o < runbytes; o += 128) cp_async4s(dst + o, src + o);
                }
            }
            fused::cp_async_commit();
            fused::cp_async_wait_group<1>();           // my previous tile has landed
            __syncwarp();
            if (prev_b >= 0 && lane == 0) mbar_arrive(full0 + 8 * prev_b);
            prev_b = b;
        }
        TR(0, j, 2);
        b += npw;
        if (b >= nb) { b -= nb; ++round; }
    }
    if (!bulk) {
        fused::cp_async_wait_group<0>();
        __syncwarp();
        if (prev_b >= 0 && lane == 0) mbar_arrive(full0 + 8 * prev_b);
    }
}

// PC: per-channel weight zero points, multipliers and shifts (an instance of its own, so that
// the per-tensor form keeps its registers).
template <class S, int G, bool PC>
__global__ void __launch_bounds__((PWN + 1 + 4 * G) * 32, 1)
conv_tc_kernel(const Params p)
{
    using L = Layout<S>;
    constexpr int THREADS = (PWN + 1 + 4 * G) * 32;
    constexpr int N = S::N, KS = S::KS, WW = S::WW, P = S::P, OC = S::OC;
    constexpr int TMEM_COLS = pow2_at_least(G * (S::ACCW + S::ACOLS));
    static_assert(G >= 1 && G <= GMAX && G * (S::ACCW + S::ACOLS) <= 512, "tensor memory budget");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    int32_t* colterm = reinterpret_cast<int32_t*>(smem + L::OFF_CT);
    const uint32_t colterm_s = sbase + L::OFF_CT;
    int4* geo_s = reinterpret_cast<int4*>(smem + L::OFF_GEO);
    const uint32_t bar0 = sbase + L::OFF_BAR;
    const uint32_t full0 = bar0, empty0 = bar0 + 8 * NBMAX;
    auto bar_a_ready  = [&](int g) { return bar0 + 8u * (uint32_t)(2 * NBMAX + g); };
    auto bar_mma_done = [&](int g) { return bar0 + 8u * (uint32_t)(2 * NBMAX + GMAX + g); };
    const uint32_t bar_prep = bar0 + 8u * (uint32_t)(2 * NBMAX + 2 * GMAX);     // a prepared weight image has landed
    const int NB = p.nbuf;
    const uint32_t tmem_slot = sbase + L::OFF_MISC, abort_flag = sbase + L::OFF_MISC + 4;
    const uint32_t preload_flag = sbase + L::OFF_MISC + 8;
    const uint32_t pcslow_flag = sbase + L::OFF_MISC + 12;        // per-channel: some shift needs the 64-bit form
    const uint32_t pc_s = sbase + L::OFF_PC;
    int32_t* pcv = reinterpret_cast<int32_t*>(smem + L::OFF_PC);
    constexpr bool pc = PC;
    uint8_t* buf0 = smem + L::OFF_BUF;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- once per CTA -------------------------------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < NB; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, 4);          // the four warps of the group that took the tile
        }
        for (int g = 0; g < G; ++g) {
            mbar_init(bar_a_ready(g), 4);
            mbar_init(bar_mma_done(g), 1);
        }
        mbar_init(bar_prep, 1);
        sts32(abort_flag, 0);
        sts32(preload_flag, 0);
        sts32(pcslow_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == PWN) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(tmem_slot), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();                       // barriers initialised, tensor memory allocated
    tc_fence_after();
    // The kernel is launched with programmatic stream serialization: everything above may
    // run while the previous kernel of the stream is still finishing.  Nothing below -- no
    // read of the operands, no write of the output -- happens before that kernel has
    // completed and its writes are visible; the kernel after this one may begin its own
    // prologue from here on.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t ntiles = (p.M + S::TILE - 1) / S::TILE;
    int mytiles = (int)((ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x);
    const uint32_t M32 = (uint32_t)p.M;
    constexpr uint32_t IMAGE = (uint32_t)(S::B_BYTES + N * 4);     // B and the per-column constants, contiguous
    // A prepared weight image ends in {fallback flag, tag}.  An image with another tag (another
    // layer class, filter, channel counts, za or build) is not used: the launch does nothing and
    // the status word says why.
    uint2 trailer = make_uint2(0u, p.prep_tag);
    if (p.prep_in != nullptr) trailer = __ldg(reinterpret_cast<const uint2*>(p.prep_in + IMAGE));
    if (trailer.y != p.prep_tag) {
        mytiles = 0;
        if (tid == 0) atomicOr(p.status, kStatusWeightImage);
    }

    // The producers start copying the first tiles at once; meanwhile the other warps
    // prepare the weights (synchronising among themselves on a named barrier).
    uint32_t tmem_base = 0;
    bool use_preload = false;              // a constant beyond the digits' range: preloaded accumulators instead
    if (warp >= PWN && p.prep_in != nullptr) {
        // The weights were prepared ahead of time (the B operand, the constants, the flag):
        // one bulk copy brings them in; only the MMA warp has to wait for it.
        if (tid == PWN * 32 && mytiles > 0) {
            mbar_expect_tx(bar_prep, IMAGE);
            fused::bulk_load_row(sbase + L::OFF_B, p.prep_in, IMAGE, bar_prep);
        }
        use_preload = trailer.x != 0;
        tmem_base = (uint32_t)lds32(tmem_slot);
    } else if (warp >= PWN) {
        constexpr int NT = THREADS - PWN * 32;         // threads that prepare the weights
        constexpr int TASKS = N * KS * 4;              // eight-byte groups of B
        const int wt = tid - PWN * 32;
        auto sync_workers = [] { asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory"); };
        for (int i = wt; i < N; i += NT) colterm[i] = 0;
        sync_workers();
        // B: row n = (pixel px, channel oc); depth word wd = (window row kh, word i of it);
        // the word's eight nibbles are window nibbles 8i .. 8i+7, i.e. input column
        // j = nibble / C and channel c = nibble % C, which is tap kw = j - px*sw of pixel px
        // if that is a tap at all.  Even nibbles go to bytes 0..3, odd ones to bytes 4..7 of
        // the eight-byte group -- the order the workers give A.
        // Two passes: first every packed word this thread needs is requested (the loads'
        // latencies overlap), then the words are expanded and stored.
        constexpr int NIT = (TASKS + NT - 1) / NT;
        // where task idx finds its packed word: row n, depth word wd -> (valid, channel, tap, word)
        auto locate = [&](int idx, int& n, int& wd, int& px, int& oc, int& kh, int& i) {
            n = idx / (KS * 4); wd = idx - n * (KS * 4);
            px = n / OC;
            const int ocp = n - px * OC;
            oc = (ocp & ~7) + ch8(ocp & 7);            // the channel this column stands for
            kh = wd / WW; i = wd - kh * WW;
        };
        uint32_t wv[NIT];
        if constexpr (!S::NIB) {
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                const int idx = wt + it * NT;
                wv[it] = 0;
                int n, wd, px, oc, kh, i;
                locate(idx, n, wd, px, oc, kh, i);
                // word i of the window row is word cw of input column j: one packed word
                // of the weights where that column is a tap of pixel px
                const int j = i / S::CW, cw = i - j * S::CW;
                const int kw = j - px * S::SW;
                if (idx < TASKS && wd < S::NW && kw >= 0 && kw < S::KW) {
                    const uint8_t* src = p.Wt + (int64_t)oc * p.ldw + ((kh * S::KW + kw) * S::C) / 2 + 4 * cw;
                    if (p.wt_words) {
                        wv[it] = __ldg(reinterpret_cast<const uint32_t*>(src));
                    } else {
                        for (int q = 0; q < 4; ++q) wv[it] |= (uint32_t)__ldg(src + q) << (8 * q);
                    }
                }
            }
        }
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int idx = wt + it * NT;
            if (idx >= TASKS) break;
            int n, wd, px, oc, kh, i;
            locate(idx, n, wd, px, oc, kh, i);
            uint32_t lo = 0, hi = 0;
            int raw = 0;
            const int zbo = pc ? (p.zb_ch ? __ldg(p.zb_ch + oc) : 0) : p.zb;      // this channel's weight zero point
            if (wd < S::NW) {
                if constexpr (S::NIB) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int j = 8 * i + e;       // window column of this nibble
                        const int kw = j - px * S::SW;
                        if (kw >= 0 && kw < S::KW && j < S::COLS) {
                            const int nib = (int)fused::weight_nibble(p, oc, kh * S::KW + kw);
                            raw += nib;
                            const uint32_t byte = (uint32_t)(nib - zbo) & 0xFFu;
                            if (e & 1) hi |= byte << (8 * (e >> 1)); else lo |= byte << (8 * (e >> 1));
                        }
                    }
                } else {
                    const int j = i / S::CW;
                    const int kw = j - px * S::SW;
                    if (kw >= 0 && kw < S::KW) {
                        raw = nibble_sum(wv[it]);
                        lo = fused::sub_zb(wv[it] & 0x0F0F0F0Fu, (uint32_t)zbo);
                        hi = fused::sub_zb((wv[it] >> 4) & 0x0F0F0F0Fu, (uint32_t)zbo);
                    }
                }
            }
            if (wd < S::NW) {                          // (the words past the depth hold the constants' digits)
                const int kbyte = 8 * wd;
                uint8_t* dst = smem + L::OFF_B + (kbyte >> 7) * (N * 128) + n * 128 +
                               ((((kbyte & 127) >> 4) ^ (n & 7)) << 4) + (kbyte & 15);
                *reinterpret_cast<uint2*>(dst) = make_uint2(lo, hi);
            }
            if (px == 0 && !p.colsum_w && raw) atomicAdd(&colterm[oc], raw);     // every tap once
        }
        sync_workers();
        // per-column constant: what is left of Eq. 3 (column n = px*OC + oc)
        int cterm = 0;
        if (wt < OC) {
            const int cs = p.colsum_w ? p.colsum_w[wt] : colterm[wt];
            const int zbo = pc ? (p.zb_ch ? p.zb_ch[wt] : 0) : p.zb;
            cterm = (int)((uint32_t)(p.K * p.za * zbo) - (uint32_t)(p.za * cs) +
                          (uint32_t)(p.bias ? p.bias[wt] : 0));
            if (pc) {
                const int sh = p.shift_ch[wt];
                if (sh < 2 || sh > 27) sts32(pcslow_flag, 1);
            }
            int d0 = cterm % 255;
            if (d0 > 127) d0 -= 255;
            if (d0 < -127) d0 += 255;
            const int qd = (cterm - d0) / 255;
            if (qd > S::QMAX || qd < -S::QMAX) sts32(preload_flag, 1);
        }
        sync_workers();                    // every weight sum has been read, the flag is final
        use_preload = lds32(preload_flag) != 0;
        if (wt < OC) {
            // column position of channel wt within its group of eight: the inverse of ch8
            const int pos = (wt & ~7) + 2 * (wt & 3) + ((wt >> 2) & 1);
            int d0 = cterm % 255;
            if (d0 > 127) d0 -= 255;
            if (d0 < -127) d0 += 255;
            int qd = use_preload ? 0 : (cterm - d0) / 255;
            if (use_preload) d0 = 0;
            // the digits, eight per spare word (low four bytes, then high four)
            uint32_t dw[2 * S::SPARE];
#pragma unroll
            for (int i = 0; i < 2 * S::SPARE; ++i) {
                uint32_t word = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    int dgt;
                    if (i == 0 && b == 0) {
                        dgt = d0;
                    } else {
                        dgt = qd > 127 ? 127 : qd < -127 ? -127 : qd;
                        qd -= dgt;
                    }
                    word |= ((uint32_t)dgt & 0xFFu) << (8 * b);
                }
                dw[i] = word;
            }
            // per channel: multiplier, rounding constant, shift of every column of the channel
            int pmul = 0, prnd = 0, psh = 0;
            if (pc) {
                const bool pfast = lds32(pcslow_flag) == 0;
                const int sh = p.shift_ch[wt];
                pmul = p.mult_ch[wt];
                psh = pfast ? sh - 1 : sh;
                prnd = pfast ? (1 << (psh - 1)) + (p.rq.zo - p.rq.lo) * (1 << psh) : 0;
            }
            for (int px = 0; px < P; ++px) {
                const int n = px * OC + pos;
                colterm[n] = cterm;
                if (pc) {
                    pcv[n] = pmul;
                    pcv[N + n] = prnd;
                    pcv[2 * N + n] = psh;
                }
#pragma unroll
                for (int i = 0; i < S::SPARE; ++i) {
                    const int kbyte = 8 * (S::NW + i);
                    uint8_t* dst = smem + L::OFF_B + (kbyte >> 7) * (N * 128) + n * 128 +
                                   ((((kbyte & 127) >> 4) ^ (n & 7)) << 4) + (kbyte & 15);
                    *reinterpret_cast<uint2*>(dst) = make_uint2(dw[2 * i], dw[2 * i + 1]);
                }
            }
        }
        fence_async_smem();                // B, before the async proxy (the MMA) reads it
        tc_fence_before();
        sync_workers();
        tc_fence_after();
        tmem_base = (uint32_t)lds32(tmem_slot);
        if (p.prep_out != nullptr) {
            // preparation only: the image goes to memory (this launch has no tiles)
            const uint4* src = reinterpret_cast<const uint4*>(smem + L::OFF_B);
            uint4* dst = reinterpret_cast<uint4*>(p.prep_out);
            for (int i = wt; i < (int)(IMAGE / 16); i += NT) dst[i] = src[i];
            if (wt == 0) dst[IMAGE / 16] = make_uint4(use_preload ? 1u : 0u, p.prep_tag, 0u, 0u);
        }
    }

    if (warp < PWN) {
        // ---------------------------------------------------------------- producers
        producer(p, mytiles, NB, warp, buf0, geo_s, full0, empty0, abort_flag, lane, blockIdx.x, gridDim.x);
    } else if (warp == PWN) {
        // ---------------------------------------------------------------- MMA issuer
        // D = s32, A = unsigned bytes (tensor memory), B = signed bytes, K-major, M = 128
        constexpr uint32_t idesc = (2u << 4) | (1u << 10) | ((uint32_t)(N >> 3) << 17) |
                                   ((uint32_t)(ROWS >> 4) << 24);
        const uint64_t bdesc0 = make_kmajor_sw128_desc(sbase + L::OFF_B);
        int g = 0;
        uint32_t t = 0;                                // tile k is group g's t-th tile
        if (p.prep_in != nullptr && mytiles > 0) mbar_wait(bar_prep, 0, abort_flag, p.status);
        for (int k = 0; k < mytiles; ++k) {
            TR(1, k, 0);
            if (!wait_idle(bar_a_ready(g), t & 1u, abort_flag, p.status)) break;
            TR(1, k, 1);
            tc_fence_after();
            if (elect_one()) {
                const uint32_t d_tmem = tmem_base + (uint32_t)(g * S::ACCW);
                const uint32_t a_tmem = tmem_base + (uint32_t)(G * S::ACCW + g * S::ACOLS);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks)
                    tc_mma_i8_ts(d_tmem, a_tmem + (uint32_t)(8 * ks),
                                 bdesc0 + (uint64_t)((ks >> 2) * ((N * 128) >> 4) + 2 * (ks & 3)), idesc,
                                 (ks > 0 || use_preload) ? 1u : 0u);
                tc_commit(bar_mma_done(g));
            }
            __syncwarp();
            TR(1, k, 2);
            if (++g == G) { g = 0; ++t; }
        }
    } else {
        // ---------------------------------------------------------------- workers
        const int g = (warp - (PWN + 1)) >> 2;         // my group: tiles g, g + G, ...
        const int q = warp & 3;                        // my tensor-memory lane quarter
        const int row = q * 32 + lane;                 // my GEMM row
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t acc_taddr = lane_taddr + (uint32_t)(g * S::ACCW);
        const uint32_t a_taddr = lane_taddr + (uint32_t)(G * S::ACCW + g * S::ACOLS);
        const uint32_t zfill = (uint32_t)p.za * 0x11111111u;
        // the 32-bit form of the rounding shift with the output zero point folded into the
        // rounding constant (see requant8())
        const bool fast = p.rq.shift >= 2 && p.rq.shift <= 27;
        const int sh1 = p.rq.shift - 1;
        const int rnd = fast ? (1 << (sh1 - 1)) + (p.rq.zo - p.rq.lo) * (1 << sh1) : 0;
        const uint32_t hml2 = (uint32_t)(p.rq.hi - p.rq.lo) * 0x00010001u;
        const uint32_t lofill = (uint32_t)p.rq.lo * 0x11111111u;
        const bool pc_fast = pc && lds32(pcslow_flag) == 0;
        const uint32_t mstep = gridDim.x * (uint32_t)(S::TILE * G);
        uint32_t mbase = (blockIdx.x + (uint32_t)g * gridDim.x) * (uint32_t)S::TILE;
        int kb = g;                                    // k % NB (G <= NB)
        uint32_t phase = 0, t = 0;                     // (k / NB) % 2; k is my group's t-th tile
        for (int k = g; k < mytiles; k += G, mbase += mstep, ++t) {
            const bool tr = (warp & 3) == ((PWN + 1) & 3);
            if (tr) TR(2, k, 0);
            if (!wait_idle(full0 + 8 * kb, phase, abort_flag, p.status)) break;
            if (tr) TR(2, k, 1);
            const int4 gv = geo_s[kb];                 // n_first, oh_first, s0 (published with the tile)
            const uint32_t bufaddr = smem_u32(buf0 + kb * p.bufbytes);     // 16 bytes of slack, then the rows
            const uint32_t done_bar = empty0 + 8 * kb;
            kb += G;
            if (kb >= NB) { kb -= NB; phase ^= 1; }
            // my row's first pixel (rows past the end read the tile's first pixel: a valid place)
            const uint32_t mrow = mbase + (uint32_t)(row * P);
            const uint32_t mm = mrow < M32 ? mrow : mbase;
            const uint32_t qq = fdiv(mm, p.div_ow);
            const int ow = (int)(mm - qq * (uint32_t)p.OW);
            const uint32_t n0 = fdiv(qq, p.div_oh);
            const int oh = (int)(qq - n0 * (uint32_t)p.OH);
            const int seg = (int)n0 - gv.x;
            const int slot0 = seg == 0 ? (oh - gv.y) * p.sh : gv.z + (seg - 1) * p.sfull + oh * p.sh;
            // Window words that fall left or right of the image (horizontal padding 1: at most
            // one input column on either side, in the first and the last group of an output
            // row) are replaced by the zero point; rows above or below it were staged as such.
            uint32_t w[KS * 4];
            if constexpr (S::NIB) {
                // nibble offset of my window in the dense copy; its words are unaligned bit fields
                const int b = (16 + slot0 * p.rowbytes) * 2 + ow * S::SW - 1;
                const int shf = (b & 7) * 4;
                const uint32_t src = bufaddr + (uint32_t)((b >> 3) << 2);
                // window nibbles [nl, r0) lie inside the image (input columns 0 .. W-1)
                const int nl = ow == 0 ? 1 : 0;
                const int r0 = p.W - (ow * S::SW - 1);         // window nibble index of input column W
#pragma unroll
                for (int kh = 0; kh < S::KH; ++kh) {
                    uint32_t a[WW + 1];
                    load_row<0, WW + 1, -1>(src + (uint32_t)(kh * p.rowbytes), a);
#pragma unroll
                    for (int i = 0; i < WW; ++i) w[kh * WW + i] = __funnelshift_r(a[i], a[i + 1], shf);
                }
#pragma unroll
                for (int i = 0; i < WW; ++i) {
                    // word i holds window nibbles 8i .. 8i+7
                    uint32_t keep = 0xFFFFFFFFu;
                    if (i == 0 && nl) keep = 0xFFFFFFF0u;
                    const int re = r0 - 8 * i;                 // first nibble of this word past the image
                    if (re < 8) keep &= re <= 0 ? 0u : (1u << (4 * re)) - 1u;
                    const uint32_t fill = zfill & ~keep;
#pragma unroll
                    for (int kh = 0; kh < S::KH; ++kh) w[kh * WW + i] = (w[kh * WW + i] & keep) | fill;
                }
            } else {
                const uint32_t src = bufaddr + (uint32_t)(16 + slot0 * p.rowbytes + (ow * S::SW - 1) * (4 * S::CW));
                const bool left = ow == 0, right = ow * S::SW - 1 + S::COLS > p.W;
#pragma unroll
                for (int kh = 0; kh < S::KH; ++kh) {
                    load_row<0, WW, S::PH>(src + (uint32_t)(kh * p.rowbytes), w + kh * WW);
#pragma unroll
                    for (int i = 0; i < S::CW; ++i) {
                        if (left) w[kh * WW + i] = zfill;
                        if (right) w[kh * WW + WW - S::CW + i] = zfill;
                    }
                }
            }
            // (the words past the depth are the constants' step: see below)
            // Everyone in my group finished the previous tile's epilogue before arriving
            // below, so the A slot and the accumulator are free: A, then the constants the
            // accumulator columns start from.
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t r8[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int wd = 4 * ks + j;
                    if (wd < S::NW) {
                        r8[2 * j] = w[wd] & 0x0F0F0F0Fu;
                        r8[2 * j + 1] = (w[wd] >> 4) & 0x0F0F0F0Fu;
                    } else {
                        // the constants' bytes: 1, then 255s
                        r8[2 * j] = wd == S::NW ? 0xFFFFFF01u : 0xFFFFFFFFu;
                        r8[2 * j + 1] = 0xFFFFFFFFu;
                    }
                }
                tc_st8(a_taddr + (uint32_t)(8 * ks), r8);
            }
            if (use_preload) {
                if (p.prep_in != nullptr) mbar_wait(bar_prep, 0, abort_flag, p.status);     // the constants are in the image
#pragma unroll
                for (int j = 0; j < N / 8; ++j) {
                    const uint4 x = lds128(colterm_s + 4 * (8 * j)), y = lds128(colterm_s + 4 * (8 * j + 4));
                    const uint32_t r8[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
                    tc_st8(acc_taddr + (uint32_t)(8 * j), r8);
                }
            }
            if (tr) TR(2, k, 2);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_a_ready(g));
                mbar_arrive(done_bar);                 // the staged copy has been read
            }
            if (tr) TR(2, k, 3);
            if (!wait_idle(bar_mma_done(g), t & 1u, abort_flag, p.status)) break;
            if (tr) TR(2, k, 4);
            tc_fence_after();
            uint8_t* dst = p.Y + (uint64_t)mrow * (OC / 2);
            // 64 columns at a time where the register budget allows: both loads in flight
            // before the one wait
            constexpr int CB = (N >= 64 && G <= 4) ? 2 : 1;
#pragma unroll
            for (int cb = 0; cb < N / 32; cb += CB) {
                uint32_t r[CB][32];
#pragma unroll
                for (int c = 0; c < CB; ++c) tc_ld32(acc_taddr + (uint32_t)((cb + c) * 32), r[c]);
                tc_wait_ld();
#pragma unroll
                for (int c = 0; c < CB; ++c) {
                    uint32_t o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        o[j] = (pc ? requant8_channels(r[c] + 8 * j, p.rq, pc_s, N, (cb + c) * 32 + 8 * j, pc_fast, hml2)
                                : fast ? requant8<true>(r[c] + 8 * j, p.rq, sh1, rnd, hml2)
                                       : requant8<false>(r[c] + 8 * j, p.rq, sh1, rnd, hml2)) + lofill;
                    if (mrow < M32)
                        *reinterpret_cast<uint4*>(dst + (cb + c) * 16) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            tc_fence_before();                         // my tcgen05.ld are done before the next tile's MMA may write
            if (tr) TR(2, k, 5);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == PWN) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}


// ---------------------------------------------------------------------------------------
// Layers whose input pixels are whole 16-byte pieces (C a multiple of 32): any filter size,
// strides and paddings, 32 .. 128 output channels per CTA (more are split over CTAs, each
// with its own share of the weights), geometry taken at run time.  These are the layers with
// enough depth to keep the tensor pipe busy, so the tile is pipelined in depth as a GEMM is:
//   warps 0..1      producers, as above (a tile is one bulk copy per image: two keep up)
//   warp 2          MMA issuer
//   8 build warps   two sets of four (one warp per lane quarter) that take the depth
//                   chunks of a tile in turn: a GEMM row is one pixel, a 32-byte depth step is
//                   32 channels of one tap -- one 16-byte load from the staged copy, one
//                   tcgen05.st --, so the depth needs no padding and the steps are
//                   consecutive 16-byte pieces of a weight row; a chunk of CK steps goes
//                   into one slot of a ring in tensor memory
//   8 epilogue warps  two per lane quarter, sharing the 32-column chunks of the accumulator
// with two accumulators, so that the MMAs of a tile overlap the epilogue of the tile before
// and the build of the chunks after.
// ---------------------------------------------------------------------------------------
constexpr int WCK = 8;              // depth steps per chunk (64 columns of tensor memory)
constexpr int WNCH = 4;             // chunks in the ring
#ifndef Q4_CTC_WSB
#define Q4_CTC_WSB 2
#endif
#ifndef Q4_CTC_WSE
#define Q4_CTC_WSE 2
#endif
constexpr int WSB = Q4_CTC_WSB, WSE = Q4_CTC_WSE;     // build / epilogue warps per lane quarter
constexpr int WPW = 2;              // producer warps (a tile is one bulk copy per image; two keep up)
constexpr int WNBAR = 2 * NBMAX + 2 * WNCH + 6;     // (even: what follows stays 16-byte aligned)
// A build set's consecutive chunks are WSB chunks apart.  A set that waits for a ring slot must
// not be more than one use of that slot ahead of the MMA warp (mbarrier phases are told apart
// by one parity bit), so the distance has to stay within the ring.
static_assert(WSB <= WNCH, "build sets may run at most one ring round ahead");

struct WideLayout {
    int off_tab, off_ct, off_pc, off_geo, off_bar, off_misc, off_buf;     // after B (at 0)
};
__host__ __device__ inline WideLayout wide_layout(int N, int KS)
{
    WideLayout l;
    l.off_tab = ((KS + 1 + 3) / 4) * N * 128;          // B holds KS + 1 steps; then int2 [KS]: offset of the
                                                       // step's 16 bytes, its window column
    l.off_ct = l.off_tab + (KS * 8 + 15) / 16 * 16;
    l.off_pc = l.off_ct + N * 4;                      // int32 [3][N]: per-column multiplier, rounding, shift
    l.off_geo = l.off_pc + 3 * N * 4;
    l.off_bar = l.off_geo + NBMAX * 16;
    l.off_misc = l.off_bar + WNBAR * 8;
    l.off_buf = l.off_misc + 16;
    return l;
}

constexpr int WIDE_THREADS = (WPW + 1 + 4 * WSB + 4 * WSE) * 32;

// PC: per-channel weight zero points, multipliers and shifts (see conv_tc_kernel).
template <bool PC>
__global__ void __launch_bounds__(WIDE_THREADS, 1)
conv_tc_wide_kernel(const Params p)
{
    constexpr bool pc = PC;
    const int N = p.tcN, KS = p.KS, CW4 = p.C / 32;   // columns of my tile, depth steps, steps per tap
    // One more depth step carries the per-channel constants of Eq. 3 into the product: its A
    // bytes are the same for every row, 1 then thirty-one times 255, and its B bytes are the
    // constant's digits d0 + 255 * (d1 + ... + d31), each a signed byte.  The accumulators
    // then need no preloading and can be handed back as soon as they have been read.  A
    // constant beyond the digits' range (about a million) switches the whole CTA to
    // preloaded accumulators, the step's B bytes being zero then.
    const int KSX = KS + 1;
    const int nchunks = (KSX + WCK - 1) / WCK;
    const WideLayout L = wide_layout(N, KS);
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    int2* tab = reinterpret_cast<int2*>(smem + L.off_tab);
    int32_t* colterm = reinterpret_cast<int32_t*>(smem + L.off_ct);
    const uint32_t colterm_s = sbase + L.off_ct, tab_s = sbase + L.off_tab;
    int4* geo_s = reinterpret_cast<int4*>(smem + L.off_geo);
    const uint32_t bar0 = sbase + L.off_bar;
    const uint32_t full0 = bar0, empty0 = bar0 + 8 * NBMAX;
    auto bar_a_ready   = [&](int c) { return bar0 + 8u * (uint32_t)(2 * NBMAX + c); };
    auto bar_a_free    = [&](int c) { return bar0 + 8u * (uint32_t)(2 * NBMAX + WNCH + c); };
    auto bar_acc_full  = [&](int a) { return bar0 + 8u * (uint32_t)(2 * NBMAX + 2 * WNCH + a); };
    auto bar_acc_empty = [&](int a) { return bar0 + 8u * (uint32_t)(2 * NBMAX + 2 * WNCH + 2 + a); };
    const uint32_t bar_prep = bar0 + 8u * (uint32_t)(2 * NBMAX + 2 * WNCH + 4);      // a prepared weight image has landed
    const int NB = p.nbuf;
    const uint32_t tmem_slot = sbase + L.off_misc, abort_flag = sbase + L.off_misc + 4;
    const uint32_t preload_flag = sbase + L.off_misc + 8;
    const uint32_t pcslow_flag = sbase + L.off_misc + 12;         // per-channel: some shift needs the 64-bit form
    const uint32_t pc_s = sbase + L.off_pc;
    int32_t* pcv = reinterpret_cast<int32_t*>(smem + L.off_pc);
    uint8_t* buf0 = smem + L.off_buf;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // my share of the output channels, and my pixel tiles
    const int nsplit = p.tcSplit;
    const int oc0 = (int)(blockIdx.x % nsplit) * N;
    const int64_t tile0 = blockIdx.x / nsplit, tstride = gridDim.x / nsplit;
    constexpr int ACC0 = 0, ARING0 = 256;              // tensor-memory columns: two accumulators, then the ring

    if (tid == 0) {
        for (int i = 0; i < NB; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, 4 * WSB);
        }
        for (int c = 0; c < WNCH; ++c) {
            mbar_init(bar_a_ready(c), 4);
            mbar_init(bar_a_free(c), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_acc_full(a), 1);
            mbar_init(bar_acc_empty(a), 4 * WSE);
        }
        mbar_init(bar_prep, 1);
        sts32(abort_flag, 0);
        sts32(preload_flag, 0);
        sts32(pcslow_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == WPW) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(tmem_slot), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.wait;" ::: "memory");             // see conv_tc_kernel
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t ntiles = (p.M + ROWS - 1) / ROWS;
    int mytiles = (int)((ntiles - tile0 + tstride - 1) / tstride);
    const uint32_t M32 = (uint32_t)p.M;
    // a CTA's share of a prepared image: B, the per-column constants, {fallback flag, tag} (see conv_tc_kernel)
    const uint32_t b_bytes = (uint32_t)L.off_tab, share_bytes = b_bytes + (uint32_t)N * 4u + 16u;
    uint2 trailer = make_uint2(0u, p.prep_tag);
    if (p.prep_in != nullptr)
        trailer = __ldg(reinterpret_cast<const uint2*>(p.prep_in + (size_t)(blockIdx.x % nsplit) * share_bytes + b_bytes +
                                                       (uint32_t)N * 4u));
    if (trailer.y != p.prep_tag) {
        mytiles = 0;
        if (tid == 0) atomicOr(p.status, kStatusWeightImage);
    }

    uint32_t tmem_base = 0;
    bool use_preload = false;
    if (warp >= WPW) {
        constexpr int NT = WIDE_THREADS - WPW * 32;
        const int wt = tid - WPW * 32;
        auto sync_workers = [] { asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory"); };
        const bool prepared = p.prep_in != nullptr;
        if (!prepared)
            for (int i = wt; i < N; i += NT) colterm[i] = 0;
        // depth step ks = (kh, kw, c4): where its 16 bytes sit relative to a pixel's window
        // start, and which window column it belongs to
        for (int ks = wt; ks < KS; ks += NT) {
            const int tap = ks / CW4, c4 = ks - tap * CW4;
            const int kh = tap / p.KW, kw = tap - kh * p.KW;
            tab[ks] = make_int2(kh * p.rowbytes + kw * p.unit + 16 * c4, kw);
        }
        sync_workers();
        if (prepared) {
            const uint8_t* img = p.prep_in + (size_t)(blockIdx.x % nsplit) * share_bytes;
            if (wt == 0 && mytiles > 0) {
                mbar_expect_tx(bar_prep, b_bytes + (uint32_t)N * 4u);
                fused::bulk_load_row(sbase, img, b_bytes, bar_prep);
                fused::bulk_load_row(colterm_s, img + b_bytes, (uint32_t)N * 4u, bar_prep);
            }
            use_preload = trailer.x != 0;
            tmem_base = (uint32_t)lds32(tmem_slot);
        } else {
        // B: row n is output channel oc0 + (n with the ch8 order inside each group of eight);
        // depth step ks is bytes 16 ks .. 16 ks + 15 of the weight row
        const int tasks = N * KS;
        const bool wt_vec = (((uintptr_t)p.Wt | (uintptr_t)p.ldw) & 15) == 0;
        // four tasks at a time: all their loads are requested before any is expanded
        for (int base = wt; base < tasks; base += 4 * NT) {
            uint4 wq[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base + u * NT;
                wq[u] = make_uint4(0, 0, 0, 0);
                if (idx < tasks) {
                    const int n = idx / KS, ks = idx - n * KS;
                    const int oc = oc0 + (n & ~7) + ch8(n & 7);
                    const uint8_t* src = p.Wt + (int64_t)oc * p.ldw + 16 * ks;
                    if (wt_vec) {
                        wq[u] = __ldg(reinterpret_cast<const uint4*>(src));
                    } else if (p.wt_words) {
                        const uint32_t* s4 = reinterpret_cast<const uint32_t*>(src);
                        wq[u] = make_uint4(__ldg(s4), __ldg(s4 + 1), __ldg(s4 + 2), __ldg(s4 + 3));
                    } else {
                        uint32_t t[4] = {0, 0, 0, 0};
                        for (int b = 0; b < 16; ++b) t[b >> 2] |= (uint32_t)__ldg(src + b) << (8 * (b & 3));
                        wq[u] = make_uint4(t[0], t[1], t[2], t[3]);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base + u * NT;
                if (idx >= tasks) break;
                const int n = idx / KS, ks = idx - n * KS;
                const int zbo = pc ? (p.zb_ch ? __ldg(p.zb_ch + oc0 + (n & ~7) + ch8(n & 7)) : 0) : p.zb;
                const uint32_t wv[4] = {wq[u].x, wq[u].y, wq[u].z, wq[u].w};
                uint32_t o[8];
                int raw = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    raw += nibble_sum(wv[j]);
                    o[2 * j] = fused::sub_zb(wv[j] & 0x0F0F0F0Fu, (uint32_t)zbo);
                    o[2 * j + 1] = fused::sub_zb((wv[j] >> 4) & 0x0F0F0F0Fu, (uint32_t)zbo);
                }
                uint8_t* row = smem + (ks >> 2) * (N * 128) + n * 128;
                const int c = 2 * (ks & 3);
                *reinterpret_cast<uint4*>(row + ((c ^ (n & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4*>(row + (((c + 1) ^ (n & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
                if (!p.colsum_w && raw) atomicAdd(&colterm[n], raw);          // by column position
            }
        }
        sync_workers();
        int cterm = 0;
        if (wt < N) {
            const int oc = oc0 + (wt & ~7) + ch8(wt & 7);
            const int cs = p.colsum_w ? p.colsum_w[oc] : colterm[wt];
            const int zbo = pc ? (p.zb_ch ? p.zb_ch[oc] : 0) : p.zb;
            cterm = (int)((uint32_t)(p.K * p.za * zbo) - (uint32_t)(p.za * cs) +
                          (uint32_t)(p.bias ? p.bias[oc] : 0));
            if (pc) {
                const int sh = p.shift_ch[oc];
                if (sh < 2 || sh > 27) sts32(pcslow_flag, 1);
            }
            // digits: cterm = d0 + 255 * q, d0 in -127..127, q spread over thirty-one bytes
            int d0 = cterm % 255;
            if (d0 > 127) d0 -= 255;
            if (d0 < -127) d0 += 255;
            const int qd = (cterm - d0) / 255;
            if (qd > 31 * 127 || qd < -31 * 127) sts32(preload_flag, 1);
        }
        sync_workers();
        use_preload = lds32(preload_flag) != 0;
        if (wt < N) {
            colterm[wt] = cterm;
            if (pc) {
                // this column's multiplier, rounding constant and shift
                const int oc = oc0 + (wt & ~7) + ch8(wt & 7);
                const bool pfast = lds32(pcslow_flag) == 0;
                const int sh = p.shift_ch[oc];
                const int psh = pfast ? sh - 1 : sh;
                pcv[wt] = p.mult_ch[oc];
                pcv[N + wt] = pfast ? (1 << (psh - 1)) + (p.rq.zo - p.rq.lo) * (1 << psh) : 0;
                pcv[2 * N + wt] = psh;
            }
            int d0 = cterm % 255;
            if (d0 > 127) d0 -= 255;
            if (d0 < -127) d0 += 255;
            int qd = use_preload ? 0 : (cterm - d0) / 255;
            if (use_preload) d0 = 0;
            uint32_t o[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint32_t word = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    int dgt;
                    if (i == 0 && b == 0) {
                        dgt = d0;
                    } else {
                        dgt = qd > 127 ? 127 : qd < -127 ? -127 : qd;
                        qd -= dgt;
                    }
                    word |= ((uint32_t)dgt & 0xFFu) << (8 * b);
                }
                o[i] = word;
            }
            uint8_t* row = smem + (KS >> 2) * (N * 128) + wt * 128;
            const int c = 2 * (KS & 3);
            *reinterpret_cast<uint4*>(row + ((c ^ (wt & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<uint4*>(row + (((c + 1) ^ (wt & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
        }
        fence_async_smem();                // B, before the async proxy (the MMA) reads it
        tc_fence_before();
        sync_workers();
        tc_fence_after();
        tmem_base = (uint32_t)lds32(tmem_slot);
        if (p.prep_out != nullptr) {
            // preparation only: my share of the image goes to memory (this launch has no tiles)
            uint8_t* img = p.prep_out + (size_t)(blockIdx.x % nsplit) * share_bytes;
            const uint4* src = reinterpret_cast<const uint4*>(smem);
            uint4* dst = reinterpret_cast<uint4*>(img);
            for (int i = wt; i < (int)(b_bytes / 16); i += NT) dst[i] = src[i];
            const uint4* cs = reinterpret_cast<const uint4*>(smem + L.off_ct);
            for (int i = wt; i < N / 4; i += NT) dst[b_bytes / 16 + i] = cs[i];
            if (wt == 0) dst[b_bytes / 16 + N / 4] = make_uint4(use_preload ? 1u : 0u, p.prep_tag, 0u, 0u);
        }
        }
    }

    if (warp < WPW) {
        // ---------------------------------------------------------------- producers
        producer(p, mytiles, NB, warp, buf0, geo_s, full0, empty0, abort_flag, lane, tile0, tstride, WPW);
    } else if (warp == WPW) {
        // ---------------------------------------------------------------- MMA issuer
        const uint32_t idesc = (2u << 4) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(ROWS >> 4) << 24);
        const uint64_t bdesc0 = make_kmajor_sw128_desc(sbase);
        const uint32_t blk = (uint32_t)(N * 128) >> 4;          // descriptor units per 128-byte depth block of B
        uint32_t cg = 0;                               // chunks issued so far
        bool ok = true;
        if (p.prep_in != nullptr && mytiles > 0) mbar_wait(bar_prep, 0, abort_flag, p.status);
        for (int k = 0; k < mytiles && ok; ++k) {
            const int acc = k & 1;
            TR(1, k, 0);
            // the accumulator has been read back (and, where the constants do not ride in
            // the product, preloaded with them)
            if (!wait_idle(bar_acc_empty(acc), ((uint32_t)k >> 1) & 1u, abort_flag, p.status)) break;
            TR(1, k, 1);
            const uint32_t d_tmem = tmem_base + (uint32_t)(ACC0 + acc * 128);
            for (int c = 0; c < nchunks; ++c, ++cg) {
                const int slot = (int)(cg % WNCH);
                if (!wait_idle(bar_a_ready(slot), (cg / WNCH) & 1u, abort_flag, p.status)) { ok = false; break; }
                TR(1, k, 2 + c);
                tc_fence_after();
                if (elect_one()) {
                    // the chunk's steps with compile-time offsets: issuing must not cost more
                    // than the 64 clocks an MMA takes
                    const uint32_t a_tmem = tmem_base + (uint32_t)(ARING0 + slot * (8 * WCK));
                    const uint64_t bd = bdesc0 + (uint64_t)((uint32_t)(c * (WCK / 4)) * blk);
                    const int nst = KSX - c * WCK;     // steps of this chunk (WCK unless it is the last)
#pragma unroll
                    for (int j = 0; j < WCK; ++j)
                        if (j < nst)
                            tc_mma_i8_ts(d_tmem, a_tmem + (uint32_t)(8 * j),
                                         bd + (uint64_t)((uint32_t)(j >> 2) * blk + 2u * (uint32_t)(j & 3)), idesc,
                                         (c > 0 || j > 0 || use_preload) ? 1u : 0u);
                    tc_commit(bar_a_free(slot));
                    if (c == nchunks - 1) tc_commit(bar_acc_full(acc));
                }
                __syncwarp();
            }
        }
    } else if (warp < WPW + 1 + 4 * WSB) {
        // ---------------------------------------------------------------- build warps
        const int sb = (warp - (WPW + 1)) >> 2;        // my set: every WSB-th chunk, counted across tiles
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t a_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)ARING0;
        const uint32_t zfill = (uint32_t)p.za * 0x11111111u;
        const uint32_t mstep = (uint32_t)tstride * (uint32_t)ROWS;
        uint32_t mbase = (uint32_t)tile0 * (uint32_t)ROWS;
        int kb = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int k = 0; k < mytiles && ok; ++k, mbase += mstep) {
            if (warp == WPW + 1) TR(2, k, 0);
            if (!wait_idle(full0 + 8 * kb, phase, abort_flag, p.status)) break;
            if (warp == WPW + 1) TR(2, k, 1);
            const int4 gv = geo_s[kb];
            const uint32_t bufaddr = smem_u32(buf0 + kb * p.bufbytes);
            const uint32_t done_bar = empty0 + 8 * kb;
            if (++kb == NB) { kb = 0; phase ^= 1; }
            const uint32_t mrow = mbase + (uint32_t)row;
            const uint32_t mm = mrow < M32 ? mrow : mbase;
            const uint32_t qq = fdiv(mm, p.div_ow);
            const int ow = (int)(mm - qq * (uint32_t)p.OW);
            const uint32_t n0 = fdiv(qq, p.div_oh);
            const int oh = (int)(qq - n0 * (uint32_t)p.OH);
            const int seg = (int)n0 - gv.x;
            const int slot0 = seg == 0 ? (oh - gv.y) * p.sh : gv.z + (seg - 1) * p.sfull + oh * p.sh;
            const int col0 = ow * p.sw - p.pw;         // input column of my window's first column
            const uint32_t src = bufaddr + (uint32_t)(16 + slot0 * p.rowbytes + col0 * p.unit);
            const uint32_t cg0 = (uint32_t)k * (uint32_t)nchunks;
            // chunks are dealt to the sets round-robin over the whole run of tiles, so that a tile of
            // three chunks does not leave one set with two of them every time
            for (int c = (int)(((uint32_t)sb + (uint32_t)WSB - cg0 % (uint32_t)WSB) % (uint32_t)WSB); c < nchunks; c += WSB) {
                const uint32_t cg = cg0 + (uint32_t)c;
                const int slot = (int)(cg % WNCH);
                // the MMAs that read this slot WNCH chunks ago are complete
                if (warp == WPW + 1 && c == 0) TR(2, k, 2);
                if (!wait_idle(bar_a_free(slot), ((cg / WNCH) & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                if (warp == WPW + 1 && c == 0) TR(2, k, 3);
                const int ks0 = c * WCK;
                // a depth step is 16 bytes of one tap; taps left or right of the image read as
                // the zero point.  All table entries, then all loads, then the unpacking: the
                // loads' latencies overlap.
                uint2 te[WCK];
                uint4 v[WCK];
#pragma unroll
                for (int j = 0; j < WCK; ++j)
                    if (ks0 + j < KS) te[j] = lds64(tab_s + 8 * (ks0 + j));
                if (warp == WPW + 1 && c == 0) TR(2, k, 4);
#pragma unroll
                for (int j = 0; j < WCK; ++j) {
                    v[j] = make_uint4(zfill, zfill, zfill, zfill);
                    if (ks0 + j < KS && (unsigned)(col0 + (int)te[j].y) < (unsigned)p.W) v[j] = lds128(src + te[j].x);
                }
#pragma unroll
                for (int j = 0; j < WCK; ++j) {
                    const int ks = ks0 + j;
                    if (ks < KS) {
                        const uint32_t r8[8] = {v[j].x & 0x0F0F0F0Fu, (v[j].x >> 4) & 0x0F0F0F0Fu,
                                                v[j].y & 0x0F0F0F0Fu, (v[j].y >> 4) & 0x0F0F0F0Fu,
                                                v[j].z & 0x0F0F0F0Fu, (v[j].z >> 4) & 0x0F0F0F0Fu,
                                                v[j].w & 0x0F0F0F0Fu, (v[j].w >> 4) & 0x0F0F0F0Fu};
                        tc_st8(a_taddr + (uint32_t)(slot * (8 * WCK) + 8 * j), r8);
                    } else if (ks == KS) {
                        // the step of the constants: 1, then thirty-one times 255
                        const uint32_t r8[8] = {0xFFFFFF01u, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu,
                                                0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
                        tc_st8(a_taddr + (uint32_t)(slot * (8 * WCK) + 8 * j), r8);
                    }
                }
                if (warp == WPW + 1 && c == 0) TR(2, k, 5);
                tc_wait_st();
                if (warp == WPW + 1 && c == 0) TR(2, k, 6);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_a_ready(slot));
            }
            __syncwarp();
            if (warp == WPW + 1) TR(2, k, 7);
            if (lane == 0) mbar_arrive(done_bar);      // the staged copy has been read
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps
        const int se = (warp - (WPW + 1 + 4 * WSB)) >> 2;      // my share of the 32-column chunks
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t acc_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)ACC0;
        const bool fast = p.rq.shift >= 2 && p.rq.shift <= 27;
        const int sh1 = p.rq.shift - 1;
        const int rnd = fast ? (1 << (sh1 - 1)) + (p.rq.zo - p.rq.lo) * (1 << sh1) : 0;
        const uint32_t hml2 = (uint32_t)(p.rq.hi - p.rq.lo) * 0x00010001u;
        const uint32_t lofill = (uint32_t)p.rq.lo * 0x11111111u;
        const bool pc_fast = pc && lds32(pcslow_flag) == 0;
        auto preload = [&](int acc) {                  // my chunks start from the channels' constants
            for (int ch = se; ch < N / 32; ch += WSE) {
#pragma unroll
                for (int j = 4 * ch; j < 4 * ch + 4; ++j) {
                    const uint4 x = lds128(colterm_s + 4 * (8 * j)), y = lds128(colterm_s + 4 * (8 * j + 4));
                    const uint32_t r8[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
                    tc_st8(acc_taddr + (uint32_t)(acc * 128 + 8 * j), r8);
                }
            }
        };
        if (use_preload) {
            if (p.prep_in != nullptr) mbar_wait(bar_prep, 0, abort_flag, p.status);     // the constants are in the image
            preload(0);
            preload(1);
            tc_wait_st();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(bar_acc_empty(0));
            mbar_arrive(bar_acc_empty(1));
        }
        const uint32_t mstep = (uint32_t)tstride * (uint32_t)ROWS;
        uint32_t mbase = (uint32_t)tile0 * (uint32_t)ROWS;
        const int nch = N / 32;
        for (int k = 0; k < mytiles; ++k, mbase += mstep) {
            const int acc = k & 1;
            if (warp == WPW + 1 + 4 * WSB) TR(3, k, 0);
            if (!wait_idle(bar_acc_full(acc), ((uint32_t)k >> 1) & 1u, abort_flag, p.status)) break;
            if (warp == WPW + 1 + 4 * WSB) TR(3, k, 1);
            tc_fence_after();
            const uint32_t mrow = mbase + (uint32_t)row;
            uint8_t* dst = p.Y + (uint64_t)mrow * (p.OCtot / 2) + (oc0 >> 1);
            for (int ch = se; ch < nch; ch += WSE) {
                uint32_t r[32];
                tc_ld32(acc_taddr + (uint32_t)(acc * 128 + ch * 32), r);
                tc_wait_ld();
                if (!use_preload && ch + WSE >= nch) {
                    // my last chunk is in registers: the accumulator can take the next tile
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_acc_empty(acc));
                }
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    o[j] = (pc ? requant8_channels(r + 8 * j, p.rq, pc_s, N, ch * 32 + 8 * j, pc_fast, hml2)
                            : fast ? requant8<true>(r + 8 * j, p.rq, sh1, rnd, hml2)
                                   : requant8<false>(r + 8 * j, p.rq, sh1, rnd, hml2)) + lofill;
                if (mrow < M32) *reinterpret_cast<uint4*>(dst + ch * 16) = make_uint4(o[0], o[1], o[2], o[3]);
            }
            if (warp == WPW + 1 + 4 * WSB) TR(3, k, 2);
            if (use_preload || se >= nch) {
                // (a warp without a chunk of its own still reports)
                if (use_preload) {
                    preload(acc);
                    tc_wait_st();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty(acc));
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == WPW) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace convtc

// ---- host side ------------------------------------------------------------------------
namespace {

// Pixels per GEMM row (P) and worker groups (G) of each instance.
#ifndef Q4_CTC_P0
#define Q4_CTC_P0 8
#endif
#ifndef Q4_CTC_G0
#define Q4_CTC_G0 4
#endif
#ifndef Q4_CTC_P1
#define Q4_CTC_P1 4
#endif
#ifndef Q4_CTC_G1
#define Q4_CTC_G1 4
#endif
#ifndef Q4_CTC_P2
#define Q4_CTC_P2 2
#endif
#ifndef Q4_CTC_G2
#define Q4_CTC_G2 4
#endif
#ifndef Q4_CTC_P3
#define Q4_CTC_P3 1
#endif
#ifndef Q4_CTC_G3
#define Q4_CTC_G3 3
#endif
#ifndef Q4_CTC_P4
#define Q4_CTC_P4 2
#endif
#ifndef Q4_CTC_G4
#define Q4_CTC_G4 4
#endif

struct TcChoice {
    int id;          // which instance, -1 = none
    int P;
    bool nib;
};

// The layer classes the kernel has instances for: 3x3 filters, horizontal padding 1, the
// channel counts and strides of the workloads' layers.
TcChoice choose_instance(const q4_conv_desc& d)
{
    TcChoice c{-1, 1, false};
    if (d.KH != 3 || d.KW != 3 || d.pad_w != 1 || d.stride_w != d.stride_h) return c;
    const int s = d.stride_w;
    if (d.C == 1 && d.OC == 8 && s == 1) c = {0, Q4_CTC_P0, true};
    else if (d.C == 8 && d.OC == 16 && s == 2) c = {1, Q4_CTC_P1, false};
    else if (d.C == 16 && d.OC == 32 && s == 2) c = {2, Q4_CTC_P2, false};
    else if (d.C == 32 && d.OC == 64 && s == 2) c = {3, Q4_CTC_P3, false};
    else if (d.C == 16 && d.OC == 32 && s == 1) c = {4, Q4_CTC_P4, false};
    return c;
}

// Staging geometry of a tile of `tile` consecutive output pixels (the fields the shared
// producer warp reads); returns the bytes of one input buffer, 0 if the layer does not fit.
int64_t plan_staging(fused::Params& p, const q4_conv_desc& d, const uint8_t* X, int tile, bool nib)
{
    p.H = d.H; p.W = d.W; p.C = d.C; p.KH = d.KH; p.KW = d.KW;
    p.sh = d.stride_h; p.sw = d.stride_w; p.ph = d.pad_h; p.pw = d.pad_w;
    p.OH = (d.H + 2 * d.pad_h - d.KH) / d.stride_h + 1;
    p.OW = (d.W + 2 * d.pad_w - d.KW) / d.stride_w + 1;
    p.M = (int64_t)d.N * p.OH * p.OW;
    p.K = d.KH * d.KW * d.C;
    p.tile = tile;
    // dense rows: one image row after the other, 16 bytes of slack before the first
    int64_t unit, rowbytes;
    if (nib) {
        if (((int64_t)d.W * d.C) % 8 != 0 || (uintptr_t)X % 4 != 0) return 0;
        unit = d.C;                                                // nibbles per pixel
        rowbytes = (int64_t)d.W * d.C / 2;
    } else {
        if (d.C % 8 != 0 || (uintptr_t)X % 4 != 0) return 0;
        unit = d.C / 2;
        rowbytes = (int64_t)d.W * unit;
    }
    const int64_t data0 = 16, pitch = rowbytes;
    const int64_t pix0 = nib ? 2 * data0 - (int64_t)d.pad_w * d.C : data0 - d.pad_w * unit;
    // a tile's consecutive pixels touch at most `rows` output rows in `nseg` images
    const int64_t rows = (tile - 1 + p.OW - 1) / p.OW + 1;
    const int64_t nseg = (rows - 1 + p.OH - 1) / p.OH + 1;
    const int64_t slots = rows * d.stride_h + nseg * (d.KH > d.stride_h ? d.KH - d.stride_h : 0);
    const int64_t bufbytes = (16 + slots * pitch + 32 + 15) / 16 * 16;     // slack on both sides for the edge windows' over-read
    p.unit = (int32_t)unit; p.rowbytes = (int32_t)rowbytes; p.data0 = (int32_t)data0; p.pix0 = (int32_t)pix0;
    p.pitch = (int32_t)pitch; p.bufbytes = (int32_t)bufbytes; p.segw = 1; p.KS = 0;
    p.sfull = (p.OH - 1) * d.stride_h + d.KH;
    p.vec16 = rowbytes % 16 == 0 && (uintptr_t)X % 16 == 0;
    if (rowbytes % 4 != 0) return 0;
    // bytes per asynchronous copy where rows are not whole 16-byte pieces
    p.cpr = (rowbytes % 8 == 0 && (uintptr_t)X % 8 == 0) ? 8 : 4;
    p.div_ow = make_fastdiv((uint32_t)p.OW);
    p.div_oh = make_fastdiv((uint32_t)p.OH);
    p.div_sfull = make_fastdiv((uint32_t)p.sfull);
    p.div_cpr = make_fastdiv((uint32_t)p.cpr);
    p.step8 = p.rowwrap = p.imgwrap = 0;
    return bufbytes;
}

template <class S, int G>
cudaError_t launch_instance(const fused::Params& p, cudaStream_t st)
{
    using L = convtc::Layout<S>;
    auto kernel = p.mult_ch ? convtc::conv_tc_kernel<S, G, true> : convtc::conv_tc_kernel<S, G, false>;
    const size_t smem = (size_t)L::FIXED + (size_t)p.nbuf * (size_t)p.bufbytes;
    if (p.nbuf < G || p.nbuf <= convtc::PWN || smem > (size_t)convtc::SMEM_LIMIT) return cudaErrorInvalidValue;
    // the attribute is per kernel and per device: set on every call, it is cheap
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         convtc::SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        sms = 148;
    const int64_t tiles = (p.M + S::TILE - 1) / S::TILE;
    const int grid = p.prep_out ? 1 : (int)(tiles < sms ? tiles : sms);      // preparation: one CTA, no tiles
    // Programmatic stream serialization: the grid may be scheduled while the previous
    // kernel of the stream drains; the kernel itself waits (griddepcontrol.wait) before it
    // touches memory.
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((convtc::PWN + 1 + 4 * G) * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kernel, p);
    count_launch();
    return e;
}

// Input buffers of the ring: enough bytes in flight to cover the memory latency (about
// 64 KB per SM), more than there are producer warps and at least one per worker group, at
// most NBMAX, within the shared-memory limit; 0 = no room.
template <class S>
int ring_size(const fused::Params& p)
{
    const int64_t room = ((int64_t)convtc::SMEM_LIMIT - convtc::Layout<S>::FIXED) / p.bufbytes;
    int64_t nb = (64 * 1024 + p.bufbytes - 1) / p.bufbytes + 2;
#ifdef Q4_CTC_NB
    nb = Q4_CTC_NB;
#endif
    const int64_t least = convtc::GMAX > convtc::PWN + 1 ? convtc::GMAX : convtc::PWN + 1;
    if (nb > convtc::NBMAX) nb = convtc::NBMAX;
    if (nb < least) nb = least;
    if (nb > room) nb = room;
    return nb < least ? 0 : (int)nb;
}

using convtc::Shape;
using S_gray  = Shape<0, 1, 3, 3, Q4_CTC_P0, 8, 0>;      // 1 -> 8 channels, stride 1
using S_8_16  = Shape<1, 2, 3, 3, Q4_CTC_P1, 16, 3>;     // 8 -> 16, stride 2
using S_16_32 = Shape<2, 2, 3, 3, Q4_CTC_P2, 32, 2>;     // 16 -> 32, stride 2
using S_32_64 = Shape<4, 2, 3, 3, Q4_CTC_P3, 64, 0>;     // 32 -> 64, stride 2
using S_16_32s1 = Shape<2, 1, 3, 3, Q4_CTC_P4, 32, 2>;   // 16 -> 32, stride 1

}  // namespace

static int ring_for(int id, const fused::Params& p)
{
    switch (id) {
        case 0: return ring_size<S_gray>(p);
        case 1: return ring_size<S_8_16>(p);
        case 2: return ring_size<S_16_32>(p);
        case 3: return ring_size<S_32_64>(p);
        default: return ring_size<S_16_32s1>(p);
    }
}

// The run-time-geometry kernel for layers with C a multiple of 32: fills the plan and the
// dynamic shared memory it needs; false = the layer does not fit it.
static bool plan_wide(fused::Params& p, const q4_conv_desc& d, const uint8_t* X, const uint8_t* Y, size_t* smem)
{
    if (d.C % 32 != 0 || d.OC % 32 != 0 || d.OC < 32) return false;
    if ((uintptr_t)X % 16 != 0 || (uintptr_t)Y % 16 != 0) return false;
    const int nsplit = (d.OC + 127) / 128;
    const int N = d.OC / nsplit;
    if (N * nsplit != d.OC || N % 32 != 0) return false;
    const int64_t KS = (int64_t)d.KH * d.KW * d.C / 32;
    if (KS < 1 || KS > 4096) return false;
    const int64_t bufbytes = plan_staging(p, d, X, convtc::ROWS, false);
    if (bufbytes <= 0 || !p.vec16) return false;
    const int64_t fixed = convtc::wide_layout(N, (int)KS).off_buf + 1024;
    const int64_t least = convtc::WPW + 2;             // the ring: more buffers than producer warps
    int64_t nb = (64 * 1024 + bufbytes - 1) / bufbytes + 2;
    const int64_t room = (convtc::SMEM_LIMIT_WIDE - fixed) / bufbytes;
    if (nb > convtc::NBMAX) nb = convtc::NBMAX;
    if (nb < least) nb = least;
    if (nb > room) nb = room;
    if (nb < least) return false;
    p.nbuf = (int32_t)nb;
    p.KS = (int32_t)KS;
    p.tcN = N; p.tcSplit = nsplit; p.OCtot = d.OC;
    *smem = (size_t)(fixed + nb * bufbytes);
    return true;
}

static cudaError_t launch_wide(const fused::Params& p, size_t smem, cudaStream_t st)
{
    auto kernel = p.mult_ch ? convtc::conv_tc_wide_kernel<true> : convtc::conv_tc_wide_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         convtc::SMEM_LIMIT_WIDE);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        sms = 148;
    const int64_t ptiles = (p.M + convtc::ROWS - 1) / convtc::ROWS;
    int64_t grid = ptiles * p.tcSplit < sms ? ptiles * p.tcSplit : sms / p.tcSplit * p.tcSplit;
    if (grid < p.tcSplit) grid = p.tcSplit;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(convtc::WIDE_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kernel, p);
    count_launch();
    return e;
}

bool conv_tc_supported(const q4_conv_desc& d, const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                       const uint8_t* Y)
{
    (void)Wt; (void)ldw;
    const TcChoice c = choose_instance(d);
    if (c.id < 0) {
        fused::Params pw;
        size_t smem = 0;
        return plan_wide(pw, d, X, Y, &smem);
    }
    if ((uintptr_t)Y % 16 != 0) return false;
    const int OW = (d.W + 2 * d.pad_w - d.KW) / d.stride_w + 1;
    if (OW % c.P != 0) return false;
    fused::Params p;
    const int64_t bufbytes = plan_staging(p, d, X, convtc::ROWS * c.P, c.nib);
    if (bufbytes <= 0) return false;
    // a row's first window word must sit at the same place of its 16-byte line in every row
    if (!c.nib && (!p.vec16 || (c.P * d.stride_w * p.unit) % 16 != 0)) return false;
    return ring_for(c.id, p) > 0;
}

// What a weight image is for: everything its contents depend on besides the weights, their zero
// point and the bias -- the kernel (instance or run-time geometry, with its pixels per row), the
// filter, the channel counts, the horizontal stride, za, and this build's image format.  Batch,
// image size, vertical stride and paddings do not enter: one image serves them all.
static uint32_t image_tag(const q4_conv_desc& d, int32_t za, int instance, int P)
{
    const uint32_t f[] = {0x51345747u /* format 1 */, (uint32_t)instance, (uint32_t)P, (uint32_t)d.C, (uint32_t)d.OC,
                          (uint32_t)d.KH, (uint32_t)d.KW, (uint32_t)d.stride_w, (uint32_t)za};
    uint32_t h = 2166136261u;                          // FNV-1a over the words' bytes
    for (uint32_t w : f)
        for (int b = 0; b < 4; ++b) { h ^= (w >> (8 * b)) & 0xFFu; h *= 16777619u; }
    return h ? h : 1u;
}

template <class S> static size_t image_bytes_of() { return (size_t)S::B_BYTES + (size_t)S::N * 4 + 16; }

// Bytes of the prepared weight image of a layer (see launch_conv_tc), 0 if no tensor-memory
// kernel serves the layer's geometry.
size_t conv_tc_image_bytes(const q4_conv_desc& d)
{
    if (!conv_tc_supported(d, nullptr, nullptr, 0, nullptr)) return 0;
    const TcChoice c = choose_instance(d);
    switch (c.id) {
        case 0: return image_bytes_of<S_gray>();
        case 1: return image_bytes_of<S_8_16>();
        case 2: return image_bytes_of<S_16_32>();
        case 3: return image_bytes_of<S_32_64>();
        case 4: return image_bytes_of<S_16_32s1>();
        default: break;
    }
    fused::Params p{};
    size_t smem = 0;
    if (!plan_wide(p, d, nullptr, nullptr, &smem)) return 0;
    return (size_t)p.tcSplit * ((size_t)convtc::wide_layout(p.tcN, p.KS).off_tab + (size_t)p.tcN * 4 + 16);
}

// prep_out: only prepare the weights (B operand, per-column constants, fallback flag) into
// that buffer of conv_tc_image_bytes(d) bytes; X and Y are not touched.  prep_in: run the layer
// from such an image; Wt, colsum_w, bias and zb are not read.  mult_ch / shift_ch (both or
// neither) and zb_ch (optional): per output channel; zb, rq.mult and rq.shift are then unused.
cudaError_t launch_conv_tc(const uint8_t* X, const uint8_t* Wt, int64_t ldw, const int32_t* colsum_w,
                           const int32_t* bias, const q4_conv_desc& d, int32_t za, int32_t zb,
                           const RequantParams& rq, uint8_t* Y, cudaStream_t st, const uint8_t* prep_in,
                           uint8_t* prep_out, const int32_t* zb_ch, const int32_t* mult_ch,
                           const int32_t* shift_ch)
{
    if (mult_ch && (prep_in || prep_out)) return cudaErrorInvalidValue;    // images are per-tensor
    const TcChoice c = choose_instance(d);
    if (c.id < 0) {
        fused::Params p{};
        size_t smem = 0;
        if (!plan_wide(p, d, X, Y, &smem)) return cudaErrorInvalidValue;
        p.X = X; p.Wt = Wt; p.ldw = ldw; p.colsum_w = colsum_w; p.bias = bias; p.Y = Y;
        p.zb_ch = zb_ch; p.mult_ch = mult_ch; p.shift_ch = shift_ch;
        p.za = za; p.zb = zb; p.rq = rq;
        p.wt_words = (uintptr_t)Wt % 4 == 0 && ldw % 4 == 0;
        p.prep_in = prep_in; p.prep_out = prep_out; p.prep_tag = image_tag(d, za, 100, 1);
        p.status = device_status_ptr();
        if (!p.status) return cudaErrorUnknown;
        if (prep_out) p.M = 0;                         // no tiles: the CTAs prepare their shares and leave
        else if (p.M == 0) return cudaSuccess;
        log_choice(prep_out ? "q4_conv2d_prepare_weights" : "q4_conv2d",
                   "fused implicit GEMM on tcgen05, run-time geometry (C a multiple of 32)");
        return launch_wide(p, smem, st);
    }
    fused::Params p{};
    if (plan_staging(p, d, X, convtc::ROWS * c.P, c.nib) <= 0) return cudaErrorInvalidValue;
    p.X = X; p.Wt = Wt; p.ldw = ldw; p.colsum_w = colsum_w; p.bias = bias; p.Y = Y;
    p.zb_ch = zb_ch; p.mult_ch = mult_ch; p.shift_ch = shift_ch;
    p.za = za; p.zb = zb; p.rq = rq;
    p.wt_words = (uintptr_t)Wt % 4 == 0 && ldw % 4 == 0;
    p.nbuf = ring_for(c.id, p);
    p.prep_in = prep_in; p.prep_out = prep_out; p.prep_tag = image_tag(d, za, c.id, c.P);
    p.status = device_status_ptr();
    if (!p.status) return cudaErrorUnknown;
    if (prep_out) p.M = 0;                             // no tiles: one CTA prepares the image and leaves
    else if (p.M == 0) return cudaSuccess;
    log_choice(prep_out ? "q4_conv2d_prepare_weights" : "q4_conv2d",
               "fused implicit GEMM on tcgen05 (A built in tensor memory)");
    switch (c.id) {
        case 0: return launch_instance<S_gray, Q4_CTC_G0>(p, st);
        case 1: return launch_instance<S_8_16, Q4_CTC_G1>(p, st);
        case 2: return launch_instance<S_16_32, Q4_CTC_G2>(p, st);
        case 3: return launch_instance<S_32_64, Q4_CTC_G3>(p, st);
        default: return launch_instance<S_16_32s1, Q4_CTC_G4>(p, st);
    }
}

#ifdef Q4_CTC_TRACE
extern "C" int q4_debug_set_trace(long long* buf)
{
    return (int)cudaMemcpyToSymbol(convtc::g_trace, &buf, sizeof(buf));
}
#endif

}  // namespace q4
