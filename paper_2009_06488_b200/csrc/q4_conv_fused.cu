// Fused quantized convolution layer: the unrolled activation matrix of GEMM-based
// convolution (Section I; depth D = kh*kw*c, Section III-A) is never written to
// memory.  A CTA takes 224 consecutive output pixels.  It first copies the input rows
// those pixels touch into shared memory -- with the padding materialised as the input
// zero point, so the gather below needs no bounds checks -- while the previous tile is
// still being multiplied (a ring of buffers).  Each warp then gathers its 32 pixels' taps from
// that copy into the A fragments of the warp-level integer MMA (u8 x s8 -> s32,
// m16n8k32), multiplies against the layer's weights held as B fragments in shared
// memory, and applies the remaining zero-point term of Eq. 3, the bias, the
// re-quantization and the nibble packing to the accumulators it holds.
//
// Zero points.  The B fragments hold w - zb as signed bytes, so the accumulator is
// sum a*(w - zb) = sum a*w - zb*sum a: Eq. 2's second term (the row sums taken "while
// unrolling", Section II-B) is absorbed by the multiplication and never formed.  What
// is left of Eq. 3 is one constant per output channel, K*za*zb - za*sum w.
//
// Two input modes:
//  * packed   (C % 8 == 0, X 4-byte aligned): the copy in shared memory stays packed;
//    a 32-bit word of a tap is split into its even and odd nibbles, which are exactly
//    the two A registers of one thread, the same depth permutation being applied to
//    the weights;
//  * expanded (any C, e.g. the single-channel first layer): pixels are nibble-granular,
//    so the copy in shared memory holds one byte per value; the depth is laid out as
//    KH segments of KW*C contiguous bytes, each padded to a multiple of four with zero
//    weights, and an A register is one (possibly unaligned) 32-bit word of a segment.
//
// Why not the tcgen05 path here: these layers have tiny depth and few output channels
// (K = 9..288, N = 8..64), so the work per output tile is a few hundred clocks of
// tensor time -- far less than the hand-offs of a TMA / tensor-memory pipeline -- and
// the traffic saved by not materialising the unrolled matrix (2 * M * K/2 bytes) is
// what matters.
//
// Requirements (else the caller falls back to unroll + GEMM): OC a multiple of 8 up to
// 64, Y 8-byte aligned, and the weights, tables and the ring of input buffers fit in
// shared memory.
#include <type_traits>

#include "q4_common.cuh"
#include "q4_conv_stage.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {

unsigned* device_status_ptr();     // the device status word (q4_api.cu)

namespace fused {

constexpr int WARPS = 7;                 // multiplying warps; one more warp produces
constexpr int ROWS_PER_WARP = 32;
constexpr int ROWS_PER_CTA = WARPS * ROWS_PER_WARP;
constexpr int SMEM_LIMIT = 160 * 1024;
constexpr int NBUF_MMA = 3;              // input buffers: the producer runs NBUF - 1 tiles ahead
constexpr int NBUF_LANE = 4;
constexpr int SYNC_BYTES = 96;             // the buffers' "landed" and "read" mbarriers and the abort flag

__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
        "{%8, %9}, {%0, %1, %2, %3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ int dp4a_u8s8(uint32_t a, uint32_t b, int c)
{
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// A multiplying warp is done reading a buffer.
__device__ __forceinline__ void release_buffer(uint32_t empty_bar, int lane)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(empty_bar);
}

// NT = OC / 8 output-channel tiles.  Fragment column f of tile nt is output channel
// 2 * (NT * (f / 2) + nt) + f % 2, so that the NT packed output bytes a thread ends up
// with are contiguous in memory.
//
// Warps 0..6 multiply; warp 7 is the producer: it runs up to NB tiles ahead, deriving a
// tile's geometry and copying its input rows into the next buffer of the ring.  Buffers
// change hands through two mbarriers each ("landed", "read"), so no warp waits for
// another multiplying warp.
constexpr int THREADS = (WARPS + 1) * 32;


// KS_T: the number of depth steps when known at compile time (packed mode only): the loop
// over the depth unrolls and each thread keeps its tap offsets in registers; 0 = taken
// from the parameters.
// CONSEC (with KS_T; output rows are whole groups of four pixels): the four MMA rows a thread
// feeds and reads back (g, g + 8, g + 16, g + 24 of its warp's two 16-row tiles) are assigned
// to four CONSECUTIVE pixels 4g .. 4g + 3 instead of pixels eight apart -- which pixel an MMA
// row stands for is free --, so a thread decodes one pixel per tile and the other three are
// a constant step away.
// PC: every output channel has its own weight zero point and re-quantization multiplier
// and shift (device arrays in the parameters) instead of the layer-wide ones.
template <int NT, bool EXP, int KS_T = 0, bool CONSEC = false, bool PC = false>
__global__ void __launch_bounds__(THREADS, NT <= 2 ? 4 : NT <= 4 ? 3 : 2)
conv_fused_kernel(const Params p)
{
    static_assert(!(EXP && KS_T), "the unrolled depth loop is for the packed mode");
    static_assert(!CONSEC || KS_T, "consecutive pixels per thread come with the unrolled depth loop");
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int TW = EXP ? 8 : 4;                    // table entries per depth step
    constexpr int N = 8 * NT;
    uint2* bfrag = reinterpret_cast<uint2*>(smem);                                   // [KS][NT][32]
    int32_t* tab = reinterpret_cast<int32_t*>(smem + (size_t)p.KS * NT * 32 * 8);    // [KS][TW]
    int32_t* colsum_s = tab + p.KS * TW;                                             // [N]
    constexpr int NB = NBUF_MMA;
    int32_t* pc_s = colsum_s + N;                                                    // [2][N] multipliers, shifts (PC)
    int4* geo_s = reinterpret_cast<int4*>(pc_s + 2 * N);                             // [NB]
    uint64_t* full_s = reinterpret_cast<uint64_t*>(geo_s + NB);                      // [NB] "tile landed"
    uint8_t* buf0 = reinterpret_cast<uint8_t*>(geo_s + NB) + SYNC_BYTES;             // 16-byte aligned
    const uint32_t full0 = smem_u32(full_s), empty0 = full0 + 8 * NB, abort_flag = full0 + 16 * NB;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int kbytes = p.K / 2;                        // packed mode: K is a multiple of 8
    const int segbytes = p.KW * p.C;                   // expanded mode: bytes per kh segment

    // ---- once per CTA: weights -> signed B fragments, depth table, weight sums, and
    //      the input buffers filled with the zero point (this is what stays in the halo)
    for (int i = tid; i < N; i += THREADS) colsum_s[i] = 0;
    int pc_fast = 1;                                   // every channel's shift allows the 32-bit rounding
    if (PC) {
        int ok = 1;
        for (int i = tid; i < N; i += THREADS) {
            pc_s[i] = p.mult_ch[i];
            pc_s[N + i] = p.shift_ch[i];
            ok = ok && p.shift_ch[i] >= 2;
        }
        pc_fast = __syncthreads_and(ok);
    }
    {
        const uint32_t zfill = (uint32_t)p.za * (EXP ? 0x01010101u : 0x11111111u);
        uint32_t* b = reinterpret_cast<uint32_t*>(buf0);
        for (int i = tid; i < NB * p.bufbytes / 4; i += THREADS) b[i] = zfill;
        fence_async_smem();                            // before the copy engine writes the same bytes
    }
    if (tid == 0) {
        for (int i = 0; i < NB; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, WARPS);
        }
        sts32(abort_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    for (int i = tid; i < p.KS * NT * 32; i += THREADS) {
        const int l = i & 31, nt = (i >> 5) % NT, j = (i >> 5) / NT;
        const int fg = l >> 2, ft = l & 3;
        const int n = 2 * (NT * (fg >> 1) + nt) + (fg & 1);
        const uint32_t zbn = PC ? (uint32_t)p.zb_ch[n] : (uint32_t)p.zb;
        uint32_t b0 = 0, b1 = 0;
        int raw = 0;
        if (!EXP) {
            const int kb = 16 * j + 4 * ft;
            if (kb < kbytes) {
                uint32_t w;
                if (p.wt_words) {
                    w = *reinterpret_cast<const uint32_t*>(p.Wt + (int64_t)n * p.ldw + kb);
                } else {
                    w = 0;
                    for (int q = 0; q < 4; ++q) w |= (uint32_t)p.Wt[(int64_t)n * p.ldw + kb + q] << (8 * q);
                }
                raw = nibble_sum(w);
                b0 = sub_zb(w & 0x0F0F0F0Fu, zbn);
                b1 = sub_zb((w >> 4) & 0x0F0F0F0Fu, zbn);
            }
        } else {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int wi = 8 * j + 4 * h + ft;
                const int kh = wi / p.segw, ws = wi % p.segw;
                uint32_t word = 0;
                if (kh < p.KH) {
                    for (int q = 0; q < 4; ++q) {
                        const int bs = 4 * ws + q;
                        if (bs < segbytes) {
                            const uint32_t nib = weight_nibble(p, n, kh * segbytes + bs);
                            raw += (int)nib;
                            word |= ((nib - zbn) & 0xFFu) << (8 * q);
                        }
                    }
                }
                if (h == 0) b0 = word; else b1 = word;
            }
        }
        bfrag[i] = make_uint2(b0, b1);
        if (!p.colsum_w && raw) atomicAdd(&colsum_s[n], raw);
    }
    for (int i = tid; i < p.KS * TW; i += THREADS) {
        int delta = -1;
        if (!EXP) {
            const int kb = 16 * (i >> 2) + 4 * (i & 3);
            if (kb < kbytes) {
                const int kh = kb / (p.KW * p.unit);
                delta = kh * p.pitch + (kb - kh * p.KW * p.unit);
            }
        } else {
            const int kh = i / p.segw, ws = i % p.segw;      // i = 8 j + 4 h + t
            if (kh < p.KH) delta = kh * p.pitch + 4 * ws;
        }
        tab[i] = delta;
    }
    __syncthreads();

    // This CTA's tiles: blockIdx.x, blockIdx.x + gridDim.x, ... (the grid never exceeds the
    // tile count).
    const int64_t ntiles = (p.M + ROWS_PER_CTA - 1) / ROWS_PER_CTA;
    const int mytiles = (int)((ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x);

    if (warp == WARPS) {
        // ---------------- producer ----------------
        producer_loop<NB, EXP>(p, mytiles, buf0, geo_s, full0, empty0, abort_flag, lane);
        return;
    }

    // ---------------- consumers ----------------
    // per-thread epilogue constants: what is left of Eq. 3 for my NT channel pairs
    int colterm[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int n = 2 * (NT * t + nt) + e;
            const int cs = p.colsum_w ? p.colsum_w[n] : colsum_s[n];
            const int kzz = p.K * p.za * (PC ? p.zb_ch[n] : p.zb);
            colterm[nt][e] = (int)((uint32_t)kzz - (uint32_t)(p.za * cs) +
                                   (uint32_t)(p.bias ? p.bias[n] : 0));
        }
    const int pix0 = p.pix0;
    const int yoff = (warp * ROWS_PER_WARP + (CONSEC ? 4 * g : g)) * (N / 2) + NT * t;    // my first row within a tile
    // my tap offset of every depth step; steps past the depth read offset 0 (any valid place:
    // their weights are zero)
    int dl[KS_T ? KS_T : 1];
#pragma unroll
    for (int j = 0; j < KS_T; ++j) {
        const int d = tab[4 * j + t];
        dl[j] = d < 0 ? 0 : d;
    }

    // pixel indices fit 32 bits (M < 2^31, and a tile starts below M)
    const uint32_t M32 = (uint32_t)p.M, mstep = gridDim.x * (uint32_t)ROWS_PER_CTA;
    uint32_t mbase = blockIdx.x * (uint32_t)ROWS_PER_CTA;
    int kb = 0;                                        // k % NB
    uint32_t phase = 0;                                // (k / NB) % 2
    for (int k = 0; k < mytiles; ++k, mbase += mstep) {
        const uint8_t* buf = buf0 + kb * p.bufbytes;
        mbar_wait_suspend(full0 + 8 * kb, phase, abort_flag, p.status);    // the tile's rows have landed
        const int4 gv = geo_s[kb];                     // n_first, oh_first, s0 (published with the tile)
        const uint32_t done_bar = empty0 + 8 * kb;
        if (++kb == NB) { kb = 0; phase ^= 1; }
        const uint32_t left = M32 - mbase;             // > 0
        const int myrows = (int)(left < (uint32_t)ROWS_PER_CTA ? left : (uint32_t)ROWS_PER_CTA) -
                           warp * ROWS_PER_WARP;
        if (myrows > 0) {                              // warp-uniform
            // my four rows: g, g+8 (first 16-row tile), 16+g, 24+g (second)
            int base[4], shf[4];
            if (CONSEC) {
                // pixels 4g .. 4g + 3 of my warp: same output row (rows are whole groups of four,
                // so the tile's pixel count, a multiple of four, is reached group-wise)
                const uint32_t mm = mbase + (uint32_t)(warp * ROWS_PER_WARP) +
                                    (uint32_t)(4 * g < myrows ? 4 * g : 0);
                const uint32_t q = fdiv(mm, p.div_ow);
                const int ow = (int)(mm - q * (uint32_t)p.OW);
                const uint32_t n0 = fdiv(q, p.div_oh);
                const int oh = (int)(q - n0 * (uint32_t)p.OH);
                const int seg = (int)n0 - gv.x;
                const int slot0 = seg == 0 ? (oh - gv.y) * p.sh : gv.z + (seg - 1) * p.sfull + oh * p.sh;
                const int b = slot0 * p.pitch + pix0 + ow * p.sw * p.unit;
                const int step = p.step8 >> 3;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    shf[i] = 0;
                    base[i] = b + i * step;
                }
            } else {
                const uint32_t mm = mbase + (uint32_t)(warp * ROWS_PER_WARP) +
                                    (uint32_t)(g < myrows ? g : 0);
                const uint32_t q = fdiv(mm, p.div_ow);
                int ow = (int)(mm - q * (uint32_t)p.OW);
                const uint32_t n0 = fdiv(q, p.div_oh);
                int oh = (int)(q - n0 * (uint32_t)p.OH);
                int seg = (int)n0 - gv.x;
                const int slot0 = seg == 0 ? (oh - gv.y) * p.sh : gv.z + (seg - 1) * p.sfull + oh * p.sh;
                int b = slot0 * p.pitch + pix0 + ow * p.sw * p.unit;
                const int first = b;
                if (p.OW >= 8) {
                    // eight pixels on: at most one step into the next output row (+sh staged
                    // rows), which may be the next image's first (+KH instead)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int bi = g + 8 * i < myrows ? b : first;   // rows past the end read a valid place
                        shf[i] = (bi & 3) * 8;
                        base[i] = EXP ? (bi & ~3) : bi;
                        ow += 8;
                        b += p.step8;
                        if (ow >= p.OW) {
                            ow -= p.OW;
                            b += p.rowwrap;
                            if (++oh == p.OH) { oh = 0; b += p.imgwrap; }
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int s0i = seg == 0 ? (oh - gv.y) * p.sh : gv.z + (seg - 1) * p.sfull + oh * p.sh;
                        const int bb = s0i * p.pitch + pix0 + ow * p.sw * p.unit;
                        const int bi = g + 8 * i < myrows ? bb : first;
                        shf[i] = (bi & 3) * 8;
                        base[i] = EXP ? (bi & ~3) : bi;
                        ow += 8;
                        while (ow >= p.OW) {
                            ow -= p.OW;
                            if (++oh == p.OH) { oh = 0; ++seg; }
                        }
                    }
                }
            }
            int acc[2][NT][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[mt][nt][e] = colterm[nt][e & 1];   // columns 2t + e % 2

#pragma unroll
            for (int j = 0; j < (KS_T ? KS_T : p.KS); ++j) {
                uint32_t a[2][4];
                if (!EXP) {
                    // one packed word per row: even nibbles feed depth 4t.., odd ones 16+4t..
                    const int delta = KS_T ? dl[KS_T ? j : 0] : tab[4 * j + t];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t w = 0;
                        if (KS_T || delta >= 0) w = *reinterpret_cast<const uint32_t*>(buf + base[i] + delta);
                        a[0][i] = w & 0x0F0F0F0Fu;
                        a[1][i] = (w >> 4) & 0x0F0F0F0Fu;
                    }
                } else {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int delta = tab[8 * j + 4 * h + t];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint32_t w = 0;
                            if (delta >= 0) {
                                const uint32_t* src = reinterpret_cast<const uint32_t*>(buf + base[i] + delta);
                                w = __funnelshift_r(src[0], src[1], shf[i]);
                            }
                            a[h][i] = w;
                        }
                    }
                }
                const uint2* bj = bfrag + (size_t)j * NT * 32 + lane;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint2 b = bj[nt * 32];
                    mma_u8s8(acc[0][nt], a[0][0], a[0][1], a[1][0], a[1][1], b.x, b.y);
                    mma_u8s8(acc[1][nt], a[0][2], a[0][3], a[1][2], a[1][3], b.x, b.y);
                }
            }

            // epilogue: accumulator (mt, nt) holds rows g + 16 mt (c0, c1) and g + 8 + 16 mt
            // (c2, c3), fragment columns 2t, 2t+1
            uint8_t* ytile = p.Y + (uint64_t)mbase * (N / 2) + yoff;
            auto epilogue = [&](auto fast_tag) {
                constexpr bool FAST = decltype(fast_tag)::value;
                const int s = p.rq.shift - 1, rnd = FAST ? 1 << (s - 1) : 0;
                const int zml = p.rq.zo - p.rq.lo, hml = p.rq.hi - p.rq.lo;
                const uint32_t lofill = (uint32_t)p.rq.lo * 0x11111111u;     // lo in every nibble
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int mt = i >> 1, hrow = i & 1;
                    if ((CONSEC ? 4 * g + i : g + 8 * i) >= myrows) continue;
                    uint32_t bytes[NT];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        uint32_t qv[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int v = acc[mt][nt][2 * hrow + e];       // started from the column's constant
                            if (PC) {
                                const int n = 2 * (NT * t + nt) + e;
                                const int mlt = pc_s[n], sh = pc_s[N + n];
                                if (FAST) {
                                    qv[e] = clamp_above_lo(mulhi_add(v, mlt, 1 << (sh - 2)) >> (sh - 1), zml, hml);
                                } else {
                                    const RequantParams rqn{mlt, sh, p.rq.zo, p.rq.lo, p.rq.hi};
                                    qv[e] = requant_wide(v, rqn) - (uint32_t)p.rq.lo;
                                }
                            } else if (FAST) {
                                qv[e] = clamp_above_lo(mulhi_add(v, p.rq.mult, rnd) >> s, zml, hml);
                            } else {
                                qv[e] = requant_wide(v, p.rq) - (uint32_t)p.rq.lo;
                            }
                        }
                        bytes[nt] = mad_u32(qv[1], 16u, qv[0]);     // fields do not overlap: add = or
                    }
                    uint8_t* dst = ytile + (CONSEC ? i : 8 * i) * (N / 2);
                    if (NT % 4 == 0) {
#pragma unroll
                        for (int q = 0; q < NT / 4; ++q)
                            reinterpret_cast<uint32_t*>(dst)[q] =
                                mad_u32(bytes[(4 * q + 3) % NT], 1u << 24,
                                        mad_u32(bytes[(4 * q + 2) % NT], 1u << 16,
                                                mad_u32(bytes[(4 * q + 1) % NT], 1u << 8,
                                                        bytes[(4 * q) % NT] + lofill)));
                    } else if (NT % 2 == 0) {
#pragma unroll
                        for (int q = 0; q < NT / 2; ++q)
                            reinterpret_cast<uint16_t*>(dst)[q] =
                                (uint16_t)mad_u32(bytes[(2 * q + 1) % NT], 1u << 8, bytes[(2 * q) % NT] + lofill);
                    } else {
#pragma unroll
                        for (int q = 0; q < NT; ++q) dst[q] = (uint8_t)(bytes[q] + lofill);
                    }
                }
            };
            // the 32-bit form of the rounding shift needs shift >= 2 (see requant())
            if (PC ? pc_fast != 0 : p.rq.shift >= 2) epilogue(std::true_type{}); else epilogue(std::false_type{});
        }
        release_buffer(done_bar, lane);
    }
}


// ---------------------------------------------------------------------------------
// One output pixel per lane.  For the thinnest layers (a single-channel first layer:
// depth 9 or 25, eight outputs) an MMA tile is almost empty and the fragment layout --
// four pixels per thread, two columns each -- costs more index arithmetic than the layer
// has multiplications.  Here a lane owns one pixel and all its output channels: it reads
// its taps from the same expanded copy in shared memory, one 32-bit word of a kh segment
// at a time, and multiplies with 4-way byte dot products (u8 x s8) against weight words
// that every lane reads from the same shared-memory address.  The packed output of a
// pixel is one 4- or 8-byte store, a warp's is contiguous.
// ---------------------------------------------------------------------------------
// KH_T, SEGW_T: the filter height and the words per kh segment when known at compile time
// (the loops over the depth unroll), 0 = taken from the parameters.
template <int OC, bool NIB, int KH_T, int SEGW_T>
__global__ void __launch_bounds__(THREADS, 3)
conv_lane_kernel(const Params p)
{
    const int KH = KH_T ? KH_T : p.KH, SEGW = SEGW_T ? SEGW_T : p.segw;
    extern __shared__ __align__(16) uint8_t smem[];
    const int nw = p.KH * p.segw;                      // 32-bit depth words per pixel
    uint32_t* wsm = reinterpret_cast<uint32_t*>(smem);                               // [nw][OC]
    int32_t* colterm_s = reinterpret_cast<int32_t*>(wsm + nw * OC);                  // [OC]
    constexpr int NB = NBUF_LANE;
    int4* geo_s = reinterpret_cast<int4*>(colterm_s + OC);                           // [NB]
    uint64_t* full_s = reinterpret_cast<uint64_t*>(geo_s + NB);                      // [NB] "tile landed"
    uint8_t* buf0 = reinterpret_cast<uint8_t*>(geo_s + NB) + SYNC_BYTES;             // 16-byte aligned
    const uint32_t full0 = smem_u32(full_s), empty0 = full0 + 8 * NB, abort_flag = full0 + 16 * NB;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int segbytes = p.KW * p.C;

    // ---- once per CTA: signed weight words, the constant left of Eq. 3, zero-point fill
    for (int i = tid; i < OC; i += THREADS) colterm_s[i] = 0;
    {
        uint32_t* b = reinterpret_cast<uint32_t*>(buf0);
        const uint32_t zfill = (uint32_t)p.za * (NIB ? 0x11111111u : 0x01010101u);
        for (int i = tid; i < NB * p.bufbytes / 4; i += THREADS) b[i] = zfill;
        fence_async_smem();                            // before the copy engine writes the same bytes
    }
    if (tid == 0) {
        for (int i = 0; i < NB; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, WARPS);
        }
        sts32(abort_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    for (int i = tid; i < nw * OC; i += THREADS) {
        const int n = i % OC, wi = i / OC;
        const int kh = wi / p.segw, ws = wi % p.segw;
        uint32_t word = 0;
        int raw = 0;
        for (int q = 0; q < 4; ++q) {
            const int bs = 4 * ws + q;
            if (bs < segbytes) {
                const uint32_t nib = weight_nibble(p, n, kh * segbytes + bs);
                raw += (int)nib;
                word |= ((nib - (uint32_t)p.zb) & 0xFFu) << (8 * q);
            }
        }
        wsm[i] = word;
        if (!p.colsum_w && raw) atomicAdd(&colterm_s[n], raw);
    }
    __syncthreads();
    if (tid < OC) {
        const int cs = p.colsum_w ? p.colsum_w[tid] : colterm_s[tid];
        colterm_s[tid] = (int)((uint32_t)(p.K * p.za * p.zb) - (uint32_t)(p.za * cs) +
                               (uint32_t)(p.bias ? p.bias[tid] : 0));
    }
    __syncthreads();

    const int64_t ntiles = (p.M + ROWS_PER_CTA - 1) / ROWS_PER_CTA;
    const int mytiles = (int)((ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x);

    if (warp == WARPS) {
        // ---------------- producer ----------------
        producer_loop<NB, !NIB>(p, mytiles, buf0, geo_s, full0, empty0, abort_flag, lane);
        return;
    }

    // ---------------- consumers ----------------
    const int pix0 = p.pix0;
    const int r = warp * ROWS_PER_WARP + lane;         // my pixel within a tile
    // pixel indices fit 32 bits (M < 2^31, and a tile starts below M)
    const uint32_t M32 = (uint32_t)p.M, mstep = gridDim.x * (uint32_t)ROWS_PER_CTA;
    uint32_t mbase = blockIdx.x * (uint32_t)ROWS_PER_CTA;
    int kb = 0;                                        // k % NB
    uint32_t phase = 0;                                // (k / NB) % 2
    for (int k = 0; k < mytiles; ++k, mbase += mstep) {
        const uint8_t* buf = buf0 + kb * p.bufbytes;
        mbar_wait_suspend(full0 + 8 * kb, phase, abort_flag, p.status);    // the tile's rows have landed
        const int4 gv = geo_s[kb];                     // n_first, oh_first, s0 (published with the tile)
        const uint32_t done_bar = empty0 + 8 * kb;
        if (++kb == NB) { kb = 0; phase ^= 1; }
        const uint32_t left = M32 - mbase;             // > 0
        const int rows = (int)(left < (uint32_t)ROWS_PER_CTA ? left : (uint32_t)ROWS_PER_CTA);
        if (warp * ROWS_PER_WARP < rows) {             // warp-uniform
            const bool valid = r < rows;
            const uint32_t mm = mbase + (uint32_t)(valid ? r : 0);
            const uint32_t q = fdiv(mm, p.div_ow);
            const int ow = (int)(mm - q * (uint32_t)p.OW);
            const uint32_t n0 = fdiv(q, p.div_oh);
            const int oh = (int)(q - n0 * (uint32_t)p.OH);
            const int seg = (int)n0 - gv.x;
            const int slot0 = seg == 0 ? (oh - gv.y) * p.sh : gv.z + (seg - 1) * p.sfull + oh * p.sh;
            // where my pixel's first tap starts: a byte offset (expanded copy), or a nibble
            // offset (packed copy); `shf` is its bit offset within the aligned word at `src`
            const int b = slot0 * p.pitch * (NIB ? 2 : 1) + pix0 + ow * p.sw * p.unit;
            const int shf = NIB ? (b & 7) * 4 : (b & 3) * 8;
            const uint8_t* src = buf + (NIB ? (b >> 3) << 2 : b & ~3);

            int acc[OC];
#pragma unroll
            for (int n = 0; n < OC; n += 4) {
                const int4 c = *reinterpret_cast<const int4*>(colterm_s + n);
                acc[n] = c.x; acc[n + 1] = c.y; acc[n + 2] = c.z; acc[n + 3] = c.w;
            }
            const uint32_t* wrow = wsm;
#pragma unroll
            for (int kh = 0; kh < KH; ++kh) {
                const uint32_t* arow = reinterpret_cast<const uint32_t*>(src + kh * p.pitch);
#pragma unroll
                for (int ws = 0; ws < SEGW; ++ws) {
                    uint32_t a;
                    if (NIB) {
                        // four nibbles -> four bytes
                        const int bo = shf + 16 * ws;
                        uint32_t x = __funnelshift_r(arow[bo >> 5], arow[(bo >> 5) + 1], bo & 31) & 0xFFFFu;
                        x = (x | (x << 8)) & 0x00FF00FFu;
                        a = (x | (x << 4)) & 0x0F0F0F0Fu;
                    } else {
                        a = __funnelshift_r(arow[ws], arow[ws + 1], shf);
                    }
#pragma unroll
                    for (int n = 0; n < OC; n += 4) {
                        const uint4 w = *reinterpret_cast<const uint4*>(wrow + n);
                        acc[n] = dp4a_u8s8(a, w.x, acc[n]);
                        acc[n + 1] = dp4a_u8s8(a, w.y, acc[n + 1]);
                        acc[n + 2] = dp4a_u8s8(a, w.z, acc[n + 2]);
                        acc[n + 3] = dp4a_u8s8(a, w.w, acc[n + 3]);
                    }
                    wrow += OC;
                }
            }

            uint32_t out[OC / 8];
            if (p.rq.shift >= 2) {
                // the 32-bit form of the rounding shift (see requant())
                const int s = p.rq.shift - 1, rnd = 1 << (s - 1);
#pragma unroll
                for (int n = 0; n < OC; ++n) {
                    int qv = (mulhi_add(acc[n], p.rq.mult, rnd) >> s) + p.rq.zo;
                    qv = min(max(qv, p.rq.lo), p.rq.hi);
                    if (n % 8 == 0) out[n / 8] = (uint32_t)qv; else out[n / 8] |= (uint32_t)qv << (4 * (n % 8));
                }
            } else {
#pragma unroll
                for (int n = 0; n < OC; ++n) {
                    const uint32_t qv = requant_wide(acc[n], p.rq);
                    if (n % 8 == 0) out[n / 8] = qv; else out[n / 8] |= qv << (4 * (n % 8));
                }
            }
            if (valid) {
                uint8_t* dst = p.Y + (uint64_t)(mbase + (uint32_t)r) * (OC / 2);
                if (OC == 8) *reinterpret_cast<uint32_t*>(dst) = out[0];
                else *reinterpret_cast<uint2*>(dst) = make_uint2(out[0], out[(OC / 8 - 1)]);
            }
        }
        release_buffer(done_bar, lane);
    }
}

// ---------------------------------------------------------------------------------
// Four horizontally adjacent output pixels per lane, for 3x3 stride-1 layers on a
// single-channel input with eight output channels (a gray-image first layer) whose
// output rows are whole groups of four.  The four pixels' taps of one filter row are
// six consecutive nibbles of the packed copy in shared memory: one unaligned 32-bit
// window per filter row is split into its even and odd nibbles (as bytes), from which
// each pixel's three taps are picked by one byte permutation.  Pixel decode, window
// loads and weight loads are paid once per four pixels, and a lane's 16 packed output
// bytes leave in one store (a warp's stores are 512 contiguous bytes).  A CTA tile is
// 4 * 224 pixels; staging protocol and weight set-up are those of conv_lane_kernel.
// ---------------------------------------------------------------------------------
constexpr int QUAD = 4;
constexpr int QUAD_TILE = QUAD * ROWS_PER_CTA;

template <bool PC>
__global__ void __launch_bounds__(THREADS, 4)
conv_quad_kernel(const Params p)
{
    constexpr int OC = 8, KH = 3;
    extern __shared__ __align__(16) uint8_t smem[];
    uint32_t* wsm = reinterpret_cast<uint32_t*>(smem);                               // [KH][OC]
    int32_t* colterm_s = reinterpret_cast<int32_t*>(wsm + KH * OC);                  // [OC]
    constexpr int NB = NBUF_LANE;
    int32_t* pc_s = colterm_s + OC;                                                  // [2][OC] multipliers, shifts (PC)
    int4* geo_s = reinterpret_cast<int4*>(pc_s + 2 * OC);                            // [NB]
    uint64_t* full_s = reinterpret_cast<uint64_t*>(geo_s + NB);                      // [NB] "tile landed"
    uint8_t* buf0 = reinterpret_cast<uint8_t*>(geo_s + NB) + SYNC_BYTES;             // 16-byte aligned
    const uint32_t full0 = smem_u32(full_s), empty0 = full0 + 8 * NB, abort_flag = full0 + 16 * NB;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- once per CTA: signed weight words, the constant left of Eq. 3, zero-point fill
    for (int i = tid; i < OC; i += THREADS) colterm_s[i] = 0;
    {
        uint32_t* b = reinterpret_cast<uint32_t*>(buf0);
        const uint32_t zfill = (uint32_t)p.za * 0x11111111u;
        for (int i = tid; i < NB * p.bufbytes / 4; i += THREADS) b[i] = zfill;
        fence_async_smem();                            // before the copy engine writes the same bytes
    }
    if (tid == 0) {
        for (int i = 0; i < NB; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, WARPS);
        }
        sts32(abort_flag, 0);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    for (int i = tid; i < KH * OC; i += THREADS) {
        const int n = i % OC, kh = i / OC;
        uint32_t word = 0;
        int raw = 0;
        for (int q = 0; q < 3; ++q) {
            const uint32_t nib = weight_nibble(p, n, kh * 3 + q);
            raw += (int)nib;
            word |= ((nib - (PC ? (uint32_t)p.zb_ch[n] : (uint32_t)p.zb)) & 0xFFu) << (8 * q);
        }
        wsm[i] = word;                                 // fourth byte 0: the window's next nibble counts for nothing
        if (!p.colsum_w && raw) atomicAdd(&colterm_s[n], raw);
    }
    __syncthreads();
    if (tid < OC) {
        const int cs = p.colsum_w ? p.colsum_w[tid] : colterm_s[tid];
        colterm_s[tid] = (int)((uint32_t)(p.K * p.za * (PC ? p.zb_ch[tid] : p.zb)) - (uint32_t)(p.za * cs) +
                               (uint32_t)(p.bias ? p.bias[tid] : 0));
        if (PC) {
            pc_s[tid] = p.mult_ch[tid];
            pc_s[OC + tid] = p.shift_ch[tid];
        }
    }
    const int pc_fast = PC ? __syncthreads_and(tid >= OC || p.shift_ch[tid] >= 2) : 1;
    __syncthreads();

    const int64_t ntiles = (p.M + QUAD_TILE - 1) / QUAD_TILE;
    const int mytiles = (int)((ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x);

    if (warp == WARPS) {
        // ---------------- producer ----------------
        producer_loop<NB, false>(p, mytiles, buf0, geo_s, full0, empty0, abort_flag, lane);
        return;
    }

    // ---------------- consumers ----------------
    const int r = warp * ROWS_PER_WARP + lane;         // my group of four within a tile
    const uint32_t M32 = (uint32_t)p.M, mstep = gridDim.x * (uint32_t)QUAD_TILE;
    uint32_t mbase = blockIdx.x * (uint32_t)QUAD_TILE;
    const int s = p.rq.shift - 1, rnd = s > 0 ? 1 << (s - 1) : 0;
    const int zml = p.rq.zo - p.rq.lo, hml = p.rq.hi - p.rq.lo;
    const uint32_t lofill = (uint32_t)p.rq.lo * 0x11111111u;         // lo in every nibble
    int kb = 0;                                        // k % NB
    uint32_t phase = 0;                                // (k / NB) % 2
    for (int k = 0; k < mytiles; ++k, mbase += mstep) {
        const uint8_t* buf = buf0 + kb * p.bufbytes;
        mbar_wait_suspend(full0 + 8 * kb, phase, abort_flag, p.status);    // the tile's rows have landed
        const int4 gv = geo_s[kb];                     // n_first, oh_first, s0 (published with the tile)
        const uint32_t done_bar = empty0 + 8 * kb;
        if (++kb == NB) { kb = 0; phase ^= 1; }
        const uint32_t left = M32 - mbase;             // > 0, a multiple of four
        const int groups = (int)(left < (uint32_t)QUAD_TILE ? left : (uint32_t)QUAD_TILE) / QUAD;
        if (warp * ROWS_PER_WARP < groups) {           // warp-uniform
            const bool valid = r < groups;
            const uint32_t mm = mbase + (uint32_t)(valid ? QUAD * r : 0);
            const uint32_t q = fdiv(mm, p.div_ow);
            const int ow = (int)(mm - q * (uint32_t)p.OW);
            const uint32_t n0 = fdiv(q, p.div_oh);
            const int oh = (int)(q - n0 * (uint32_t)p.OH);
            const int seg = (int)n0 - gv.x;
            const int slot0 = seg == 0 ? oh - gv.y : gv.z + (seg - 1) * p.sfull + oh;
            const int b = slot0 * p.pitch * 2 + p.pix0 + ow;       // nibble offset of my first tap
            const int shf = (b & 7) * 4;
            const uint8_t* src = buf + ((b >> 3) << 2);

            int acc[QUAD][OC];
            {
                const int4 c0 = *reinterpret_cast<const int4*>(colterm_s);
                const int4 c1 = *reinterpret_cast<const int4*>(colterm_s + 4);
#pragma unroll
                for (int px = 0; px < QUAD; ++px) {
                    acc[px][0] = c0.x; acc[px][1] = c0.y; acc[px][2] = c0.z; acc[px][3] = c0.w;
                    acc[px][4] = c1.x; acc[px][5] = c1.y; acc[px][6] = c1.z; acc[px][7] = c1.w;
                }
            }
#pragma unroll
            for (int kh = 0; kh < KH; ++kh) {
                const uint32_t* arow = reinterpret_cast<const uint32_t*>(src + kh * p.pitch);
                const uint32_t win = __funnelshift_r(arow[0], arow[1], shf);   // nibble i = column ow - pw + i
                const uint32_t ev = win & 0x0F0F0F0Fu, od = (win >> 4) & 0x0F0F0F0Fu;
                uint32_t a[QUAD];
                a[0] = __byte_perm(ev, od, 0x0140);    // nibbles 0 1 2
                a[1] = __byte_perm(ev, od, 0x0514);    //         1 2 3
                a[2] = __byte_perm(ev, od, 0x0251);    //         2 3 4
                a[3] = __byte_perm(ev, od, 0x0625);    //         3 4 5
                const uint4 w0 = *reinterpret_cast<const uint4*>(wsm + kh * OC);
                const uint4 w1 = *reinterpret_cast<const uint4*>(wsm + kh * OC + 4);
#pragma unroll
                for (int px = 0; px < QUAD; ++px) {
                    acc[px][0] = dp4a_u8s8(a[px], w0.x, acc[px][0]);
                    acc[px][1] = dp4a_u8s8(a[px], w0.y, acc[px][1]);
                    acc[px][2] = dp4a_u8s8(a[px], w0.z, acc[px][2]);
                    acc[px][3] = dp4a_u8s8(a[px], w0.w, acc[px][3]);
                    acc[px][4] = dp4a_u8s8(a[px], w1.x, acc[px][4]);
                    acc[px][5] = dp4a_u8s8(a[px], w1.y, acc[px][5]);
                    acc[px][6] = dp4a_u8s8(a[px], w1.z, acc[px][6]);
                    acc[px][7] = dp4a_u8s8(a[px], w1.w, acc[px][7]);
                }
            }

            uint32_t out[QUAD];
            if (PC) {
                int mlt[OC], shf_n[OC];
                {
                    const int4 m0 = *reinterpret_cast<const int4*>(pc_s), m1 = *reinterpret_cast<const int4*>(pc_s + 4);
                    const int4 s0 = *reinterpret_cast<const int4*>(pc_s + 8), s1 = *reinterpret_cast<const int4*>(pc_s + 12);
                    mlt[0] = m0.x; mlt[1] = m0.y; mlt[2] = m0.z; mlt[3] = m0.w;
                    mlt[4] = m1.x; mlt[5] = m1.y; mlt[6] = m1.z; mlt[7] = m1.w;
                    shf_n[0] = s0.x; shf_n[1] = s0.y; shf_n[2] = s0.z; shf_n[3] = s0.w;
                    shf_n[4] = s1.x; shf_n[5] = s1.y; shf_n[6] = s1.z; shf_n[7] = s1.w;
                }
#pragma unroll
                for (int px = 0; px < QUAD; ++px) {
                    uint32_t o = 0;
#pragma unroll
                    for (int n = 0; n < OC; ++n) {
                        uint32_t qv;
                        if (pc_fast) {
                            qv = clamp_above_lo(mulhi_add(acc[px][n], mlt[n], 1 << (shf_n[n] - 2)) >> (shf_n[n] - 1),
                                                zml, hml);
                        } else {
                            const RequantParams rqn{mlt[n], shf_n[n], p.rq.zo, p.rq.lo, p.rq.hi};
                            qv = requant_wide(acc[px][n], rqn) - (uint32_t)p.rq.lo;
                        }
                        o = n == 0 ? qv : mad_u32(qv, 1u << (4 * n), o);
                    }
                    out[px] = o + lofill;
                }
            } else if (p.rq.shift >= 2) {
                // the 32-bit form of the rounding shift (see requant())
#pragma unroll
                for (int px = 0; px < QUAD; ++px) {
                    uint32_t o = 0;
#pragma unroll
                    for (int n = 0; n < OC; ++n) {
                        const uint32_t qv = clamp_above_lo(mulhi_add(acc[px][n], p.rq.mult, rnd) >> s, zml, hml);
                        o = n == 0 ? qv : mad_u32(qv, 1u << (4 * n), o);   // nibble fields do not overlap
                    }
                    out[px] = o + lofill;
                }
            } else {
#pragma unroll
                for (int px = 0; px < QUAD; ++px) {
                    uint32_t o = 0;
#pragma unroll
                    for (int n = 0; n < OC; ++n) o |= requant_wide(acc[px][n], p.rq) << (4 * n);
                    out[px] = o;
                }
            }
            if (valid)
                *reinterpret_cast<uint4*>(p.Y + (uint64_t)(mbase + (uint32_t)(QUAD * r)) * (OC / 2)) =
                    make_uint4(out[0], out[1], out[2], out[3]);
        }
        release_buffer(done_bar, lane);
    }
}

}  // namespace fused

// Fills the host-derived fields of the launch parameters; returns the dynamic shared
// memory the kernel needs (0 = the layer does not fit this kernel).
static size_t plan_fused(fused::Params& p, const q4_conv_desc& d, const uint8_t* X, const uint8_t* Wt,
                         int64_t ldw, const uint8_t* Y, bool& expanded, bool& per_lane, bool& nibbles,
                         bool& quad, bool allow_lane = true)
{
    if (d.OC % 8 != 0 || d.OC < 8 || d.OC > 64) return 0;
    if (d.KH > 64 || d.KW > 64 || d.stride_h > 64 || d.stride_w > 64) return 0;
    p.H = d.H; p.W = d.W; p.C = d.C; p.KH = d.KH; p.KW = d.KW;
    p.sh = d.stride_h; p.sw = d.stride_w; p.ph = d.pad_h; p.pw = d.pad_w;
    p.OH = (d.H + 2 * d.pad_h - d.KH) / d.stride_h + 1;
    p.OW = (d.W + 2 * d.pad_w - d.KW) / d.stride_w + 1;
    p.M = (int64_t)d.N * p.OH * p.OW;
    p.K = d.KH * d.KW * d.C;
    expanded = !(d.C % 8 == 0 && (uintptr_t)X % 4 == 0);
    const int64_t segw = expanded ? ((int64_t)d.KW * d.C + 3) / 4 : 1;
    // thinnest layers: one pixel per lane, byte dot products (at most 128 per pixel); their
    // copy in shared memory stays packed when image rows are whole 32-bit words
    per_lane = expanded && (d.OC == 8 || d.OC == 16) && (int64_t)d.KH * segw * d.OC <= 128;
    nibbles = per_lane && ((int64_t)d.W * d.C) % 8 == 0 && (uintptr_t)X % 4 == 0;
    // a gray-image first layer: four pixels per lane, four times the tile
    quad = nibbles && d.C == 1 && d.OC == 8 && d.KH == 3 && d.KW == 3 && d.stride_h == 1 &&
           d.stride_w == 1 && p.OW % 4 == 0 && (uintptr_t)Y % 16 == 0;
    // per-channel parameters: the four-pixel kernel and the MMA kernel have instances for them,
    // the pixel-per-lane kernel has not
    if (!allow_lane && !quad) per_lane = nibbles = false;
    p.tile = quad ? fused::QUAD_TILE : fused::ROWS_PER_CTA;
    int64_t unit, rowbytes, data0, pix0, pitch;
    if (nibbles) {
        const int64_t halo = ((int64_t)d.pad_w * d.C + 1) / 2;     // bytes that hold a side's halo
        unit = d.C;                                                // nibbles per pixel
        rowbytes = (int64_t)d.W * d.C / 2;
        data0 = (halo + 15) / 16 * 16;
        pix0 = 2 * data0 - (int64_t)d.pad_w * d.C;
        pitch = (data0 + rowbytes + halo + 15) / 16 * 16;
    } else {
        unit = expanded ? d.C : d.C / 2;
        rowbytes = (int64_t)d.W * unit;
        data0 = (d.pad_w * unit + 15) / 16 * 16;
        pix0 = data0 - d.pad_w * unit;
        pitch = (data0 + rowbytes + d.pad_w * unit + 15) / 16 * 16;
    }
    // a tile's consecutive pixels touch at most `rows` output rows in `nseg` images
    const int64_t rows = (p.tile - 1 + p.OW - 1) / p.OW + 1;
    const int64_t nseg = (rows - 1 + p.OH - 1) / p.OH + 1;
    const int64_t slots = rows * d.stride_h + nseg * (d.KH > d.stride_h ? d.KH - d.stride_h : 0);
    const int64_t bufbytes = slots * pitch + 16;       // the slack takes the unaligned words' over-read
    const int64_t KS = expanded ? ((int64_t)d.KH * segw + 7) / 8 : ((int64_t)p.K + 31) / 32;
    const int64_t smem = per_lane
        ? (int64_t)d.KH * segw * d.OC * 4 + (int64_t)d.OC * 12 + 16 * fused::NBUF_LANE + fused::SYNC_BYTES +
              fused::NBUF_LANE * bufbytes
        : KS * (d.OC / 8) * 256 + KS * (expanded ? 8 : 4) * 4 + (int64_t)d.OC * 12 + 16 * fused::NBUF_MMA + fused::SYNC_BYTES +
              fused::NBUF_MMA * bufbytes;
    if (smem > fused::SMEM_LIMIT) return 0;
    p.unit = (int32_t)unit; p.rowbytes = (int32_t)rowbytes; p.data0 = (int32_t)data0; p.pix0 = (int32_t)pix0;
    p.pitch = (int32_t)pitch; p.bufbytes = (int32_t)bufbytes; p.segw = (int32_t)segw;
    p.KS = (int32_t)KS;
    p.sfull = (p.OH - 1) * d.stride_h + d.KH;
    p.vec16 = (!expanded || nibbles) && rowbytes % 16 == 0 && (uintptr_t)X % 16 == 0;
    p.wt_words = (uintptr_t)Wt % 4 == 0 && ldw % 4 == 0;
    p.div_ow = make_fastdiv((uint32_t)p.OW);
    p.div_oh = make_fastdiv((uint32_t)p.OH);
    p.div_sfull = make_fastdiv((uint32_t)p.sfull);
    p.cpr = (int32_t)(rowbytes / 4);
    if (p.cpr < 1) p.cpr = 1;                          // expanded mode does not use it
    p.div_cpr = make_fastdiv((uint32_t)p.cpr);
    p.step8 = (int32_t)(8 * d.stride_w * unit);
    p.rowwrap = (int32_t)(d.stride_h * pitch - (int64_t)p.OW * d.stride_w * unit);
    p.imgwrap = (int32_t)((d.KH - d.stride_h) * pitch);
    return (size_t)smem;
}

bool conv_fused_supported(const q4_conv_desc& d, const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                          const uint8_t* Y, bool per_channel)
{
    if ((uintptr_t)Y % 8) return false;
    fused::Params p;
    bool expanded, per_lane, nibbles, quad;
    return plan_fused(p, d, X, Wt, ldw, Y, expanded, per_lane, nibbles, quad, !per_channel) != 0;
}

// Launches one of the kernels above as persistent CTAs: as many as are resident at
// once, so the per-CTA set-up (weights to fragments) is paid once per SM slot and there
// is no second wave.
using FusedKernel = void (*)(const fused::Params);

static cudaError_t launch_kernel(FusedKernel kernel, const fused::Params& p, size_t smem, int64_t tiles,
                                 cudaStream_t st)
{
    // the attribute is per kernel (and per device: set on every call, it is cheap)
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         fused::SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148, per_sm = 1;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        sms = 148;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, fused::THREADS, smem) != cudaSuccess ||
        per_sm < 1)
        per_sm = 1;
    // every CTA converts the weights once: with fewer than three tiles per resident CTA,
    // launch one CTA per SM fewer (where that still leaves two)
    if (per_sm >= 3 && tiles < 3ll * sms * per_sm) --per_sm;
    const int64_t resident = (int64_t)sms * per_sm;
    const int grid = (int)(tiles < resident ? tiles : resident);
    kernel<<<grid, fused::THREADS, smem, st>>>(p);
    count_launch();
    return cudaGetLastError();
}

template <int NT, int KS>
static cudaError_t launch_ks(const fused::Params& p, size_t smem, int64_t tiles, cudaStream_t st)
{
    if (p.mult_ch) {
        if (p.OW % 4 == 0)
            return launch_kernel(fused::conv_fused_kernel<NT, false, KS, true, true>, p, smem, tiles, st);
        return launch_kernel(fused::conv_fused_kernel<NT, false, KS, false, true>, p, smem, tiles, st);
    }
    if (p.OW % 4 == 0)
        return launch_kernel(fused::conv_fused_kernel<NT, false, KS, true>, p, smem, tiles, st);
    return launch_kernel(fused::conv_fused_kernel<NT, false, KS, false>, p, smem, tiles, st);
}

template <int NT, bool EXP>
static cudaError_t launch_nt(const fused::Params& p, size_t smem, int64_t tiles, cudaStream_t st)
{
    // 3x3 layers with 8, 16 or 32 input channels (3, 5, 9 depth steps) get instances with the
    // depth loop unrolled, for the channel counts the workloads pair them with
    if constexpr (!EXP && NT <= 2) {
        if (p.KS == 3) return launch_ks<NT, 3>(p, smem, tiles, st);
    }
    if constexpr (!EXP && NT >= 2 && NT <= 4) {
        if (p.KS == 5) return launch_ks<NT, 5>(p, smem, tiles, st);
    }
    if constexpr (!EXP && NT == 8) {
        if (p.KS == 9) return launch_ks<NT, 9>(p, smem, tiles, st);
    }
    if (p.mult_ch) return launch_kernel(fused::conv_fused_kernel<NT, EXP, 0, false, true>, p, smem, tiles, st);
    return launch_kernel(fused::conv_fused_kernel<NT, EXP>, p, smem, tiles, st);
}

template <bool EXP>
static cudaError_t launch_mode(int NT, const fused::Params& p, size_t smem, int64_t tiles, cudaStream_t st)
{
    switch (NT) {
        case 1: return launch_nt<1, EXP>(p, smem, tiles, st);
        case 2: return launch_nt<2, EXP>(p, smem, tiles, st);
        case 3: return launch_nt<3, EXP>(p, smem, tiles, st);
        case 4: return launch_nt<4, EXP>(p, smem, tiles, st);
        case 5: return launch_nt<5, EXP>(p, smem, tiles, st);
        case 6: return launch_nt<6, EXP>(p, smem, tiles, st);
        case 7: return launch_nt<7, EXP>(p, smem, tiles, st);
        default: return launch_nt<8, EXP>(p, smem, tiles, st);
    }
}

cudaError_t launch_conv_fused(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                              const int32_t* colsum_w, const int32_t* bias, const q4_conv_desc& d,
                              int32_t za, int32_t zb, const RequantParams& rq, uint8_t* Y,
                              cudaStream_t st, const int32_t* zb_ch, const int32_t* mult_ch,
                              const int32_t* shift_ch)
{
    fused::Params p;
    bool expanded = false, per_lane = false, nibbles = false, quad = false;
    // layers with per-channel parameters always take the MMA kernel
    const size_t smem = plan_fused(p, d, X, Wt, ldw, Y, expanded, per_lane, nibbles, quad, mult_ch == nullptr);
    p.zb_ch = zb_ch; p.mult_ch = mult_ch; p.shift_ch = shift_ch;
    if (smem == 0) return cudaErrorInvalidValue;
    p.X = X; p.Wt = Wt; p.ldw = ldw; p.colsum_w = colsum_w; p.bias = bias; p.Y = Y;
    p.za = za; p.zb = zb; p.rq = rq;
    p.status = device_status_ptr();
    if (!p.status) return cudaErrorUnknown;
    if (p.M == 0) return cudaSuccess;
    const int64_t tiles = (p.M + p.tile - 1) / p.tile;
    log_choice(mult_ch ? "q4_conv2d_channels" : "q4_conv2d",
               quad ? "fused, four pixels per lane" : per_lane ? "fused, one pixel per lane"
                    : expanded ? "fused implicit GEMM (MMA), expanded copy" : "fused implicit GEMM (MMA), packed copy");
    if (quad)
        return mult_ch ? launch_kernel(fused::conv_quad_kernel<true>, p, smem, tiles, st)
                       : launch_kernel(fused::conv_quad_kernel<false>, p, smem, tiles, st);
    if (per_lane) {
        // the 3x3 single-channel first layer gets its own fully unrolled instance
        if (nibbles && d.OC == 8 && d.KH == 3 && p.segw == 1)
            return launch_kernel(fused::conv_lane_kernel<8, true, 3, 1>, p, smem, tiles, st);
        if (nibbles)
            return d.OC == 8 ? launch_kernel(fused::conv_lane_kernel<8, true, 0, 0>, p, smem, tiles, st)
                             : launch_kernel(fused::conv_lane_kernel<16, true, 0, 0>, p, smem, tiles, st);
        // a 5x5 single-channel first layer whose rows are not whole words (25-pixel rows)
        if (d.OC == 8 && d.KH == 5 && p.segw == 2)
            return launch_kernel(fused::conv_lane_kernel<8, false, 5, 2>, p, smem, tiles, st);
        return d.OC == 8 ? launch_kernel(fused::conv_lane_kernel<8, false, 0, 0>, p, smem, tiles, st)
                         : launch_kernel(fused::conv_lane_kernel<16, false, 0, 0>, p, smem, tiles, st);
    }
    return expanded ? launch_mode<true>(d.OC / 8, p, smem, tiles, st)
                    : launch_mode<false>(d.OC / 8, p, smem, tiles, st);
}

}  // namespace q4
