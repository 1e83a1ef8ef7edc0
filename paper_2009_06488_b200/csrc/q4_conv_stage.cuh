// Shared pieces of the fused convolution kernels: the launch parameters, the geometry of a
// tile's copy in shared memory (which input rows a run of consecutive output pixels
// touches), and the producer warp that keeps a ring of such copies filled -- with the
// padding materialised as the input zero point, so that consumers gather without bounds
// checks -- plus small integer helpers of the re-quantizing epilogues.
#pragma once

#include "q4_common.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {
namespace fused {

struct Params {
    const uint8_t* X;
    const uint8_t* Wt;
    int64_t ldw;
    const int32_t* colsum_w;   // optional
    const int32_t* bias;       // optional
    // per output channel (all three or none): weight zero points, multipliers, shifts
    const int32_t* zb_ch;
    const int32_t* mult_ch;
    const int32_t* shift_ch;
    uint8_t* Y;
    // the tensor-memory kernels' weight image (the B operand, the per-column constants, a flag):
    // prep_out = build it and write it there, do nothing else; prep_in = take it from there
    const uint8_t* prep_in;
    uint8_t* prep_out;
    uint32_t prep_tag;         // what the image is for (layer class, filter, channels, za, build): written / checked
    int64_t M;
    int32_t H, W, C, KH, KW, OH, OW, sh, sw, ph, pw;
    int32_t K, KS;             // depth, number of 32-byte MMA depth steps
    int32_t za, zb;
    RequantParams rq;
    // staging geometry (host-derived)
    int32_t unit;              // bytes per input pixel in shared memory (C/2 packed, C expanded)
    int32_t rowbytes;          // W * unit: bytes of one image row in shared memory
    int32_t data0;             // byte offset of input column 0 in a staged row (multiple of 16)
    int32_t pix0;              // offset of input column -pw in a staged row, in bytes (nibbles in
                               // the per-lane kernel's packed mode)
    int32_t pitch;             // bytes per staged row (multiple of 16)
    int32_t bufbytes;          // one input buffer
    int32_t segw;              // expanded: 32-bit words per kh segment
    int32_t sfull;             // staged rows of an image all of whose output rows are in the tile
    int32_t vec16;             // packed: image rows are whole 16-byte pieces, 16-byte aligned: each
                               // is copied by one bulk copy that reports to the buffer's mbarrier
    unsigned* status;          // device status word (a wait that ran out is recorded there)
    int32_t wt_words;          // weights can be read as aligned 32-bit words
    int32_t cpr;               // packed: copy pieces (16 or 4 bytes) per image row (the tensor-memory
                               // kernel: bytes per asynchronous copy, 8 or 4)
    int32_t tile;              // output pixels per CTA tile
    int32_t nbuf;              // input buffers of the ring where the kernel takes it at run time
    // the tensor-memory kernel for wide layers: output channels per CTA, CTAs that share the
    // channels of one pixel tile, all output channels
    int32_t tcN, tcSplit, OCtot;
    int32_t step8;             // staged-buffer offset of the pixel eight further in the same output row
    int32_t rowwrap;           // ... added when that pixel is in the next output row
    int32_t imgwrap;           // ... added on top when that row is the next image's first
    FastDiv div_ow, div_oh, div_sfull, div_cpr;
};

__device__ __forceinline__ void cp_async4(void* dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;"
                 :: "r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;" ::: "memory");
}
// Waits until at most PENDING of this thread's most recent copy groups are still in flight.
template <int PENDING>
__device__ __forceinline__ void cp_async_wait_group()
{
    asm volatile("cp.async.wait_group %0;" :: "n"(PENDING) : "memory");
}

// Four nibbles in the low halves of four bytes, minus zb, as four signed bytes.  Setting
// bit 7 of every byte first keeps the subtraction from borrowing across bytes
// (128 + x - zb > 0); flipping it back leaves x - zb in two's complement.
__device__ __forceinline__ uint32_t sub_zb(uint32_t x, uint32_t zb)
{
    return ((x | 0x80808080u) - zb * 0x01010101u) ^ 0x80808080u;
}

__device__ __forceinline__ int mulhi_add(int a, int b, int c)
{
    int d;
    asm("mad.hi.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// clamp(q + zo, lo, hi) - lo = max(min(q + (zo - lo), hi - lo), 0): one instruction (add, min
// and the lower clamp at zero fused).  The kernels keep this value per nibble and add lo to
// all nibbles of a packed word at once (no carries: value + lo <= hi <= 15).
__device__ __forceinline__ uint32_t clamp_above_lo(int q, int zo_minus_lo, int hi_minus_lo)
{
    return (uint32_t)__viaddmin_s32_relu(q, zo_minus_lo, hi_minus_lo);
}

// a * b + c in one instruction (the compiler otherwise splits a shift-and-or into two).
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ uint32_t weight_nibble(const Params& p, int n, int k)
{
    const uint8_t byte = p.Wt[(int64_t)n * p.ldw + (k >> 1)];
    return (k & 1) ? (uint32_t)(byte >> 4) : (uint32_t)(byte & 0x0F);
}

// Which input rows a tile's copy in shared memory holds.  The tile's output rows
// (index q = n * OH + oh) run from q_first to q_last; the images they belong to are
// "segments".  A segment's staged rows are the input rows from its first output row's
// first tap row to its last output row's last tap row.
struct Geo {
    int32_t n_first, oh_first;   // image and output row of the tile's first pixel
    int32_t s0;                  // staged rows of the first segment
    int32_t nslots;              // staged rows in all
};

__device__ __forceinline__ Geo tile_geometry(const Params& p, int64_t tile)
{
    const int64_t mb = tile * p.tile;
    const int64_t me = (mb + p.tile < p.M ? mb + p.tile : p.M) - 1;
    const uint32_t q_first = fdiv((uint32_t)mb, p.div_ow), q_last = fdiv((uint32_t)me, p.div_ow);
    const uint32_t n_first = fdiv(q_first, p.div_oh), n_last = fdiv(q_last, p.div_oh);
    const int oh_first = (int)(q_first - n_first * (uint32_t)p.OH);
    const int oh_last = (int)(q_last - n_last * (uint32_t)p.OH);
    Geo g;
    g.n_first = (int)n_first;
    g.oh_first = oh_first;
    if (n_first == n_last) {
        g.s0 = (oh_last - oh_first) * p.sh + p.KH;
        g.nslots = g.s0;
    } else {
        g.s0 = (p.OH - 1 - oh_first) * p.sh + p.KH;
        g.nslots = g.s0 + (int)(n_last - n_first - 1) * p.sfull + oh_last * p.sh + p.KH;
    }
    return g;
}

__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Which image row staged row `s` of a tile holds: returns the row index n * H + ih, or
// -1 for a row above or below the image.
__device__ __forceinline__ int64_t staged_row(const Params& p, const Geo& g, int s)
{
    int seg = 0, ih = g.oh_first * p.sh - p.ph + s;
    if (s >= g.s0) {
        const uint32_t r = (uint32_t)(s - g.s0);
        const uint32_t sq = fdiv(r, p.div_sfull);
        seg = 1 + (int)sq;
        ih = (int)(r - sq * (uint32_t)p.sfull) - p.ph;
    }
    if ((unsigned)ih >= (unsigned)p.H) return -1;
    return (int64_t)(g.n_first + seg) * p.H + ih;
}

// Producer warp, packed mode, rows of whole 16-byte pieces: one bulk copy per staged
// row, a lane per row; the copies report their bytes to `bar`, which lane 0 has armed
// with the tile's total.  Only the image columns are written: the halo columns hold the
// zero point from the kernel's start.  Rows above or below the image are filled with
// the zero point by ordinary stores.
__device__ __forceinline__ void stage_packed_bulk(const Params& p, const Geo& g, uint8_t* buf, uint32_t bar,
                                                  int lane)
{
    // ordinary stores to this buffer (the initial fill, earlier border rows) come before
    // the copy engine's writes
    fence_async_smem();
    const uint32_t zfill = (uint32_t)p.za * 0x11111111u;
    int inside = 0;
    for (int s = lane; s < g.nslots; s += 32) {
        if (staged_row(p, g, s) >= 0) {
            ++inside;
        } else {
            uint8_t* dst = buf + s * p.pitch + p.data0;
            for (int c = 0; c < p.rowbytes; c += 16)
                *reinterpret_cast<uint4*>(dst + c) = make_uint4(zfill, zfill, zfill, zfill);
        }
    }
    inside = __reduce_add_sync(0xFFFFFFFFu, inside);   // also orders the fills before lane 0's arrive
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)inside * (uint32_t)p.rowbytes);
    __syncwarp();
    for (int s = lane; s < g.nslots; s += 32) {
        const int64_t row = staged_row(p, g, s);
        if (row >= 0)
            bulk_load_row(smem_u32(buf + s * p.pitch + p.data0), p.X + row * p.rowbytes,
                          (uint32_t)p.rowbytes, bar);
    }
}

// Producer warp, packed mode, any 4-byte-aligned rows: asynchronous 4-byte copies, one
// piece per lane and step.
__device__ __forceinline__ void stage_packed(const Params& p, const Geo& g, uint8_t* buf, int lane)
{
    const int total = g.nslots * p.cpr;
    const uint32_t zfill = (uint32_t)p.za * 0x11111111u;
    for (int idx = lane; idx < total; idx += 32) {
        const int s = (int)fdiv((uint32_t)idx, p.div_cpr);
        const int c = (idx - s * p.cpr) * 4;
        const int64_t row = staged_row(p, g, s);
        uint8_t* dst = buf + s * p.pitch + p.data0 + c;
        if (row >= 0) cp_async4(dst, p.X + row * p.rowbytes + c);
        else *reinterpret_cast<uint32_t*>(dst) = zfill;
    }
}

// Producer warp, expanded mode: one byte per value.  A lane takes one packed byte of
// a row (two values); the loads of eight staged rows are issued before any of them is
// used, so a tile costs one or two memory round trips.
__device__ __forceinline__ void stage_expanded(const Params& p, const Geo& g, uint8_t* buf, int lane)
{
    constexpr int BATCH = 8;
    const int data0 = p.data0;
    const int wc = p.rowbytes;                         // values per image row
    const int ih_first = g.oh_first * p.sh - p.ph;
    for (int sb = 0; sb < g.nslots; sb += BATCH) {
        for (int jb = 0; jb < (wc + 2) / 2; jb += 32) {
            const int j = jb + lane;                   // my packed byte of each row
            uint32_t raw[BATCH];
            int v0[BATCH];                             // row position of my low nibble; INT_MIN/2 = no row
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int s = sb + u;
                raw[u] = (uint32_t)p.za * 0x11u;
                v0[u] = -(1 << 30);
                if (s < g.nslots) {
                    int seg = 0, ih = ih_first + s;
                    if (s >= g.s0) {
                        const uint32_t r = (uint32_t)(s - g.s0);
                        const uint32_t sq = fdiv(r, p.div_sfull);
                        seg = 1 + (int)sq;
                        ih = (int)(r - sq * (uint32_t)p.sfull) - p.ph;
                    }
                    v0[u] = 2 * j;
                    if ((unsigned)ih < (unsigned)p.H) {
                        const int64_t e0 = ((int64_t)(g.n_first + seg) * p.H + ih) * wc;
                        v0[u] = 2 * j - (int)(e0 & 1);
                        if (v0[u] < wc) raw[u] = p.X[(e0 >> 1) + j];
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                uint8_t* dst = buf + (sb + u) * p.pitch + data0;
                if (v0[u] >= 0 && v0[u] < wc) dst[v0[u]] = (uint8_t)(raw[u] & 0x0Fu);
                if (v0[u] + 1 >= 0 && v0[u] + 1 < wc) dst[v0[u] + 1] = (uint8_t)(raw[u] >> 4);
            }
        }
    }
}

// The producer warp's loop.  Tile j lives in buffer j % NB.  A buffer is refilled once every
// multiplying warp has reported (on its "read" mbarrier) that it is done with the tile that
// was there; a tile is announced on the buffer's "landed" mbarrier -- by the bulk copies
// themselves, or by lane 0 once this warp's copies of that tile have landed, which is
// checked NB - 2 tiles later so that copies stay in flight.  The tile's geometry is
// written before the arrive that publishes it.
template <int NB, bool EXPANDED>
__device__ __forceinline__ void producer_loop(const Params& p, int mytiles, uint8_t* buf0, int4* geo_s,
                                              uint32_t full0, uint32_t empty0, uint32_t abort_flag, int lane)
{
    constexpr int LOOK = NB - 2;
    const bool bulk = !EXPANDED && p.vec16;
    int b = 0;                                         // j % NB
    uint32_t round = 0;                                // j / NB
    for (int j = 0; j < mytiles + LOOK; ++j) {
        if (j < mytiles) {
            if (round > 0) mbar_wait_suspend(empty0 + 8 * b, (round - 1) & 1, abort_flag, p.status);
            const Geo gn = tile_geometry(p, blockIdx.x + (int64_t)j * gridDim.x);
            if (lane == 0) geo_s[b] = make_int4(gn.n_first, gn.oh_first, gn.s0, gn.nslots);
            uint8_t* buf = buf0 + b * p.bufbytes;
            if (EXPANDED) stage_expanded(p, gn, buf, lane);
            else if (bulk) stage_packed_bulk(p, gn, buf, full0 + 8 * b, lane);
            else stage_packed(p, gn, buf, lane);
            if (++b == NB) { b = 0; ++round; }
        }
        cp_async_commit();                             // one group per tile, empty past the end
        if (!bulk) {
            cp_async_wait_group<LOOK>();
            __syncwarp();
            const int d = j - LOOK;                    // this tile's copies have landed
            if (lane == 0 && d >= 0) mbar_arrive(full0 + 8 * (d % NB));
        }
    }
}


}  // namespace fused
}  // namespace q4
