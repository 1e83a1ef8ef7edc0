// Re-quantization of eight accumulators at a time (Eq. 3 followed by the clamp and the
// packing to 4 bits), shared by the convolution kernels and the GEMM epilogues.
#pragma once

#include "q4_common.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {

// (a * b >> 32) + c in one instruction.
__device__ __forceinline__ int mulhi_add(int a, int b, int c)
{
    int d;
    asm("mad.hi.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// a * b + c in one instruction (the compiler otherwise splits a shift-and-or into two).
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// Saturating pack of two 32-bit integers into the signed 16-bit halves of one register.
__device__ __forceinline__ uint32_t pack_sat16(int hi, int lo)
{
    uint32_t d;
    asm("cvt.pack.sat.s16.s32 %0, %1, %2;" : "=r"(d) : "r"(hi), "r"(lo));
    return d;
}

// Position c of a group of eight accumulator columns holds output channel ch8(c) of the
// group: a register pair (columns 2i, 2i+1) then holds channels i and i+4, which lets the
// epilogue clamp two values per instruction in 16-bit halves and gather the four pairs
// into one word of eight nibbles with three multiply-adds.
__host__ __device__ constexpr int ch8(int c) { return (c >> 1) + 4 * (c & 1); }

// Eight accumulators (columns in the ch8 order) -> the eight re-quantized nibbles of one
// 32-bit word, channel k in nibble k.  Fast form (shift >= 2, see requant(); and shift <= 27
// so that the output zero point can ride in the rounding constant): the caller passes
// rnd = 2^(s-1) + ((zo - lo) << s), so (mulhi + rnd) >> s is already q + zo - lo; two such
// values are packed with saturation into 16-bit halves and clamped to [0, hi - lo] by one
// instruction.  The result holds value - lo per nibble; the caller adds lo to all nibbles.
template <bool FAST>
__device__ __forceinline__ uint32_t requant8(const uint32_t* r, const RequantParams& rq, int s, int rnd,
                                             uint32_t hml2)
{
    if (FAST) {
        uint32_t c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int q0 = mulhi_add((int)r[2 * i], rq.mult, rnd) >> s;
            const int q1 = mulhi_add((int)r[2 * i + 1], rq.mult, rnd) >> s;
            c[i] = __vimin_s16x2_relu(pack_sat16(q1, q0), hml2);
        }
        // c[i] = channel i | channel (i + 4) << 16, each 0..15
        return mad_u32(c[3], 1u << 12, mad_u32(c[2], 1u << 8, mad_u32(c[1], 1u << 4, c[0])));
    }
    uint32_t o = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e)
        o |= (requant_wide((int)r[e], rq) - (uint32_t)rq.lo) << (4 * ch8(e));
    return o;
}

// The same with every column's own multiplier, rounding constant and shift (per output
// channel), read from shared memory at pc_s + 4 * (array * n_cols + column): columns
// col0 .. col0 + 7.  fast: every shift allows the 32-bit form (the arrays then hold
// rnd = 2^(s-1) + ((zo - lo) << s) and s = shift - 1), else they hold the shifts themselves.
// NATURAL: the eight accumulators (and their parameters) are channels 0..7 in order -- the
// halves of a packed pair may be any two registers, so channels i and i + 4 are paired directly;
// otherwise they come in the ch8 order of the convolution kernels' B operand.
template <bool NATURAL = false>
__device__ __forceinline__ uint32_t requant8_channels(const uint32_t* r, const RequantParams& rq, uint32_t pc_s,
                                                      int n_cols, int col0, bool fast, uint32_t hml2)
{
    const uint4 m0 = lds128(pc_s + 4 * col0), m1 = lds128(pc_s + 4 * (col0 + 4));
    const uint4 s0 = lds128(pc_s + 4 * (2 * n_cols + col0)), s1 = lds128(pc_s + 4 * (2 * n_cols + col0 + 4));
    const int mu[8] = {(int)m0.x, (int)m0.y, (int)m0.z, (int)m0.w, (int)m1.x, (int)m1.y, (int)m1.z, (int)m1.w};
    const int sh[8] = {(int)s0.x, (int)s0.y, (int)s0.z, (int)s0.w, (int)s1.x, (int)s1.y, (int)s1.z, (int)s1.w};
    if (fast) {
        const uint4 r0 = lds128(pc_s + 4 * (n_cols + col0)), r1 = lds128(pc_s + 4 * (n_cols + col0 + 4));
        const int rn[8] = {(int)r0.x, (int)r0.y, (int)r0.z, (int)r0.w, (int)r1.x, (int)r1.y, (int)r1.z, (int)r1.w};
        uint32_t c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int a = NATURAL ? i : 2 * i, b = NATURAL ? i + 4 : 2 * i + 1;     // channels i and i + 4
            const int q0 = mulhi_add((int)r[a], mu[a], rn[a]) >> sh[a];
            const int q1 = mulhi_add((int)r[b], mu[b], rn[b]) >> sh[b];
            c[i] = __vimin_s16x2_relu(pack_sat16(q1, q0), hml2);
        }
        return mad_u32(c[3], 1u << 12, mad_u32(c[2], 1u << 8, mad_u32(c[1], 1u << 4, c[0])));
    }
    uint32_t o = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const RequantParams one{mu[e], sh[e], rq.zo, rq.lo, rq.hi};
        o |= (requant_wide((int)r[e], one) - (uint32_t)rq.lo) << (4 * (NATURAL ? e : ch8(e)));
    }
    return o;
}

}  // namespace q4
