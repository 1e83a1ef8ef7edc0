// Fused quantized convolution layer: the unrolled activation matrix of GEMM-based
// convolution (Section I; depth D = kh*kw*c, Section III-A) is never written to
// memory.  Each warp gathers its 32 output pixels' taps straight from the packed NHWC
// input, expands the nibbles in registers into the A fragments of the warp-level
// integer MMA (u8 x u8 -> s32, m16n8k32), multiplies against the layer's weights held
// as B fragments in shared memory, and applies Eq. 3's zero-point terms, the bias, the
// re-quantization and the nibble packing to the accumulators it holds.  The row sums of
// Eq. 2's second term are taken from the same registers "while unrolling" (Section
// II-B).
//
// Why not the tcgen05 path here: these layers have tiny depth and few output channels
// (K = 72..288, N = 8..64), so the work per output tile is a few hundred clocks of
// tensor time -- far less than the hand-offs of a TMA / tensor-memory pipeline -- and
// the traffic saved by not materialising the unrolled matrix (2 * M * K/2 bytes) is
// what matters.  The register-fragment MMA needs no staging at all: a packed 32-bit
// word of a row is exactly the two A registers of one thread (even nibbles, odd
// nibbles), the same depth permutation being applied to the weights.
//
// Requirements (else the caller falls back to unroll + GEMM): C % 8 == 0 (a 32-bit
// packed word never straddles two taps), OC in {8, 16, 32, 64}, X and Y 16-byte
// aligned.
#include "q4_common.cuh"

namespace q4 {
namespace fused {

constexpr int WARPS = 8;
constexpr int ROWS_PER_WARP = 32;
constexpr int ROWS_PER_CTA = WARPS * ROWS_PER_WARP;

struct Params {
    const uint8_t* X;
    const uint8_t* Wt;
    int64_t ldw;
    const int32_t* colsum_w;   // optional
    const int32_t* bias;       // optional
    uint8_t* Y;
    int64_t M;
    int32_t H, W, C, KH, KW, OH, OW, sh, sw, ph, pw;
    int32_t K, KS;             // depth, number of 32-value depth steps
    int32_t za, zb;
    RequantParams rq;
};

__device__ __forceinline__ void mma_u8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                       uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
        "{%8, %9}, {%0, %1, %2, %3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// NT = OC / 8 output-channel tiles.  Fragment column f of tile nt is output channel
// 2 * (NT * (f / 2) + nt) + f % 2, so that the NT packed output bytes a thread ends up
// with are contiguous in memory.
#ifndef Q4_FUSED_MIN_CTAS
#define Q4_FUSED_MIN_CTAS 2
#endif
template <int NT>
__global__ void __launch_bounds__(WARPS * 32, Q4_FUSED_MIN_CTAS)
conv_fused_kernel(const Params p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    uint2* bfrag = reinterpret_cast<uint2*>(smem);                       // [KS][NT][32]
    int32_t* tab = reinterpret_cast<int32_t*>(smem + (size_t)p.KS * NT * 32 * 8);   // [KS][4] x 2
    int32_t* colsum_s = tab + p.KS * 4 * 2;                               // [8 * NT]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int tapb = p.C / 2;                  // bytes per tap
    const int kbytes = p.K / 2;
    constexpr int N = 8 * NT;

    // ---- once per CTA: weights -> B fragments, tap table, weight sums
    for (int i = tid; i < N; i += blockDim.x) colsum_s[i] = 0;
    __syncthreads();
    for (int i = tid; i < p.KS * NT * 32; i += blockDim.x) {
        const int l = i & 31, nt = (i >> 5) % NT, j = (i >> 5) / NT;
        const int fg = l >> 2, ft = l & 3;
        const int n = 2 * (NT * (fg >> 1) + nt) + (fg & 1);
        const int kb = 16 * j + 4 * ft;
        uint32_t w = 0;
        if (kb < kbytes) w = *reinterpret_cast<const uint32_t*>(p.Wt + (int64_t)n * p.ldw + kb);
        bfrag[i] = make_uint2(w & 0x0F0F0F0Fu, (w >> 4) & 0x0F0F0F0Fu);
        if (!p.colsum_w && w) atomicAdd(&colsum_s[n], nibble_sum(w));
    }
    for (int i = tid; i < p.KS * 4; i += blockDim.x) {
        const int kb = 16 * (i >> 2) + 4 * (i & 3);
        int delta = -1, khkw = 0;
        if (kb < kbytes) {
            const int tap = kb / tapb, off = kb % tapb;
            const int kh = tap / p.KW, kw = tap % p.KW;
            delta = (kh * p.W + kw) * tapb + off;
            khkw = (kh << 16) | kw;
        }
        tab[2 * i] = delta;
        tab[2 * i + 1] = khkw;
    }
    __syncthreads();

    // per-thread epilogue constants: the column term of Eq. 3 for my NT channel pairs
    int colterm[NT][2];
    const int kzz = p.K * p.za * p.zb;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int n = 2 * (NT * t + nt) + e;
            const int cs = p.colsum_w ? p.colsum_w[n] : colsum_s[n];
            colterm[nt][e] = (int)((uint32_t)kzz - (uint32_t)(p.za * cs) +
                                   (uint32_t)(p.bias ? p.bias[n] : 0));
        }
    const uint32_t zfill = (uint32_t)p.za * 0x11111111u;

    const int64_t ntiles = (p.M + ROWS_PER_CTA - 1) / ROWS_PER_CTA;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t m0 = tile * ROWS_PER_CTA + warp * ROWS_PER_WARP;
        if (m0 >= p.M) continue;                       // warp-uniform
        // my four rows: g, g+8 (first 16-row tile), 16+g, 24+g (second)
        int ih0[4], iw0[4];
        const uint8_t* base[4];
        bool valid[4];
        {
            // one division for my first row; the others are 8 pixels further each
            const int64_t mf = m0 + g;
            const uint32_t mm = mf < p.M ? (uint32_t)mf : 0u;       // M < 2^31
            int ow = (int)(mm % (uint32_t)p.OW);
            const uint32_t q = mm / (uint32_t)p.OW;
            int oh = (int)(q % (uint32_t)p.OH);
            int64_t n = q / (uint32_t)p.OH;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                valid[i] = mf + 8 * i < p.M;
                ih0[i] = oh * p.sh - p.ph;
                iw0[i] = ow * p.sw - p.pw;
                base[i] = p.X + ((n * p.H + ih0[i]) * p.W + iw0[i]) * tapb;
                ow += 8;
                while (ow >= p.OW) {
                    ow -= p.OW;
                    if (++oh == p.OH) { oh = 0; ++n; }
                }
            }
        }
        int acc[2][NT][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0;
        int rsum[4] = {0, 0, 0, 0};

        // gather of one depth step: my packed word of each of my four rows (the zero
        // point outside the image, zero past the depth)
        auto gather = [&](int j, uint32_t (&w)[4]) {
            const int delta = tab[2 * (4 * j + t)];
            const int khkw = tab[2 * (4 * j + t) + 1];
            const int kh = khkw >> 16, kw = khkw & 0xFFFF;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                w[i] = 0;
                if (delta >= 0) {
                    const int ih = ih0[i] + kh, iw = iw0[i] + kw;
                    w[i] = zfill;
                    if (valid[i] && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W)
                        w[i] = __ldg(reinterpret_cast<const uint32_t*>(base[i] + delta));
                }
            }
        };
        uint32_t wcur[4], wnext[4];
        gather(0, wcur);
        for (int j = 0; j < p.KS; ++j) {
            if (j + 1 < p.KS) gather(j + 1, wnext);      // in flight while this step multiplies
            uint32_t lo[4], hi[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                lo[i] = wcur[i] & 0x0F0F0F0Fu;
                hi[i] = (wcur[i] >> 4) & 0x0F0F0F0Fu;
                rsum[i] = dp4a_u8(lo[i] + hi[i], 0x01010101u, rsum[i]);
            }
            const uint2* bj = bfrag + (size_t)j * NT * 32 + lane;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const uint2 b = bj[nt * 32];
                mma_u8(acc[0][nt], lo[0], lo[1], hi[0], hi[1], b.x, b.y);
                mma_u8(acc[1][nt], lo[2], lo[3], hi[2], hi[3], b.x, b.y);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) wcur[i] = wnext[i];
        }

        // row sums: add the four depth slices held by the lanes of a row
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            rsum[i] += __shfl_xor_sync(0xFFFFFFFFu, rsum[i], 1);
            rsum[i] += __shfl_xor_sync(0xFFFFFFFFu, rsum[i], 2);
        }
        // epilogue: accumulator (mt, nt) holds rows g + 16 mt (c0, c1) and g + 8 + 16 mt
        // (c2, c3), fragment columns 2t, 2t+1
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int mt = i >> 1, hrow = i & 1;
            const int64_t m = m0 + g + 8 * i;
            if (m >= p.M) continue;
            const uint32_t rowterm = (uint32_t)0 - (uint32_t)(p.zb * rsum[i]);
            uint32_t bytes[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int v0 = (int)((uint32_t)acc[mt][nt][2 * hrow] + rowterm + (uint32_t)colterm[nt][0]);
                const int v1 = (int)((uint32_t)acc[mt][nt][2 * hrow + 1] + rowterm + (uint32_t)colterm[nt][1]);
                bytes[nt] = requant(v0, p.rq) | (requant(v1, p.rq) << 4);
            }
            uint8_t* dst = p.Y + m * (N / 2) + NT * t;
            if (NT == 8) {
                const uint32_t w0 = bytes[0] | (bytes[1] << 8) | (bytes[2] << 16) | (bytes[3] << 24);
                const uint32_t w1 = bytes[4 % NT] | (bytes[5 % NT] << 8) | (bytes[6 % NT] << 16) | (bytes[7 % NT] << 24);
                *reinterpret_cast<uint2*>(dst) = make_uint2(w0, w1);
            } else if (NT == 4) {
                *reinterpret_cast<uint32_t*>(dst) =
                    bytes[0] | (bytes[1 % NT] << 8) | (bytes[2 % NT] << 16) | (bytes[3 % NT] << 24);
            } else if (NT == 2) {
                *reinterpret_cast<uint16_t*>(dst) = (uint16_t)(bytes[0] | (bytes[1 % NT] << 8));
            } else {
                *dst = (uint8_t)bytes[0];
            }
        }
    }
}

}  // namespace fused

bool conv_fused_supported(const q4_conv_desc& d, const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                          const uint8_t* Y)
{
    if (d.C % 8 != 0) return false;
    if (d.OC != 8 && d.OC != 16 && d.OC != 32 && d.OC != 64) return false;
    if ((uintptr_t)X % 16 || (uintptr_t)Y % 16 || (uintptr_t)Wt % 4 || ldw % 4) return false;
    const int K = d.KH * d.KW * d.C;
    const int KS = (K + 31) / 32;
    const size_t smem = (size_t)KS * (d.OC / 8) * 32 * 8 + (size_t)KS * 4 * 8 + (size_t)d.OC * 4;
    return smem <= 96 * 1024 && d.KH < 256 && d.KW < 256;
}

template <int NT>
static cudaError_t launch_nt(const fused::Params& p, size_t smem, int64_t tiles, cudaStream_t st)
{
    static bool attr = false;
    static int sms = 148;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(fused::conv_fused_kernel<NT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        if (e != cudaSuccess) return e;
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        attr = true;
    }
    // persistent CTAs: as many as are resident at once, so the per-CTA set-up (weights to
    // fragments) is paid once per SM slot and there is no second wave
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused::conv_fused_kernel<NT>,
                                                      fused::WARPS * 32, smem) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    const int64_t resident = (int64_t)sms * per_sm;
    const int grid = (int)(tiles < resident ? tiles : resident);
    fused::conv_fused_kernel<NT><<<grid, fused::WARPS * 32, smem, st>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_conv_fused(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                              const int32_t* colsum_w, const int32_t* bias, const q4_conv_desc& d,
                              int32_t za, int32_t zb, const RequantParams& rq, uint8_t* Y,
                              cudaStream_t st)
{
    fused::Params p;
    p.X = X; p.Wt = Wt; p.ldw = ldw; p.colsum_w = colsum_w; p.bias = bias; p.Y = Y;
    p.H = d.H; p.W = d.W; p.C = d.C; p.KH = d.KH; p.KW = d.KW;
    p.sh = d.stride_h; p.sw = d.stride_w; p.ph = d.pad_h; p.pw = d.pad_w;
    p.OH = (d.H + 2 * d.pad_h - d.KH) / d.stride_h + 1;
    p.OW = (d.W + 2 * d.pad_w - d.KW) / d.stride_w + 1;
    p.M = (int64_t)d.N * p.OH * p.OW;
    p.K = d.KH * d.KW * d.C;
    p.KS = (p.K + 31) / 32;
    p.za = za; p.zb = zb; p.rq = rq;
    if (p.M == 0) return cudaSuccess;
    const int NT = d.OC / 8;
    const size_t smem = (size_t)p.KS * NT * 32 * 8 + (size_t)p.KS * 4 * 8 + (size_t)d.OC * 4;
    const int64_t tiles = (p.M + fused::ROWS_PER_CTA - 1) / fused::ROWS_PER_CTA;
    switch (NT) {
        case 1: return launch_nt<1>(p, smem, tiles, st);
        case 2: return launch_nt<2>(p, smem, tiles, st);
        case 4: return launch_nt<4>(p, smem, tiles, st);
        default: return launch_nt<8>(p, smem, tiles, st);
    }
}

}  // namespace q4
