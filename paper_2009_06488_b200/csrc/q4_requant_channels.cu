// Per-output-channel weight quantization (an extension of the paper's per-matrix scheme of
// Section II-A / III-B: every output channel n has its own weight zero point zb[n] and its
// own re-quantization multiplier).  Eq. 2 holds column by column, and the zero point of a
// column enters only through a rank-one term:
//   sum_k (a - za)(b - zb[n]) = [sum_k (a - za) b]  -  zb[n] * (sum_k a - K za),
// so the product is taken once with zb = 0 by q4_gemm and this kernel finishes it:
//   acc = C0[m][n] - zb[n] * (rowsum_a[m] - K za) + bias[n]
//   y   = clamp(floor((acc * mult[n] + 2^(30 + shift[n])) / 2^(31 + shift[n])) + zo, lo, hi)
// packed two per byte.  One pass over the int32 matrix: bound by HBM (4 bytes read and half
// a byte written per value).
#include "q4_common.cuh"
#include "q4_requant8.cuh"

namespace q4 {

struct ChannelParams {
    const int32_t* C0;
    int64_t ldc;
    int32_t M, N, K, za;
    const int32_t* rowsum_a;
    const int32_t* zb;       // optional
    const int32_t* bias;     // optional
    const int32_t* mult;
    const int32_t* shift;
    int32_t zo, lo, hi;
    uint8_t* Cq;
    int64_t ldcq;
};

__device__ __forceinline__ uint32_t requant_one(int32_t acc, int32_t mult, int32_t shift, int zo, int lo, int hi)
{
    const int t = 31 + shift;
    const long long v = (long long)acc * (long long)mult + (1ll << (t - 1));
    int q = (int)(v >> t) + zo;
    return (uint32_t)min(max(q, lo), hi);
}

// Four consecutive channels and two rows per thread.  A thread keeps its channels' parameters
// in registers (40 registers in all: 1536 threads are resident per SM, each with two 16-byte
// loads in flight; eight channels per thread took 64 registers and reached 0.69 of the copy
// bandwidth where this form reaches 0.80) and walks the row pairs blockIdx.y,
// blockIdx.y + gridDim.y, ...  The two rows' values of a channel share a packed pair, so the
// gathered word holds row r's four nibbles in its low half and row r + 1's in its high half.
__global__ void __launch_bounds__(256, 6)
requant_channels_vec_kernel(const ChannelParams p)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;      // group of four channels
    if (j >= p.N / 4) return;
    int zb[4], bias[4], mult[4], sh[4], rnd[4];
    // 32-bit form of the rounding shift (see requant() in q4_common.cuh) with zo - lo folded
    // into the rounding constant: ((hi + 2^(s-1) + (zo - lo) * 2^s) >> s), s = shift - 1, is
    // already value - lo before the clamp; it needs 2 <= shift <= 27 so that the sum stays inside
    // 32 bits.  Two values are then packed with saturation into the halves of one register,
    // clamped together, and three multiply-adds gather the four pairs.
    bool fast = true;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int n = 4 * j + e;
        zb[e] = p.zb ? p.zb[n] : 0;
        bias[e] = p.bias ? p.bias[n] : 0;
        mult[e] = p.mult[n];
        sh[e] = p.shift[n];
        fast = fast && sh[e] >= 2 && sh[e] <= 27;
        const int s = fast ? sh[e] - 1 : 1;
        rnd[e] = (1 << (s - 1)) + (p.zo - p.lo) * (1 << s);
    }
    const int kza = p.K * p.za;
    const uint32_t hml2 = (uint32_t)(p.hi - p.lo) * 0x00010001u, lofill = (uint32_t)p.lo * 0x11111111u;
    for (int r = 2 * blockIdx.y; r < p.M; r += 2 * gridDim.y) {
        const bool two = r + 1 < p.M;
        const int r1 = two ? r + 1 : r;
        const int4 c0 = __ldcs(reinterpret_cast<const int4*>(p.C0 + (int64_t)r * p.ldc + 4 * j));
        const int4 c1 = __ldcs(reinterpret_cast<const int4*>(p.C0 + (int64_t)r1 * p.ldc + 4 * j));
        const int f0 = p.rowsum_a[r] - kza, f1 = p.rowsum_a[r1] - kza;       // sum_k (a - za)
        const int a[4] = {c0.x, c0.y, c0.z, c0.w}, b[4] = {c1.x, c1.y, c1.z, c1.w};
        uint32_t word = 0;
        if (fast) {
            uint32_t pr[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int acc0 = (int)((uint32_t)a[e] - (uint32_t)(zb[e] * f0) + (uint32_t)bias[e]);
                const int acc1 = (int)((uint32_t)b[e] - (uint32_t)(zb[e] * f1) + (uint32_t)bias[e]);
                const int q0 = mulhi_add(acc0, mult[e], rnd[e]) >> (sh[e] - 1);
                const int q1 = mulhi_add(acc1, mult[e], rnd[e]) >> (sh[e] - 1);
                pr[e] = __vimin_s16x2_relu(pack_sat16(q1, q0), hml2);
            }
            word = mad_u32(pr[3], 1u << 12, mad_u32(pr[2], 1u << 8, mad_u32(pr[1], 1u << 4, pr[0]))) + lofill;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int acc0 = (int)((uint32_t)a[e] - (uint32_t)(zb[e] * f0) + (uint32_t)bias[e]);
                const int acc1 = (int)((uint32_t)b[e] - (uint32_t)(zb[e] * f1) + (uint32_t)bias[e]);
                word |= requant_one(acc0, mult[e], sh[e], p.zo, p.lo, p.hi) << (4 * e);
                word |= requant_one(acc1, mult[e], sh[e], p.zo, p.lo, p.hi) << (16 + 4 * e);
            }
        }
        *reinterpret_cast<uint16_t*>(p.Cq + (int64_t)r * p.ldcq + 2 * j) = (uint16_t)word;
        if (two) *reinterpret_cast<uint16_t*>(p.Cq + (int64_t)r1 * p.ldcq + 2 * j) = (uint16_t)(word >> 16);
    }
}

// Any shape and alignment: one output byte (two channels) per thread.
__global__ void __launch_bounds__(256)
requant_channels_byte_kernel(const ChannelParams p)
{
    const int nb = p.N / 2;
    const int64_t total = (int64_t)p.M * nb;
    const int kza = p.K * p.za;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / nb;
        const int j = (int)(i - r * nb);
        const int rowfac = p.rowsum_a[r] - kza;
        uint32_t byte = 0;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int n = 2 * j + e;
            const int zb = p.zb ? p.zb[n] : 0, bias = p.bias ? p.bias[n] : 0;
            const int acc = (int)((uint32_t)p.C0[r * p.ldc + n] - (uint32_t)(zb * rowfac) + (uint32_t)bias);
            byte |= requant_one(acc, p.mult[n], p.shift[n], p.zo, p.lo, p.hi) << (4 * e);
        }
        p.Cq[r * p.ldcq + j] = (uint8_t)byte;
    }
}

cudaError_t launch_requant_channels(const int32_t* C0, int64_t ldc, int32_t M, int32_t N, int32_t K,
                                    int32_t za, const int32_t* rowsum_a, const int32_t* zb,
                                    const int32_t* bias, const int32_t* mult, const int32_t* shift,
                                    int32_t zo, int32_t lo, int32_t hi, uint8_t* Cq, int64_t ldcq,
                                    cudaStream_t st)
{
    ChannelParams p{C0, ldc, M, N, K, za, rowsum_a, zb, bias, mult, shift, zo, lo, hi, Cq, ldcq};
    const bool vec = N % 4 == 0 && ldc % 4 == 0 && (uintptr_t)C0 % 16 == 0 && ldcq % 2 == 0 &&
                     (uintptr_t)Cq % 2 == 0;
    if (vec) {
        // one resident wave: six blocks of 256 threads per SM (more blocks than are resident
        // at once measured slower: 148 x 8 blocks 71 us against 57 us at 8192 x 8192)
        const int groups = N / 4;
        const int bx = groups < 256 ? (groups + 31) / 32 * 32 : 256;
        const unsigned gx = (unsigned)((groups + bx - 1) / bx);
        int64_t gy = (int64_t)148 * 6 / gx;
        if (gy < 1) gy = 1;
        if (gy > ((int64_t)M + 1) / 2) gy = ((int64_t)M + 1) / 2;
        if (gy > 65535) gy = 65535;
        requant_channels_vec_kernel<<<dim3(gx, (unsigned)gy), bx, 0, st>>>(p);
    } else {
        int64_t blocks = ((int64_t)M * (N / 2) + 255) / 256;
        if (blocks > 148 * 16) blocks = 148 * 16;
        requant_channels_byte_kernel<<<(int)blocks, 256, 0, st>>>(p);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace q4
