// Unrolling of a packed NHWC input into the activation matrix of the GEMM
// (GEMM-based convolution, Section I; depth D = kh*kw*c, Section III-A), with the
// per-row sums of Eq. 2's second term taken on the way (Section II-B).
//
// Three kernels:
//  * im2col_tile_kernel -- same geometry as the next one, output pitch up to 1024 bytes:
//    a warp takes 32 consecutive output rows, one row per lane.  A lane decodes its
//    pixel once, walks its row's taps (the lanes' loads of one tap are consecutive
//    pixels of the input: coalesced), sums its row's values in a register and writes
//    the row into a shared-memory tile; the warp then copies the tile, which is one
//    contiguous piece of the matrix, to memory with full-line 128-bit stores.  No
//    atomics, no 64-bit divisions.
//  * im2col_vec_kernel  -- channels give byte-aligned taps of 4, 8 or a multiple of 16
//    bytes and the output pitch is a multiple of 16: one thread per 16-byte output
//    chunk, consecutive lanes write consecutive chunks (fully coalesced 128-bit
//    stores), taps are fetched with 4/8/16-byte loads that hit L1/L2 (each input pixel
//    is re-read kh*kw times, the input itself is read from HBM once).
//  * im2col_byte_kernel -- any geometry (odd channel counts make pixels
//    nibble-granular): one thread per output byte.
// Row sums of the last two kernels: lanes of one row are contiguous in a warp, so a segmented
// warp reduction leaves one atomicAdd per row per warp (rowsum is zeroed first); the tile
// kernel writes each row's sum directly.
#include "q4_common.cuh"

namespace q4 {

struct Im2colParams {
    const uint8_t* X;
    uint8_t* A;
    int32_t* rowsum;
    int64_t lda;
    int64_t M;
    int32_t H, W, C, KH, KW, OH, OW, sh, sw, ph, pw;
    int32_t K, za;
};

// Adds v over runs of equal `row` among the lanes of a warp; the first lane of each
// run issues one atomicAdd.  Runs must be contiguous in lane order.
__device__ __forceinline__ void segmented_row_add(int64_t row, int v, bool valid, int32_t* rowsum)
{
    const unsigned full = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31;
    if (!valid) { row = -1; v = 0; }
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int64_t r2 = __shfl_down_sync(full, row, off);
        const int v2 = __shfl_down_sync(full, v, off);
        if (lane + off < 32 && r2 == row) v += v2;
    }
    const int64_t rprev = __shfl_up_sync(full, row, 1);
    if (valid && (lane == 0 || rprev != row)) atomicAdd(&rowsum[row], v);
}

__device__ __forceinline__ void decode_row(const Im2colParams& p, int64_t m, int& n, int& ih0, int& iw0)
{
    const int ow = (int)(m % p.OW);
    const int64_t t = m / p.OW;
    const int oh = (int)(t % p.OH);
    n = (int)(t / p.OH);
    ih0 = oh * p.sh - p.ph;
    iw0 = ow * p.sw - p.pw;
}

// TAPB = bytes per tap (C/2): 4, 8 or 16 (16 also serves every multiple of 16, with
// `tapb` the true size).
template <int TAPB>
__global__ void __launch_bounds__(256) im2col_vec_kernel(const Im2colParams p, int tapb)
{
    const int cpr = (int)(p.lda / 16);                 // 16-byte chunks per output row
    const int64_t total = p.M * cpr;
    const int taps = p.KH * p.KW;
    const uint32_t zfill = (uint32_t)p.za * 0x11111111u;

    // grid-stride loop with a warp-uniform trip count (shuffles below need full warps)
    const int64_t start = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x);
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    const int64_t warp_base0 = start - (threadIdx.x & 31);
    for (int64_t base = warp_base0; base < total; base += step) {
        const int64_t g = base + (threadIdx.x & 31);
        const bool valid = g < total;
        int64_t m = 0;
        uint32_t w[4] = {0, 0, 0, 0};
        if (valid) {
            m = g / cpr;
            const int j = (int)(g % cpr);
            int n, ih0, iw0;
            decode_row(p, m, n, ih0, iw0);
            if (TAPB < 16) {
                constexpr int TPC = 16 / TAPB;          // taps per chunk
                constexpr int WPT = TAPB / 4;           // words per tap
#pragma unroll
                for (int i = 0; i < TPC; ++i) {
                    const int t = j * TPC + i;
                    if (t < taps) {
                        const int kh = t / p.KW, kw = t % p.KW;
                        const int ih = ih0 + kh, iw = iw0 + kw;
                        if (ih >= 0 && ih < p.H && iw >= 0 && iw < p.W) {
                            const uint8_t* src =
                                p.X + (((int64_t)n * p.H + ih) * p.W + iw) * TAPB;
                            if (WPT == 1) {
                                w[i] = *reinterpret_cast<const uint32_t*>(src);
                            } else {
                                const uint2 v = *reinterpret_cast<const uint2*>(src);
                                w[2 * i] = v.x; w[2 * i + 1] = v.y;
                            }
                        } else {
#pragma unroll
                            for (int q = 0; q < WPT; ++q) w[i * WPT + q] = zfill;
                        }
                    }
                }
            } else {
                const int byte0 = j * 16;
                const int t = byte0 / tapb, off = byte0 % tapb;
                if (t < taps) {
                    const int kh = t / p.KW, kw = t % p.KW;
                    const int ih = ih0 + kh, iw = iw0 + kw;
                    if (ih >= 0 && ih < p.H && iw >= 0 && iw < p.W) {
                        const uint4 v = *reinterpret_cast<const uint4*>(
                            p.X + (((int64_t)n * p.H + ih) * p.W + iw) * tapb + off);
                        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
                    } else {
                        w[0] = w[1] = w[2] = w[3] = zfill;
                    }
                }
            }
            *reinterpret_cast<uint4*>(p.A + g * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (p.rowsum) {
            const int s = nibble_sum(w[0]) + nibble_sum(w[1]) + nibble_sum(w[2]) + nibble_sum(w[3]);
            segmented_row_add(m, s, valid, p.rowsum);
        }
    }
}

// One output row per lane, 32 rows per warp and step; see the head of the file.
constexpr int TILE_WARPS = 8;             // warps per block at pitches up to 256 bytes; fewer above
constexpr int TILE_SMEM = TILE_WARPS * 32 * 256;   // 64 KB of tiles per block
constexpr int TILE_MAX_LDA = 1024;        // two warps per block at least; longer rows: next kernel

template <int TAPB>
__global__ void __launch_bounds__(TILE_WARPS * 32)
im2col_tile_kernel(const Im2colParams p, int tapb, FastDiv div_ow, FastDiv div_oh)
{
    extern __shared__ __align__(16) uint8_t tile_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lda = (int)p.lda, cpr = lda >> 4;
    uint8_t* tile = tile_smem + warp * 32 * lda;
    uint8_t* myrow = tile + lane * lda;
    const uint32_t zfill = (uint32_t)p.za * 0x11111111u;
    const uint32_t M = (uint32_t)p.M;
    const int64_t groups = ((int64_t)M + 31) / 32;
    const int64_t imgbytes = (int64_t)p.H * p.W * tapb;

    const int wpb = blockDim.x >> 5;                     // warps per block
    for (int64_t gi = (int64_t)blockIdx.x * wpb + warp; gi < groups; gi += (int64_t)gridDim.x * wpb) {
        const uint32_t m0 = (uint32_t)(gi * 32);
        const bool valid = m0 + lane < M;
        const uint32_t m = valid ? m0 + lane : m0;      // lanes past the end redo row m0 (not stored)
        const uint32_t q = fdiv(m, div_ow);
        const int ow = (int)(m - q * (uint32_t)p.OW);
        const uint32_t n = fdiv(q, div_oh);
        const int oh = (int)(q - n * (uint32_t)p.OH);
        const int ih0 = oh * p.sh - p.ph, iw0 = ow * p.sw - p.pw;
        const uint8_t* img = p.X + (int64_t)n * imgbytes;

        // row sum = (sum of low nibbles) + (sum of bytes - sum of low nibbles) / 16
        int sum_bytes = 0, sum_low = 0, kh = 0, kw = 0, off = 0;
#pragma unroll 4
        for (int j = 0; j < cpr; ++j) {
            uint32_t w[4] = {0, 0, 0, 0};
            if (TAPB < 16) {
                constexpr int TPC = 16 / TAPB;          // taps per chunk
                constexpr int WPT = TAPB / 4;           // words per tap
#pragma unroll
                for (int i = 0; i < TPC; ++i) {
                    if (kh < p.KH) {
                        const int ih = ih0 + kh, iw = iw0 + kw;
                        if ((unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W) {
                            const uint8_t* src = img + (ih * p.W + iw) * TAPB;
                            if (WPT == 1) {
                                w[i] = *reinterpret_cast<const uint32_t*>(src);
                            } else {
                                const uint2 v = *reinterpret_cast<const uint2*>(src);
                                w[2 * i] = v.x; w[2 * i + 1] = v.y;
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < WPT; ++e) w[i * WPT + e] = zfill;
                        }
                        if (++kw == p.KW) { kw = 0; ++kh; }
                    }
                }
            } else {
                if (kh < p.KH) {
                    const int ih = ih0 + kh, iw = iw0 + kw;
                    if ((unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W) {
                        const uint4 v = *reinterpret_cast<const uint4*>(
                            img + (int64_t)(ih * p.W + iw) * tapb + off);
                        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
                    } else {
                        w[0] = w[1] = w[2] = w[3] = zfill;
                    }
                    off += 16;
                    if (off == tapb) {
                        off = 0;
                        if (++kw == p.KW) { kw = 0; ++kh; }
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                sum_bytes = dp4a_u8(w[e], 0x01010101u, sum_bytes);
                sum_low = dp4a_u8(w[e] & 0x0F0F0F0Fu, 0x01010101u, sum_low);
            }
            *reinterpret_cast<uint4*>(myrow + 16 * j) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        __syncwarp();
        const uint32_t left = M - m0;
        const int nchunks = (int)(left < 32u ? left : 32u) * cpr;
        uint8_t* out = p.A + (int64_t)m0 * lda;
        for (int c = lane; c < nchunks; c += 32)
            __stcs(reinterpret_cast<uint4*>(out + 16 * c), *reinterpret_cast<const uint4*>(tile + 16 * c));
        if (p.rowsum && valid) p.rowsum[m] = sum_low + ((sum_bytes - sum_low) >> 4);
        __syncwarp();                                  // the tile is rewritten in the next step
    }
}

__device__ __forceinline__ uint32_t fetch_nibble(const Im2colParams& p, int n, int ih0, int iw0, int k)
{
    if (k >= p.K) return 0;
    const int c = k % p.C, t = k / p.C;
    const int kw = t % p.KW, kh = t / p.KW;
    const int ih = ih0 + kh, iw = iw0 + kw;
    if (ih < 0 || ih >= p.H || iw < 0 || iw >= p.W) return (uint32_t)p.za;
    const int64_t e = (((int64_t)n * p.H + ih) * p.W + iw) * p.C + c;
    const uint8_t byte = p.X[e >> 1];
    return (e & 1) ? (byte >> 4) : (byte & 0x0F);
}

__global__ void __launch_bounds__(256) im2col_byte_kernel(const Im2colParams p)
{
    const int64_t total = p.M * p.lda;
    const int64_t start = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x);
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t base = start - (threadIdx.x & 31); base < total; base += step) {
        const int64_t g = base + (threadIdx.x & 31);
        const bool valid = g < total;
        int64_t m = 0;
        uint32_t lo = 0, hi = 0;
        if (valid) {
            m = g / p.lda;
            const int kb = (int)(g % p.lda);
            int n, ih0, iw0;
            decode_row(p, m, n, ih0, iw0);
            lo = fetch_nibble(p, n, ih0, iw0, 2 * kb);
            hi = fetch_nibble(p, n, ih0, iw0, 2 * kb + 1);
            p.A[g] = (uint8_t)(lo | (hi << 4));
        }
        if (p.rowsum) segmented_row_add(m, (int)(lo + hi), valid, p.rowsum);
    }
}

cudaError_t launch_im2col(const uint8_t* X, const q4_conv_desc& d, int32_t za, uint8_t* A,
                          int64_t lda, int32_t* rowsum_a, cudaStream_t st)
{
    Im2colParams p;
    p.X = X; p.A = A; p.rowsum = rowsum_a; p.lda = lda;
    p.H = d.H; p.W = d.W; p.C = d.C; p.KH = d.KH; p.KW = d.KW;
    p.sh = d.stride_h; p.sw = d.stride_w; p.ph = d.pad_h; p.pw = d.pad_w;
    p.OH = (d.H + 2 * d.pad_h - d.KH) / d.stride_h + 1;
    p.OW = (d.W + 2 * d.pad_w - d.KW) / d.stride_w + 1;
    p.M = (int64_t)d.N * p.OH * p.OW;
    p.K = d.KH * d.KW * d.C;
    p.za = za;
    if (p.M == 0) return cudaSuccess;

    const int tapb = d.C / 2;
    const bool aligned = ((uintptr_t)X % 16 == 0) && ((uintptr_t)A % 16 == 0) && (lda % 16 == 0);
    const bool vec = aligned && (d.C % 2 == 0) && (tapb == 4 || tapb == 8 || tapb % 16 == 0);

    if (vec && lda <= TILE_MAX_LDA && p.M < (1ll << 31)) {
        // as many warps per block (up to eight) as fit 64 KB of row tiles
        int wpb = (int)(TILE_SMEM / (32 * lda));
        wpb = wpb < 1 ? 1 : wpb > TILE_WARPS ? TILE_WARPS : wpb;
        const size_t smem = (size_t)wpb * 32 * (size_t)lda;
        const FastDiv dow = make_fastdiv((uint32_t)p.OW), doh = make_fastdiv((uint32_t)p.OH);
        auto kernel = tapb == 4 ? im2col_tile_kernel<4> : tapb == 8 ? im2col_tile_kernel<8>
                                                                   : im2col_tile_kernel<16>;
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TILE_SMEM);
        if (e != cudaSuccess) return e;
        int per_sm = 1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, wpb * 32, smem) != cudaSuccess ||
            per_sm < 1)
            per_sm = 1;
        const int64_t groups = (p.M + 31) / 32;
        int64_t blocks = (groups + wpb - 1) / wpb;
        if (blocks > 148ll * per_sm) blocks = 148ll * per_sm;
        kernel<<<(int)blocks, wpb * 32, smem, st>>>(p, tapb, dow, doh);
        count_launch();
        return cudaGetLastError();
    }

    if (rowsum_a) {
        cudaError_t e = cudaMemsetAsync(rowsum_a, 0, sizeof(int32_t) * (size_t)p.M, st);
        if (e != cudaSuccess) return e;
    }
    const int64_t work = vec ? p.M * (lda / 16) : p.M * lda;
    int64_t blocks = (work + 255) / 256;
    const int64_t cap = 148 * 32;
    if (blocks > cap) blocks = cap;
    if (vec) {
        if (tapb == 4)      im2col_vec_kernel<4><<<(int)blocks, 256, 0, st>>>(p, tapb);
        else if (tapb == 8) im2col_vec_kernel<8><<<(int)blocks, 256, 0, st>>>(p, tapb);
        else                im2col_vec_kernel<16><<<(int)blocks, 256, 0, st>>>(p, tapb);
    } else {
        im2col_byte_kernel<<<(int)blocks, 256, 0, st>>>(p);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace q4
