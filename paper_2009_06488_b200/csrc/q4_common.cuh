// Shared device-side pieces of the q4 library: the zero-point correction of Eq. 2,
// the integer re-quantization, and the launch-parameter structs.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "q4.h"

namespace q4 {

// Bits of the device status word (reported by q4_last_device_status).
constexpr unsigned kStatusTimeout = 1u;
constexpr unsigned kStatusWeightImage = 2u;     // a prepared weight image with another layer's tag

struct RequantParams {
    int32_t mult, shift, zo, lo, hi;
};

struct GemmParams {
    const uint8_t* A;      // [M, lda] packed
    const uint8_t* Bt;     // [N, ldb] packed
    int64_t lda, ldb;
    int32_t M, N, K;
    int32_t za, zb;
    const int32_t* rowsum_a;   // optional
    const int32_t* colsum_b;   // optional
    const int32_t* bias;       // optional (requant only)
    int32_t* C;                // int32 output (q4_gemm)
    int64_t ldc;
    uint8_t* Cq;               // packed output (q4_gemm_requant)
    int64_t ldcq;
    RequantParams rq;
    // per output channel (q4_gemm_requant_channels; mult_ch and shift_ch both or neither):
    // weight zero points (NULL = 0), multipliers, shifts.  zb, rq.mult and rq.shift are
    // then unused.
    const int32_t* zb_ch;
    const int32_t* mult_ch;
    const int32_t* shift_ch;
    unsigned* status;          // device status word
};

// Eq. 2, last line: raw product minus the two zero-point terms plus the constant.
// Wrapping int32 arithmetic; the true value is bounded by 225*K <= 2^30.
__device__ __forceinline__ int32_t correct(int32_t raw, int32_t rowsum, int32_t colsum,
                                           int32_t za, int32_t zb, int32_t kzz)
{
    return (int32_t)((uint32_t)raw - (uint32_t)(zb * rowsum) - (uint32_t)(za * colsum)
                     + (uint32_t)kzz);
}

// q = floor((acc*mult + 2^(30+shift)) / 2^(31+shift)); y = clamp(q + zo, lo, hi).
// |acc| < 2^31 and mult < 2^31 keep the 64-bit sum below 2^63; >> on a signed
// 64-bit value is an arithmetic (flooring) shift.
__device__ __forceinline__ uint32_t requant_wide(int32_t acc, const RequantParams& rq)
{
    const int t = 31 + rq.shift;
    long long v = (long long)acc * (long long)rq.mult + (1ll << (t - 1));
    int q = (int)(v >> t) + rq.zo;
    q = max(q, rq.lo);
    q = min(q, rq.hi);
    return (uint32_t)q;
}

// The same value from the high half of the product when shift >= 2.  With
// P = acc*mult = hi*2^32 + lo (0 <= lo < 2^32) and s = shift - 1 >= 1:
//   floor((P + 2^(31+shift-1)) / 2^(31+shift)) = floor((hi + 2^(s-1) + lo/2^32) / 2^s)
//                                              = floor((hi + 2^(s-1)) / 2^s),
// because hi + 2^(s-1) is an integer and lo/2^32 < 1 cannot carry it over a multiple
// of 2^s.  |hi| < 2^30, so the 32-bit sum cannot overflow.
__device__ __forceinline__ uint32_t requant(int32_t acc, const RequantParams& rq)
{
    if (rq.shift < 2) return requant_wide(acc, rq);       // uniform branch
    const int s = rq.shift - 1;
    int q = ((__mulhi(acc, rq.mult) + (1 << (s - 1))) >> s) + rq.zo;
    q = max(q, rq.lo);
    q = min(q, rq.hi);
    return (uint32_t)q;
}

// Unsigned 4 x 8-bit dot product accumulated into a (wrapping) 32-bit value.
__device__ __forceinline__ int dp4a_u8(uint32_t a, uint32_t b, int c)
{
    return (int)__dp4a(a, b, (uint32_t)c);
}

// Sum of the eight nibbles of a packed 32-bit word.
__device__ __forceinline__ int nibble_sum(uint32_t w)
{
    uint32_t s = (w & 0x0F0F0F0Fu) + ((w >> 4) & 0x0F0F0F0Fu);   // bytes <= 30
    return dp4a_u8(s, 0x01010101u, 0);
}

// n / d for n < 2^31 as (umulhi(n, mul) + n) >> shift (round-up method: shift =
// ceil(log2 d), mul = floor(2^32 * (2^shift - d) / d) + 1).
struct FastDiv {
    uint32_t mul, shift;
};

inline FastDiv make_fastdiv(uint32_t d)
{
    FastDiv f;
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    f.shift = l;
    f.mul = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
    return f;
}

__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv& f)
{
    return (__umulhi(n, f.mul) + n) >> f.shift;
}

// ----- launchers implemented in the kernel translation units -----------------------
cudaError_t launch_gemm_simt(const GemmParams& p, bool requant, cudaStream_t st);
bool        gemm_tc_supported(const GemmParams& p);
q4_status   launch_gemm_tc(const GemmParams& p, bool requant, cudaStream_t st);
bool        gemm_tc_pair_supported(const GemmParams& p);
// width: 192 or 256 columns per tile, 0 = chosen from the problem's shape
q4_status   launch_gemm_tc_pair(const GemmParams& p, bool requant, cudaStream_t st, int width = 0);
cudaError_t launch_pack_bt(const uint8_t* B_kn, int64_t ldb_kn, uint8_t* Bt, int64_t ldb,
                           int32_t K, int32_t N, cudaStream_t st);
cudaError_t launch_row_sums(const uint8_t* P, int64_t ld, int32_t rows, int32_t K,
                            int32_t* sums, cudaStream_t st);
cudaError_t launch_operand_sums(const uint8_t* A, int64_t lda, int32_t rows_a, int32_t* sums_a,
                                const uint8_t* B, int64_t ldb, int32_t rows_b, int32_t* sums_b,
                                int32_t K, cudaStream_t st);
bool        conv_fused_supported(const q4_conv_desc& d, const uint8_t* X, const uint8_t* Wt,
                                 int64_t ldw, const uint8_t* Y, bool per_channel = false);
// zb_ch / mult_ch / shift_ch: all three (per-output-channel weight zero points, multipliers
// and shifts; zb and rq.mult / rq.shift are then unused) or none.
cudaError_t launch_conv_fused(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                              const int32_t* colsum_w, const int32_t* bias, const q4_conv_desc& d,
                              int32_t za, int32_t zb, const RequantParams& rq, uint8_t* Y,
                              cudaStream_t st, const int32_t* zb_ch = nullptr,
                              const int32_t* mult_ch = nullptr, const int32_t* shift_ch = nullptr);
// The same layer on the tensor-memory path (tcgen05 implicit GEMM), for the layer classes
// it has instances for.
bool        conv_tc_supported(const q4_conv_desc& d, const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                              const uint8_t* Y);
// prep_out: only prepare the layer's weight image (conv_tc_image_bytes(d) bytes) there;
// prep_in: run the layer from such an image instead of Wt / colsum_w / bias / zb.
cudaError_t launch_conv_tc(const uint8_t* X, const uint8_t* Wt, int64_t ldw, const int32_t* colsum_w,
                           const int32_t* bias, const q4_conv_desc& d, int32_t za, int32_t zb,
                           const RequantParams& rq, uint8_t* Y, cudaStream_t st,
                           const uint8_t* prep_in = nullptr, uint8_t* prep_out = nullptr,
                           const int32_t* zb_ch = nullptr, const int32_t* mult_ch = nullptr,
                           const int32_t* shift_ch = nullptr);
size_t      conv_tc_image_bytes(const q4_conv_desc& d);
cudaError_t launch_im2col(const uint8_t* X, const q4_conv_desc& d, int32_t za, uint8_t* A,
                          int64_t lda, int32_t* rowsum_a, cudaStream_t st);

cudaError_t launch_quant_params(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                                q4_qparams* qp, cudaStream_t st);
cudaError_t launch_quantize(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                            const q4_qparams* qp, uint8_t* Q, int64_t ldq, cudaStream_t st);
cudaError_t launch_dequantize(const int32_t* C, int64_t ldc, int32_t rows, int32_t cols, float scale,
                              float* R, int64_t ldr, cudaStream_t st);

q4_status   launch_gemm_u8(const GemmParams& p, cudaStream_t st);
// depth sums of the rows of A and of Bt (one byte per value) in one launch; rows_a or rows_b
// may be 0
cudaError_t launch_byte_sums(const uint8_t* A, int64_t lda, int32_t rows_a, int32_t* sums_a,
                             const uint8_t* B, int64_t ldb, int32_t rows_b, int32_t* sums_b, int32_t K,
                             cudaStream_t st);

cudaError_t launch_wait_selftest(int* outcome_dev, cudaStream_t st);

cudaError_t launch_requant_channels(const int32_t* C0, int64_t ldc, int32_t M, int32_t N, int32_t K,
                                    int32_t za, const int32_t* rowsum_a, const int32_t* zb,
                                    const int32_t* bias, const int32_t* mult, const int32_t* shift,
                                    int32_t zo, int32_t lo, int32_t hi, uint8_t* Cq, int64_t ldcq,
                                    cudaStream_t st);

void count_launch(int n = 1);
void log_choice(const char* call, const char* kernel);   // Q4_LOG=1: which kernel a call was given

}  // namespace q4
