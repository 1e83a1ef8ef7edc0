/*
 * q4ref -- CPU oracle for the 4-bit quantized GEMM / GEMM-based convolution path.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct statement of
 * what the path computes.  It shares no code with the CUDA library and must never
 * be called from the product path; only tests, the smoke check and the benchmark's
 * CPU-baseline leg use it.
 *
 * Every function is the plain definition written out (the method reaches the
 * definition exactly, so the oracle is the definition):
 *   - quantized product with zero points: the middle expression of Eq. 2
 *     (Section II-B) without the float scales, i.e. Eq. 3 (Section III-A);
 *   - the four-term rearrangement of Eq. 2/3 as a second, independent form;
 *   - GEMM-based convolution: unrolling of the input (Section I; D = kh*kw*c,
 *     Section III-A) and, independently, the direct convolution sum.
 * The integer re-quantization step (fixed-point multiplier, rounding shift, clamp,
 * repack) has no counterpart in the paper, which re-quantizes in floating point
 * (Section III-A/B); its semantics come from the workload statement and are
 * "parity unpinned" by the paper.  The nibble packing in memory (two values per
 * byte, low nibble = even index) is likewise "parity unpinned" by the paper,
 * which keeps one value per byte in its buffers (Section II-C).
 *
 * Conventions.  C = A x B with A = activations (M x K), B = weights (K x N).  The
 * paper writes R = W X with the weights on the left, so C = R^T, za = z_x,
 * zb = z_w, K = D.  Both operands are stored K-contiguous: A as M rows, Bt (= B
 * transposed) as N rows; every row is a flat nibble array, element e in byte
 * e >> 1, low nibble when e is even.  lda / ldb / ldw / ldcq are row pitches in
 * bytes, ldc is a pitch in int32 elements.
 *
 * All functions return 0 on success and a negative code on a violated
 * precondition (nothing is written in that case).
 */
#ifndef Q4REF_H
#define Q4REF_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define Q4REF_OK          0
#define Q4REF_E_ARG      -1   /* bad size / pointer / pitch                        */
#define Q4REF_E_RANGE    -2   /* value outside its documented range                */
#define Q4REF_E_PAD      -4   /* odd-K row whose last high nibble is not zero      */

typedef struct {
    int32_t N, H, W, C;          /* input, NHWC                                */
    int32_t OC, KH, KW;          /* filters: OC x KH x KW x C                  */
    int32_t stride_h, stride_w;
    int32_t pad_h, pad_w;        /* out-of-image taps read as the input zero point */
} q4ref_conv_desc;

typedef struct {
    int32_t mult;                /* [2^30, 2^31): real multiplier = mult / 2^(31+shift) */
    int32_t shift;               /* 0..31                                              */
    int32_t zo;                  /* output zero point, 0..15                           */
    int32_t clamp_lo, clamp_hi;  /* 0 <= lo <= hi <= 15                                */
} q4ref_requant;

/* Number of OpenMP threads the row loops will use (1 if built without OpenMP). */
int q4ref_num_threads(void);
void q4ref_set_num_threads(int n);

/* Nibble helpers: unpack `count` values of a packed row into one byte each, and back.
 * pack writes ceil(count/2) bytes; an odd count leaves the last high nibble 0. */
void q4ref_unpack_row(const uint8_t* packed, int64_t count, uint8_t* values);
int  q4ref_pack_row(const uint8_t* values, int64_t count, uint8_t* packed);

/* C[m][n] = sum_k (a(m,k) - za) * (b(k,n) - zb): Eq. 2, middle expression, scales dropped. */
int q4ref_gemm(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
               int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
               int32_t za, int32_t zb);

/* Same result through the four terms of Eq. 2 / Eq. 3:
 * sum a*b - zb*sum_k a - za*sum_k b + K*za*zb.  Also returns the sums
 * (rowsum_a[M], colsum_b[N]; either may be NULL). */
int q4ref_gemm_fourterm(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                        int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
                        int32_t za, int32_t zb, int32_t* rowsum_a, int32_t* colsum_b);

/* One value: q = floor((acc*mult + 2^(30+shift)) / 2^(31+shift)), then
 * clamp(q + zo, lo, hi).  One rounding, ties toward +infinity. */
int32_t q4ref_requant_value(int64_t acc, const q4ref_requant* rq);

/* Cq[m][n] = requant(C[m][n] + bias[n]); packed two per byte along n (N even). */
int q4ref_requant_matrix(const int32_t* C, int64_t ldc, int32_t M, int32_t N,
                         const int32_t* bias, const q4ref_requant* rq,
                         uint8_t* Cq, int64_t ldcq);

/* q4ref_gemm followed by q4ref_requant_matrix. */
int q4ref_gemm_requant(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                       int32_t M, int32_t N, int32_t K, int32_t za, int32_t zb,
                       const int32_t* bias, const q4ref_requant* rq,
                       uint8_t* Cq, int64_t ldcq);

/* Output extent of a convolution axis: floor((in + 2*pad - k) / stride) + 1. */
int32_t q4ref_conv_out(int32_t in, int32_t k, int32_t stride, int32_t pad);

/* Unrolled activation matrix: A[(n,oh,ow)][(kh,kw,c)] = X[n, oh*s-p+kh, ow*s-p+kw, c],
 * or za outside the image.  Nibbles between K and the row pitch are written 0.
 * rowsum_a[m] = sum_k A[m][k] (may be NULL). */
int q4ref_im2col(const uint8_t* X, const q4ref_conv_desc* d, int32_t za,
                 uint8_t* A, int64_t lda, int32_t* rowsum_a);

/* Direct convolution, no unrolling:
 * Y32[n,oh,ow,oc] = sum_{kh,kw,c} (x~ - za) * (w[oc,kh,kw,c] - zb), x~ = za outside. */
int q4ref_conv2d_direct(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                        const q4ref_conv_desc* d, int32_t za, int32_t zb, int32_t* Y32);

/* Direct convolution + bias + requantize, packed NHWC output (OC even). */
int q4ref_conv2d(const uint8_t* X, const uint8_t* Wt, int64_t ldw, const int32_t* bias,
                 const q4ref_conv_desc* d, int32_t za, int32_t zb,
                 const q4ref_requant* rq, uint8_t* Y);

/* K x N matrix packed along n (row k, pitch ldb_kn) -> N x K packed along k (pitch ldb). */
int q4ref_pack_bt(const uint8_t* B_kn, int64_t ldb_kn, uint8_t* Bt, int64_t ldb,
                  int32_t K, int32_t N);

#ifdef __cplusplus
}
#endif
#endif
