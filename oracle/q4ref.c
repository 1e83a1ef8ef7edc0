/*
 * q4ref -- CPU oracle (see q4ref.h).  TEST INFRASTRUCTURE ONLY.
 *
 * Plain C, 64-bit accumulation, no blocking, no fusion, no intrinsics.  Each
 * function is the definition it cites, looped in the obvious order; OpenMP only
 * splits the outermost row loop.  Nothing here is shared with the CUDA library.
 *
 * Parity unpinned by the paper (semantics fixed by the workload statement only):
 * the in-memory nibble packing (q4ref_pack_row / q4ref_unpack_row) and the integer
 * re-quantization (q4ref_requant_value).  Both are pinned in the tests by
 * hand-written byte examples and by arbitrary-precision arithmetic respectively.
 */
#include "q4ref.h"

#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static int g_threads = 0; /* 0 = OpenMP default */

int q4ref_num_threads(void)
{
#ifdef _OPENMP
    return g_threads > 0 ? g_threads : omp_get_max_threads();
#else
    return 1;
#endif
}

void q4ref_set_num_threads(int n)
{
    g_threads = n > 0 ? n : 0;
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#endif
}

/* Element e of a flat nibble array: byte e >> 1, low nibble when e is even. */
static inline int nib_get(const uint8_t* p, int64_t e)
{
    uint8_t byte = p[e >> 1];
    return (e & 1) ? (byte >> 4) : (byte & 0x0F);
}

static inline void nib_set(uint8_t* p, int64_t e, int v)
{
    uint8_t byte = p[e >> 1];
    if (e & 1) byte = (uint8_t)((byte & 0x0F) | ((v & 0x0F) << 4));
    else       byte = (uint8_t)((byte & 0xF0) | (v & 0x0F));
    p[e >> 1] = byte;
}

void q4ref_unpack_row(const uint8_t* packed, int64_t count, uint8_t* values)
{
    for (int64_t e = 0; e < count; ++e) values[e] = (uint8_t)nib_get(packed, e);
}

int q4ref_pack_row(const uint8_t* values, int64_t count, uint8_t* packed)
{
    if (count < 0) return Q4REF_E_ARG;
    for (int64_t e = 0; e < count; ++e)
        if (values[e] > 15) return Q4REF_E_RANGE;
    memset(packed, 0, (size_t)((count + 1) / 2));
    for (int64_t e = 0; e < count; ++e) nib_set(packed, e, values[e]);
    return Q4REF_OK;
}

static int check_gemm_args(const void* A, int64_t lda, const void* Bt, int64_t ldb,
                           int32_t M, int32_t N, int32_t K, int32_t za, int32_t zb)
{
    if (M < 0 || N < 0 || K < 1) return Q4REF_E_ARG;
    if ((M > 0 && !A) || (N > 0 && !Bt)) return Q4REF_E_ARG;
    if (lda < (K + 1) / 2 || ldb < (K + 1) / 2) return Q4REF_E_ARG;
    if (za < 0 || za > 15 || zb < 0 || zb > 15) return Q4REF_E_RANGE;
    return Q4REF_OK;
}

/* Odd K: the unused high nibble of each row's last byte must be zero (pad contract). */
static int check_odd_k_pad(const uint8_t* P, int64_t ld, int32_t rows, int32_t K)
{
    if ((K & 1) == 0) return Q4REF_OK;
    for (int32_t r = 0; r < rows; ++r)
        if (P[(int64_t)r * ld + (K >> 1)] >> 4) return Q4REF_E_PAD;
    return Q4REF_OK;
}

/* One value per byte copies of the operands: a[m*K + k], b[n*K + k]. */
static uint8_t* unpack_matrix(const uint8_t* P, int64_t ld, int32_t rows, int32_t K)
{
    size_t bytes = (size_t)rows * (size_t)K;
    uint8_t* u = (uint8_t*)malloc(bytes ? bytes : 1);
    if (!u) return NULL;
    for (int32_t r = 0; r < rows; ++r)
        q4ref_unpack_row(P + (int64_t)r * ld, K, u + (size_t)r * K);
    return u;
}

/* Eq. 2 (Section II-B), middle expression without s_w s_x; Eq. 3 (Section III-A). */
int q4ref_gemm(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
               int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
               int32_t za, int32_t zb)
{
    int rc = check_gemm_args(A, lda, Bt, ldb, M, N, K, za, zb);
    if (rc) return rc;
    if (M == 0 || N == 0) return Q4REF_OK;
    if (!C || ldc < N) return Q4REF_E_ARG;
    if ((rc = check_odd_k_pad(A, lda, M, K)) || (rc = check_odd_k_pad(Bt, ldb, N, K))) return rc;

    uint8_t* a = unpack_matrix(A, lda, M, K);
    uint8_t* b = unpack_matrix(Bt, ldb, N, K);
    if (!a || !b) { free(a); free(b); return Q4REF_E_ARG; }

    int bad = 0;
#pragma omp parallel for schedule(static) reduction(|:bad)
    for (int32_t m = 0; m < M; ++m) {
        const uint8_t* am = a + (size_t)m * K;
        for (int32_t n = 0; n < N; ++n) {
            const uint8_t* bn = b + (size_t)n * K;
            int64_t acc = 0;
            for (int32_t k = 0; k < K; ++k)
                acc += (int64_t)((int)am[k] - za) * (int64_t)((int)bn[k] - zb);
            /* |(a-za)(b-zb)| <= 15*15 = 225 (Section III-A) */
            if (acc > (int64_t)225 * K || acc < -(int64_t)225 * K) bad |= 1;
            C[(int64_t)m * ldc + n] = (int32_t)acc;
        }
    }
    free(a); free(b);
    return bad ? Q4REF_E_RANGE : Q4REF_OK;
}

/* Eq. 2 last line / Eq. 3: sum w x - z_w sum x - z_x sum w + D z_x z_w. */
int q4ref_gemm_fourterm(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                        int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
                        int32_t za, int32_t zb, int32_t* rowsum_a, int32_t* colsum_b)
{
    int rc = check_gemm_args(A, lda, Bt, ldb, M, N, K, za, zb);
    if (rc) return rc;
    if (M > 0 && N > 0 && (!C || ldc < N)) return Q4REF_E_ARG;
    if ((rc = check_odd_k_pad(A, lda, M, K)) || (rc = check_odd_k_pad(Bt, ldb, N, K))) return rc;

    uint8_t* a = unpack_matrix(A, lda, M, K);
    uint8_t* b = unpack_matrix(Bt, ldb, N, K);
    int64_t* ra = (int64_t*)calloc((size_t)(M ? M : 1), sizeof(int64_t));
    int64_t* cb = (int64_t*)calloc((size_t)(N ? N : 1), sizeof(int64_t));
    if (!a || !b || !ra || !cb) { free(a); free(b); free(ra); free(cb); return Q4REF_E_ARG; }

    /* second term's sum: over the depth of the activation matrix */
    for (int32_t m = 0; m < M; ++m)
        for (int32_t k = 0; k < K; ++k) ra[m] += a[(size_t)m * K + k];
    /* third term's sum: over the depth of the weight matrix (computed once per weights) */
    for (int32_t n = 0; n < N; ++n)
        for (int32_t k = 0; k < K; ++k) cb[n] += b[(size_t)n * K + k];

#pragma omp parallel for schedule(static)
    for (int32_t m = 0; m < M; ++m) {
        for (int32_t n = 0; n < N; ++n) {
            int64_t raw = 0; /* first term: product of the quantized matrices */
            for (int32_t k = 0; k < K; ++k)
                raw += (int64_t)a[(size_t)m * K + k] * (int64_t)b[(size_t)n * K + k];
            int64_t r = raw - (int64_t)zb * ra[m] - (int64_t)za * cb[n]
                      + (int64_t)K * za * zb;
            C[(int64_t)m * ldc + n] = (int32_t)r;
        }
    }
    if (rowsum_a) for (int32_t m = 0; m < M; ++m) rowsum_a[m] = (int32_t)ra[m];
    if (colsum_b) for (int32_t n = 0; n < N; ++n) colsum_b[n] = (int32_t)cb[n];
    free(a); free(b); free(ra); free(cb);
    return Q4REF_OK;
}

static int check_requant(const q4ref_requant* rq)
{
    if (!rq) return Q4REF_E_ARG;
    if (rq->mult < (1 << 30)) return Q4REF_E_RANGE;           /* [2^30, 2^31) */
    if (rq->shift < 0 || rq->shift > 31) return Q4REF_E_RANGE;
    if (rq->zo < 0 || rq->zo > 15) return Q4REF_E_RANGE;
    if (rq->clamp_lo < 0 || rq->clamp_hi > 15 || rq->clamp_lo > rq->clamp_hi) return Q4REF_E_RANGE;
    return Q4REF_OK;
}

/* floor(x / 2^t) for any sign, without relying on how >> treats negatives. */
static int64_t floor_div_pow2(int64_t x, int t)
{
    int64_t d = (int64_t)1 << t;
    int64_t q = x / d;            /* truncates toward zero */
    if ((x % d) < 0) q -= 1;      /* step down for negative non-multiples */
    return q;
}

int32_t q4ref_requant_value(int64_t acc, const q4ref_requant* rq)
{
    int t = 31 + rq->shift;
    int64_t half = (int64_t)1 << (t - 1);
    int64_t q = floor_div_pow2(acc * (int64_t)rq->mult + half, t);
    int64_t y = q + rq->zo;
    if (y < rq->clamp_lo) y = rq->clamp_lo;
    if (y > rq->clamp_hi) y = rq->clamp_hi;
    return (int32_t)y;
}

int q4ref_requant_matrix(const int32_t* C, int64_t ldc, int32_t M, int32_t N,
                         const int32_t* bias, const q4ref_requant* rq,
                         uint8_t* Cq, int64_t ldcq)
{
    int rc = check_requant(rq);
    if (rc) return rc;
    if (M < 0 || N < 0 || (N & 1)) return Q4REF_E_ARG;
    if (M == 0 || N == 0) return Q4REF_OK;
    if (!C || !Cq || ldc < N || ldcq < N / 2) return Q4REF_E_ARG;
    for (int32_t m = 0; m < M; ++m) {
        for (int32_t n = 0; n < N; ++n) {
            int64_t acc = (int64_t)C[(int64_t)m * ldc + n] + (bias ? (int64_t)bias[n] : 0);
            if (acc > INT32_MAX || acc < INT32_MIN) return Q4REF_E_RANGE;
        }
    }
    for (int32_t m = 0; m < M; ++m) {
        uint8_t* row = Cq + (int64_t)m * ldcq;
        for (int32_t n = 0; n < N; ++n) {
            int64_t acc = (int64_t)C[(int64_t)m * ldc + n] + (bias ? (int64_t)bias[n] : 0);
            nib_set(row, n, q4ref_requant_value(acc, rq));
        }
    }
    return Q4REF_OK;
}

int q4ref_gemm_requant(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                       int32_t M, int32_t N, int32_t K, int32_t za, int32_t zb,
                       const int32_t* bias, const q4ref_requant* rq,
                       uint8_t* Cq, int64_t ldcq)
{
    int rc = check_requant(rq);
    if (rc) return rc;
    if (M < 0 || N < 0 || (N & 1)) return Q4REF_E_ARG;
    size_t cells = (size_t)M * (size_t)N;
    int32_t* C = (int32_t*)malloc((cells ? cells : 1) * sizeof(int32_t));
    if (!C) return Q4REF_E_ARG;
    rc = q4ref_gemm(A, lda, Bt, ldb, C, N, M, N, K, za, zb);
    if (!rc) rc = q4ref_requant_matrix(C, N, M, N, bias, rq, Cq, ldcq);
    free(C);
    return rc;
}

int32_t q4ref_conv_out(int32_t in, int32_t k, int32_t stride, int32_t pad)
{
    int32_t span = in + 2 * pad - k;
    if (span < 0 || stride < 1) return 0;
    return span / stride + 1;
}

static int check_conv(const q4ref_conv_desc* d, int32_t za)
{
    if (!d) return Q4REF_E_ARG;
    if (d->N < 0 || d->H < 1 || d->W < 1 || d->C < 1) return Q4REF_E_ARG;
    if (d->OC < 0 || d->KH < 1 || d->KW < 1) return Q4REF_E_ARG;
    if (d->stride_h < 1 || d->stride_w < 1 || d->pad_h < 0 || d->pad_w < 0) return Q4REF_E_ARG;
    if (d->H + 2 * d->pad_h < d->KH || d->W + 2 * d->pad_w < d->KW) return Q4REF_E_ARG;
    if (za < 0 || za > 15) return Q4REF_E_RANGE;
    return Q4REF_OK;
}

/* Input value seen by a tap at (h, w): the pixel, or the zero point outside the image. */
static inline int tap(const uint8_t* X, const q4ref_conv_desc* d, int32_t n,
                      int32_t h, int32_t w, int32_t c, int32_t za)
{
    if (h < 0 || h >= d->H || w < 0 || w >= d->W) return za;
    int64_t e = (((int64_t)n * d->H + h) * d->W + w) * d->C + c;
    return nib_get(X, e);
}

/* Unrolling of the input for GEMM-based convolution (Section I; depth D = kh kw c,
 * Section III-A); the per-row sums are the second term's sums of Eq. 2, taken
 * "while unrolling" as Section II-B suggests. */
int q4ref_im2col(const uint8_t* X, const q4ref_conv_desc* d, int32_t za,
                 uint8_t* A, int64_t lda, int32_t* rowsum_a)
{
    int rc = check_conv(d, za);
    if (rc) return rc;
    int32_t OH = q4ref_conv_out(d->H, d->KH, d->stride_h, d->pad_h);
    int32_t OW = q4ref_conv_out(d->W, d->KW, d->stride_w, d->pad_w);
    int64_t K = (int64_t)d->KH * d->KW * d->C;
    if (lda < (K + 1) / 2) return Q4REF_E_ARG;
    if (d->N == 0) return Q4REF_OK;
    if (!X || !A) return Q4REF_E_ARG;

    for (int32_t n = 0; n < d->N; ++n)
    for (int32_t oh = 0; oh < OH; ++oh)
    for (int32_t ow = 0; ow < OW; ++ow) {
        int64_t m = ((int64_t)n * OH + oh) * OW + ow;
        uint8_t* row = A + m * lda;
        memset(row, 0, (size_t)lda);
        int64_t sum = 0;
        for (int32_t kh = 0; kh < d->KH; ++kh)
        for (int32_t kw = 0; kw < d->KW; ++kw)
        for (int32_t c = 0; c < d->C; ++c) {
            int64_t k = ((int64_t)kh * d->KW + kw) * d->C + c;
            int v = tap(X, d, n, oh * d->stride_h - d->pad_h + kh,
                        ow * d->stride_w - d->pad_w + kw, c, za);
            nib_set(row, k, v);
            sum += v;
        }
        if (rowsum_a) rowsum_a[m] = (int32_t)sum;
    }
    return Q4REF_OK;
}

/* The convolution sum itself, without unrolling, zero points as in Eq. 2. */
int q4ref_conv2d_direct(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                        const q4ref_conv_desc* d, int32_t za, int32_t zb, int32_t* Y32)
{
    int rc = check_conv(d, za);
    if (rc) return rc;
    if (zb < 0 || zb > 15) return Q4REF_E_RANGE;
    int32_t OH = q4ref_conv_out(d->H, d->KH, d->stride_h, d->pad_h);
    int32_t OW = q4ref_conv_out(d->W, d->KW, d->stride_w, d->pad_w);
    int64_t K = (int64_t)d->KH * d->KW * d->C;
    if (ldw < (K + 1) / 2) return Q4REF_E_ARG;
    if (d->N == 0 || d->OC == 0) return Q4REF_OK;
    if (!X || !Wt || !Y32) return Q4REF_E_ARG;

#pragma omp parallel for schedule(static)
    for (int32_t n = 0; n < d->N; ++n)
    for (int32_t oh = 0; oh < OH; ++oh)
    for (int32_t ow = 0; ow < OW; ++ow)
    for (int32_t oc = 0; oc < d->OC; ++oc) {
        const uint8_t* w = Wt + (int64_t)oc * ldw;
        int64_t acc = 0;
        for (int32_t kh = 0; kh < d->KH; ++kh)
        for (int32_t kw = 0; kw < d->KW; ++kw)
        for (int32_t c = 0; c < d->C; ++c) {
            int x = tap(X, d, n, oh * d->stride_h - d->pad_h + kh,
                        ow * d->stride_w - d->pad_w + kw, c, za);
            int wv = nib_get(w, ((int64_t)kh * d->KW + kw) * d->C + c);
            acc += (int64_t)(x - za) * (int64_t)(wv - zb);
        }
        Y32[((((int64_t)n * OH + oh) * OW + ow) * d->OC) + oc] = (int32_t)acc;
    }
    return Q4REF_OK;
}

int q4ref_conv2d(const uint8_t* X, const uint8_t* Wt, int64_t ldw, const int32_t* bias,
                 const q4ref_conv_desc* d, int32_t za, int32_t zb,
                 const q4ref_requant* rq, uint8_t* Y)
{
    int rc = check_conv(d, za);
    if (rc) return rc;
    if ((rc = check_requant(rq))) return rc;
    if (d->OC & 1) return Q4REF_E_ARG;
    int32_t OH = q4ref_conv_out(d->H, d->KH, d->stride_h, d->pad_h);
    int32_t OW = q4ref_conv_out(d->W, d->KW, d->stride_w, d->pad_w);
    int64_t M = (int64_t)d->N * OH * OW;
    size_t cells = (size_t)M * (size_t)d->OC;
    int32_t* Y32 = (int32_t*)malloc((cells ? cells : 1) * sizeof(int32_t));
    if (!Y32) return Q4REF_E_ARG;
    rc = q4ref_conv2d_direct(X, Wt, ldw, d, za, zb, Y32);
    if (!rc) rc = q4ref_requant_matrix(Y32, d->OC, (int32_t)M, d->OC, bias, rq, Y, d->OC / 2);
    free(Y32);
    return rc;
}

int q4ref_pack_bt(const uint8_t* B_kn, int64_t ldb_kn, uint8_t* Bt, int64_t ldb,
                  int32_t K, int32_t N)
{
    if (K < 1 || N < 0 || ldb_kn < (N + 1) / 2 || ldb < (K + 1) / 2) return Q4REF_E_ARG;
    if (N == 0) return Q4REF_OK;
    if (!B_kn || !Bt) return Q4REF_E_ARG;
    for (int32_t n = 0; n < N; ++n) {
        uint8_t* row = Bt + (int64_t)n * ldb;
        memset(row, 0, (size_t)ldb);
        for (int32_t k = 0; k < K; ++k)
            nib_set(row, k, nib_get(B_kn + (int64_t)k * ldb_kn, n));
    }
    return Q4REF_OK;
}
