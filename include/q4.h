/*
 * q4 -- 4-bit quantized GEMM and GEMM-based convolution for NVIDIA B200 (sm_100a).
 *
 * C ABI of the CUDA library.  The operations are those of the paper "Fast
 * Implementation of 4-bit Convolutional Neural Networks for Mobile Devices"
 * (arXiv 2009.06488): the widening product of two matrices of unsigned 4-bit
 * values with per-tensor zero points (Section II-B, Eq. 2), kept as an integer
 * result (Section III-A, Eq. 3) and handed to the next layer as 4-bit values
 * again, and the convolution that reduces to it by unrolling the input
 * (Section I; depth D = kh*kw*c, Section III-A).
 *
 * Naming.  C = A x B with A = activations (M x K, one row per output pixel) and
 * B = weights (K x N, one column per output channel).  The paper writes R = W X
 * with the weights on the left; C = R^T, za = z_x, zb = z_w, K = D,
 * rowsum_a[m] = sum_k x^_{kj} (the second term's sum) and colsum_b[n] =
 * sum_k w^_{ik} (the third term's sum, computed once per weight matrix).
 *
 * Data layout.  A uint4 array is a flat nibble array: element e lives in byte
 * e >> 1, in the low nibble when e is even.  Both GEMM operands are
 * K-contiguous: A is M rows of K nibbles with a row pitch of lda bytes, Bt
 * (= B transposed) is N rows of K nibbles with a row pitch of ldb bytes.  Bytes of
 * a row past ceil(K/2) are never read.  When K is odd the high nibble of a row's
 * last byte must be 0 (q4_im2col and q4_pack_bt write it so).  int32 matrices are
 * row-major with a pitch in elements; packed uint4 outputs are row-major along n
 * with a pitch in bytes, and need an even N.
 *
 * Pointers.  Every data pointer is a DEVICE pointer owned by the caller; the
 * library allocates nothing and keeps no buffers.  q4_requant and q4_conv_desc are
 * small HOST structs read during the call.  `stream` is a cudaStream_t passed as
 * void* (NULL = the legacy default stream).  Work is enqueued on that stream and
 * the call returns without synchronizing.  The q4_*_host entry points are the
 * exception: their data pointers are HOST pointers (see below).
 *
 * Errors.  Arguments are validated on the host before anything is launched; a
 * q4_status is returned and nothing traps or aborts.  Device-side waits are
 * bounded: a wait that expires sets a status word that q4_last_device_status
 * reports.
 *
 * Fast path.  Base pointers aligned to 16 bytes and lda / ldb multiples of 16 bytes
 * select the tensor-core kernels (TMA needs both); anything else runs a slower
 * general kernel with the same results.
 */
#ifndef Q4_H
#define Q4_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    Q4_OK = 0,
    Q4_ERR_INVALID_ARG = 1,     /* NULL pointer, negative size, pitch smaller than a row   */
    Q4_ERR_ALIGNMENT = 2,       /* a pointer / pitch breaks an alignment the call requires */
    Q4_ERR_RANGE = 3,           /* zero point, multiplier, shift, clamp or K out of range  */
    Q4_ERR_WORKSPACE = 4,       /* workspace missing or smaller than *_workspace_bytes     */
    Q4_ERR_UNSUPPORTED = 5,     /* valid, but this entry point has no kernel for it         */
    Q4_ERR_CUDA = 6,            /* a CUDA runtime / driver call failed                     */
    Q4_ERR_DEVICE_TIMEOUT = 7,  /* a bounded device-side wait expired                      */
    Q4_ERR_STATIC_SCRATCH = 8,  /* problem needs more scratch than q4_conv2d_static holds  */
    Q4_ERR_WEIGHT_IMAGE = 9     /* q4_conv2d_prepared was given another layer's weight image */
} q4_status;

/* Integer re-quantization of an int32 accumulator to the next layer's uint4 input.
 * The paper re-quantizes each layer's integer result to 4 bits for the next layer
 * (Section III-A/B) in floating point; here it is the fixed-point form
 *     q = floor((acc * mult + 2^(30+shift)) / 2^(31+shift))        (one rounding,
 *     y = min(max(q + zo, clamp_lo), clamp_hi)                      ties toward +inf)
 * i.e. the real multiplier is mult / 2^(31+shift).  This is deliberately a single
 * rounding, not a rounding high-multiply followed by a rounding shift.
 * ReLU is clamp_lo = zo. */
typedef struct {
    int32_t mult;       /* [2^30, 2^31) */
    int32_t shift;      /* 0..31        */
    int32_t zo;         /* 0..15        */
    int32_t clamp_lo;   /* 0 <= clamp_lo <= clamp_hi <= 15 */
    int32_t clamp_hi;
} q4_requant;

/* Convolution geometry: NHWC input, OC filters of KH x KW x C, dilation 1, groups 1.
 * Output extent per axis: floor((in + 2*pad - k) / stride) + 1.  Taps outside the
 * image read the input zero point za, so they contribute exactly 0. */
typedef struct {
    int32_t N, H, W, C;
    int32_t OC, KH, KW;
    int32_t stride_h, stride_w;
    int32_t pad_h, pad_w;
} q4_conv_desc;

/* Largest supported depth: every term of Eq. 2 (each at most 225*K) and their
 * partial sums stay inside int32. */
#define Q4_MAX_K (1 << 22)

/*
 * Quantized product, Eq. 2 / Eq. 3 without the float scales:
 *   C[m][n] = sum_k (a(m,k) - za) * (b(k,n) - zb)
 *           = sum_k a b  -  zb * rowsum_a[m]  -  za * colsum_b[n]  +  K * za * zb.
 * A [M x K] pitch lda bytes; Bt [N x K] pitch ldb bytes; C [M x N] int32, pitch ldc
 * elements (>= N).  za, zb in 0..15.  1 <= K <= Q4_MAX_K.  M or N = 0 is a no-op.
 * rowsum_a [M] / colsum_b [N]: optional precomputed sums (e.g. from q4_im2col, or
 * computed once for the weights); NULL = computed inside the kernel.
 * ws / ws_bytes: optional workspace of at least q4_gemm_workspace_bytes(M, N, K) bytes,
 * 16-byte aligned.  With it, large problems take the sums that were not supplied in
 * one bandwidth-bound pass over the operands instead of inside the GEMM kernel, which
 * is faster; without it (NULL) the result is the same.  Its contents are scratch.
 */
q4_status q4_gemm(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                  int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
                  int32_t za, int32_t zb,
                  const int32_t* rowsum_a, const int32_t* colsum_b,
                  void* ws, size_t ws_bytes, void* stream);

/*
 * Same product with the next layer's re-quantization fused into the epilogue
 * (Section III-A: the integer result goes through the activation and is quantized
 * to 4 bits again for the next layer):
 *   Cq[m][n] = requant(C[m][n] + bias[n])       (see q4_requant)
 * bias [N] int32 or NULL.  C[m][n] + bias[n] must fit in int32.  N must be even.
 * Cq is packed along n, pitch ldcq bytes (>= N/2).  The int32 matrix is never
 * written to memory.
 */
q4_status q4_gemm_requant(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                          int32_t M, int32_t N, int32_t K, int32_t za, int32_t zb,
                          const int32_t* rowsum_a, const int32_t* colsum_b,
                          const int32_t* bias, const q4_requant* rq,
                          uint8_t* Cq, int64_t ldcq,
                          void* ws, size_t ws_bytes, void* stream);

/*
 * Unrolling of a convolution input into the activation matrix of the GEMM
 * (Section I; Section III-A):
 *   A[(n,oh,ow)][(kh,kw,c)] = X[n, oh*stride_h - pad_h + kh, ow*stride_w - pad_w + kw, c]
 * or za where that tap is outside the image.  X is the flat packed NHWC array (no
 * pitches).  A has M = N*OH*OW rows of K = KH*KW*C nibbles, pitch lda bytes
 * (>= ceil(K/2)); every nibble from K to the end of the pitch is written 0.
 * rowsum_a [M] (optional): sum_k A[m][k], the second term's sums of Eq. 2, taken
 * while unrolling as Section II-B suggests.  d->OC is ignored.
 */
q4_status q4_im2col(const uint8_t* X, const q4_conv_desc* d, int32_t za,
                    uint8_t* A, int64_t lda, int32_t* rowsum_a, void* stream);

/*
 * One quantized convolution layer (Section III-A/B): unroll, multiply (Eq. 3), add
 * bias, re-quantize.  Wt: filters [OC][KH][KW][C] packed along (kh,kw,c), pitch ldw
 * bytes -- this is Bt of the GEMM.  colsum_w [OC]: optional precomputed
 * sum_{kh,kw,c} w (the third term's sums), NULL = computed.  Y: packed NHWC output
 * N x OH x OW x OC (flat, row pitch OC/2 bytes; OC even).
 * ws: at least q4_conv2d_workspace_bytes(d) bytes, 256-byte aligned.  It is required
 * for every layer, but a layer with OC a multiple of 8 (at most 64) and Y 8-byte
 * aligned normally runs as one kernel that reads its taps straight from X and leaves
 * ws untouched; other layers unroll into ws first.  The results are identical.
 */
q4_status q4_conv2d(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                    const int32_t* colsum_w, const int32_t* bias,
                    const q4_conv_desc* d, int32_t za, int32_t zb, const q4_requant* rq,
                    uint8_t* Y, void* ws, size_t ws_bytes, void* stream);

/*
 * Convolution layers with the weight-side work done once (Section II-B: what depends only
 * on the weights -- here their zero-point-corrected, tile-ordered copy and the per-channel
 * constants of Eq. 3 -- "can be computed only once").  For the layer classes that run on
 * the tensor-memory kernels, q4_conv2d_prepare_weights writes that copy (an opaque image,
 * valid for this descriptor, za, zb, bias and this build of the library) into `prepared`,
 * and q4_conv2d_prepared runs the layer from it: the same arithmetic and the same output
 * bytes as q4_conv2d, without the per-launch weight preparation inside the kernel (3 to 5
 * thousand clocks per CTA).
 *
 * q4_conv2d_weights_bytes: bytes of the image for the layer, 0 if the layer's geometry has no
 * such kernel (then use q4_conv2d).  Host call, no device access.
 * q4_conv2d_prepare_weights: Wt, ldw, colsum_w (optional), bias (optional), za, zb as in
 * q4_conv2d; `prepared` a device buffer of at least q4_conv2d_weights_bytes(d) bytes, 16-byte
 * aligned, owned by the caller, written by one small kernel on `stream`.
 * q4_conv2d_prepared: X, Y, rq, za as in q4_conv2d (za must be the one the image was
 * prepared with); needs no workspace.
 * An image does not depend on the batch, the image size, the vertical stride or the
 * paddings: one image serves every descriptor that differs in those only.  It carries a tag
 * of what it does depend on besides the weights (kernel, filter, channel counts, horizontal
 * stride, za, image format); q4_conv2d_prepared given an image with another tag writes
 * nothing to Y, and the next q4_last_device_status on the device returns Q4_ERR_WEIGHT_IMAGE.
 * Errors: as q4_conv2d; Q4_ERR_UNSUPPORTED when the layer (or the alignment of X / Y: 16
 * bytes) has no tensor-memory kernel, Q4_ERR_WORKSPACE when prepared_bytes is too small,
 * Q4_ERR_ALIGNMENT when `prepared` is not 16-byte aligned.  Nothing is launched on error.
 */
size_t q4_conv2d_weights_bytes(const q4_conv_desc* d);
q4_status q4_conv2d_prepare_weights(const uint8_t* Wt, int64_t ldw, const int32_t* colsum_w,
                                    const int32_t* bias, const q4_conv_desc* d, int32_t za, int32_t zb,
                                    void* prepared, size_t prepared_bytes, void* stream);
q4_status q4_conv2d_prepared(const uint8_t* X, const void* prepared, size_t prepared_bytes,
                             const q4_conv_desc* d, int32_t za, const q4_requant* rq, uint8_t* Y,
                             void* stream);

/*
 * q4_conv2d for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of q4_conv2d, same arithmetic, same
 * kernels, same results.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a
 * latency-critical loop whose owner forbids allocator calls, in a plugin that is
 * handed device pointers by a host application but owns no allocator, or in a
 * process whose memory pool is fixed at start-up.  Such a caller cannot provide the
 * workspace q4_conv2d asks for, so this entry point brings its own: the unrolled
 * activation matrix and its row sums live in a fixed array compiled into the
 * library (static __device__ storage, Q4_STATIC_SCRATCH_BYTES bytes), which every
 * GPU that loads the library holds from load until the process exits.  The caller
 * still passes X, Wt, the optional sums / bias, and Y.  Nothing is allocated or
 * freed here: no cudaMalloc, no cudaFree, no allocating library routine.
 *
 * Limit: q4_conv2d_workspace_bytes(d) must not exceed Q4_STATIC_SCRATCH_BYTES;
 * a larger layer is rejected with Q4_ERR_STATIC_SCRATCH before anything is launched
 * (split the batch, or use q4_conv2d with your own workspace).
 *
 * First call on a device: the array's device address is looked up once per device
 * (with that device current) on the first call; make that first call outside any
 * stream capture.
 *
 * Sharing: there is ONE array per device.  Every call overwrites it and finds the
 * previous call's contents in it; the parts that must start from zero are cleared
 * by the call itself.  Two calls that overlap on the GPU (different streams, or
 * different host threads) race on the array -- serialize them.
 */
#define Q4_STATIC_SCRATCH_BYTES (8u << 20)
q4_status q4_conv2d_static(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                           const int32_t* colsum_w, const int32_t* bias,
                           const q4_conv_desc* d, int32_t za, int32_t zb, const q4_requant* rq,
                           uint8_t* Y, void* stream);

size_t q4_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K);
size_t q4_conv2d_workspace_bytes(const q4_conv_desc* d);

/*
 * Weight preparation, done once per weight matrix (Section II-B): a K x N matrix
 * packed along n (row k, pitch ldb_kn bytes) is rewritten as Bt, N x K packed along
 * k (pitch ldb bytes, pad nibbles 0).
 */
q4_status q4_pack_bt(const uint8_t* B_kn, int64_t ldb_kn, uint8_t* Bt, int64_t ldb,
                     int32_t K, int32_t N, void* stream);

/* Sums over the depth of a packed matrix: sums[r] = sum_k P[r][k] (the sums of
 * Eq. 2's second and third terms), for callers that want them precomputed. */
q4_status q4_row_sums(const uint8_t* P, int64_t ld, int32_t rows, int32_t K,
                      int32_t* sums, void* stream);

/*
 * Per-output-channel weight quantization: an extension of the paper's scheme, which has one
 * scale and one zero point per weight matrix (Section II-A, III-B).  Eq. 2 holds column by
 * column, and a column's zero point enters only through a rank-one term, so the product is
 * taken once with zb = 0 and finished here:
 *   C0 = q4_gemm(A, Bt, za, zb = 0)            (int32, M x N, pitch ldc elements)
 *   acc[m][n] = C0[m][n] - zb[n] * (rowsum_a[m] - K * za) + bias[n]
 *   y[m][n]   = clamp(floor((acc * mult[n] + 2^(30 + shift[n])) / 2^(31 + shift[n])) + zo, lo, hi)
 * written packed two per byte to Cq (pitch ldcq bytes >= N / 2; N even).  rowsum_a[m] =
 * sum_k A[m][k] (q4_row_sums, or q4_im2col's side output).  zb (values 0..15) and bias may be
 * NULL (= 0); mult[n] in [2^30, 2^31) and shift[n] in 0..31 are required; all are DEVICE
 * arrays of N int32 and are not range-checked.  zo, clamp_lo, clamp_hi as in q4_requant.
 */
q4_status q4_requant_channels(const int32_t* C0, int64_t ldc, int32_t M, int32_t N, int32_t K,
                              int32_t za, const int32_t* rowsum_a,
                              const int32_t* zb, const int32_t* bias,
                              const int32_t* mult, const int32_t* shift,
                              int32_t zo, int32_t clamp_lo, int32_t clamp_hi,
                              uint8_t* Cq, int64_t ldcq, void* stream);

/*
 * The product with per-output-channel weight quantization finished in the GEMM's own
 * epilogue (no int32 matrix in memory): same result as q4_gemm with zb = 0 followed by
 * q4_requant_channels,
 *   acc[m][n] = sum_k (A[m][k] - za)(B[k][n] - zb[n]) + bias[n]
 *   y[m][n]   = clamp(floor((acc * mult[n] + 2^(30 + shift[n])) / 2^(31 + shift[n])) + zo, lo, hi)
 * packed two per byte to Cq.  Extension of the paper's per-matrix scheme (Section II-A; Eq. 2
 * applied column by column).  A, Bt, rowsum_a, colsum_b, ws as in q4_gemm_requant; zb (values
 * 0..15, NULL = all 0), bias (NULL = none), mult in [2^30, 2^31) and shift in 0..31 are DEVICE
 * arrays of N int32, not range-checked.  The per-channel epilogue exists in the tensor-core
 * kernels only: operands that break their alignment rules (16-byte aligned A, Bt, lda, ldb)
 * return Q4_ERR_ALIGNMENT -- use q4_gemm with zb = 0 and q4_requant_channels for those.
 */
q4_status q4_gemm_requant_channels(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                                   int32_t M, int32_t N, int32_t K, int32_t za, const int32_t* zb,
                                   const int32_t* rowsum_a, const int32_t* colsum_b,
                                   const int32_t* bias, const int32_t* mult, const int32_t* shift,
                                   int32_t zo, int32_t clamp_lo, int32_t clamp_hi,
                                   uint8_t* Cq, int64_t ldcq, void* ws, size_t ws_bytes, void* stream);

/*
 * A convolution layer with per-output-channel weight quantization, as ONE fused kernel (the
 * unrolled matrix is never written; no workspace): like q4_conv2d, but output channel n has
 * its own weight zero point zb[n] (0..15), multiplier mult[n] in [2^30, 2^31) and shift[n] in
 * 0..31 (DEVICE arrays of OC int32, not range-checked); colsum_w and bias may be NULL.
 * The layer runs on the tensor-memory kernels where they have an instance for it (the
 * 3x3 layer classes of the workloads; any layer with C and OC multiples of 32), else on the
 * warp-level fused kernels.  Layers neither takes (e.g. OC not a multiple of 8, or above 64
 * with C not a multiple of 32; Y not 8-byte aligned; too large for shared memory) return
 * Q4_ERR_UNSUPPORTED: run those as q4_im2col, q4_gemm with zb = 0 and q4_requant_channels.  Extension of the paper's per-matrix scheme
 * (Section II-A), see q4_requant_channels.
 */
q4_status q4_conv2d_channels(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                             const int32_t* colsum_w, const int32_t* bias, const q4_conv_desc* d,
                             int32_t za, const int32_t* zb, const int32_t* mult, const int32_t* shift,
                             int32_t zo, int32_t clamp_lo, int32_t clamp_hi, uint8_t* Y, void* stream);

/*
 * The 8-bit product of the paper's comparison (Section II-B: values in 0..255 with 32-bit
 * accumulators; the experiments of Section IV measure the 4-bit product against it):
 *   C[m][n] = sum_k (A[m][k] - za) * (Bt[n][k] - zb),  za, zb in 0..255,
 * evaluated as Eq. 2's four terms like q4_gemm.  A [M][lda] and Bt [N][ldb] hold one byte
 * per value, depth-contiguous; pitches in bytes.  Tensor-core path only: A, Bt 16-byte
 * aligned and lda, ldb multiples of 16 (Q4_ERR_ALIGNMENT otherwise); 1 <= K <= 33024 so that
 * 255 * 255 * K fits the 32-bit accumulator (Q4_ERR_RANGE).  rowsum_a / colsum_b as in
 * q4_gemm; when either is NULL the workspace must hold q4_gemm_u8_workspace_bytes(M, N)
 * bytes (Q4_ERR_WORKSPACE) and the sums are taken by a pre-pass.
 */
q4_status q4_gemm_u8(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                     int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
                     int32_t za, int32_t zb,
                     const int32_t* rowsum_a, const int32_t* colsum_b,
                     void* workspace, size_t workspace_bytes, void* stream);
size_t q4_gemm_u8_workspace_bytes(int32_t M, int32_t N);

/*
 * Float boundary of a quantized layer (Section II-A, Eq. 1; Section III-B, the F -> Q and
 * Q -> F cases; Eq. 4).  All floating-point steps are IEEE binary32, correctly rounded.
 *
 * Reading of Eq. 1 (its zero point is printed in real units while Eq. 2 uses it in steps of
 * the scale): scale = (max(max x, 0) - min(min x, 0)) / 15 (1 for an all-zero tensor);
 * zero = -floor(min(min x, 0) / scale) clamped to 0..15; code = clamp(floor(x / scale) +
 * zero, 0, 15); x ~= scale * (code - zero).  Inputs must be finite.
 */
typedef struct {
    float scale;     /* s of Eq. 1 */
    int32_t zero;    /* integer zero point, 0..15: the za / zb of q4_gemm */
} q4_qparams;

/* Derives *qp (DEVICE memory, 8 bytes, 4-byte aligned, owned by the caller) from the
 * rows x cols float matrix X (device, row pitch ldx ELEMENTS >= cols).  Asynchronous on
 * `stream`; the host reads *qp back (after synchronizing) to pass `zero` to q4_gemm. */
q4_status q4_quant_params(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                          q4_qparams* qp, void* stream);

/* Quantizes X with the parameters at qp (DEVICE pointer, e.g. from q4_quant_params or
 * uploaded by the caller for a calibrated layer) into packed codes Q: row pitch ldq BYTES
 * >= ceil(cols / 2), low nibble = even column, an odd row's last high nibble 0; bytes
 * between ceil(cols / 2) and ldq are left untouched. */
q4_status q4_quantize(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                      const q4_qparams* qp, uint8_t* Q, int64_t ldq, void* stream);

/* Eq. 4: R[r][c] = scale * C[r][c] (int32 -> float32 round-to-nearest-even, one
 * multiplication).  C: int32 results with zero point 0 (q4_gemm output), pitch ldc
 * elements; R: float, pitch ldr elements; scale = s_w * s_x, or the running product of
 * Section III-B, a host value. */
q4_status q4_dequantize(const int32_t* C, int64_t ldc, int32_t rows, int32_t cols, float scale,
                        float* R, int64_t ldr, void* stream);

/*
 * q4_gemm with HOST operands: copies A and Bt to the device, runs q4_gemm and
 * copies C back, then synchronizes `stream`.  The work is ordered behind `stream`
 * and goes in row slices over `stream` and one stream of the library's own (created
 * on first use, one per device), so that a slice's copy back overlaps the next
 * slice's upload and product; when the call returns all of it is complete.  hA /
 * hBt / hC are host pointers with the same pitches as above (pinned memory makes
 * the copies asynchronous, and only then do they overlap).  dev_staging is a DEVICE
 * buffer owned by the caller of at least q4_gemm_host_staging_bytes(...) bytes,
 * 256-byte aligned; it holds the device copies and the column sums of Bt, so this
 * entry point allocates no device memory either.
 */
q4_status q4_gemm_host(const uint8_t* hA, int64_t lda, const uint8_t* hBt, int64_t ldb,
                       int32_t* hC, int64_t ldc, int32_t M, int32_t N, int32_t K,
                       int32_t za, int32_t zb,
                       void* dev_staging, size_t dev_staging_bytes, void* stream);
size_t q4_gemm_host_staging_bytes(int32_t M, int32_t N, int32_t K,
                                  int64_t lda, int64_t ldb, int64_t ldc);

/* Synchronizes `stream`, then returns Q4_ERR_DEVICE_TIMEOUT if any kernel of this
 * library gave up a bounded wait on the current device since the last call,
 * Q4_ERR_WEIGHT_IMAGE if q4_conv2d_prepared refused a weight image (the flags are cleared),
 * Q4_ERR_CUDA if the stream reports an error, else Q4_OK. */
q4_status q4_last_device_status(void* stream);

/*
 * Diagnostic (no counterpart in the paper): launches one small kernel that waits, with the
 * short limit of this library's bounded waits (about a millisecond), on a barrier nothing
 * arrives on.  The wait gives up, the kernel ends normally, and the next
 * q4_last_device_status on the device returns Q4_ERR_DEVICE_TIMEOUT once.  outcome_dev
 * (device int, may be NULL) receives 2 when the wait ran out and 1 if it completed.
 */
q4_status q4_selftest_wait_timeout(int* outcome_dev, void* stream);

/* Kernel selection for ablations and tests: 0 = automatic, 1 = general (SIMT)
 * kernels only, 2 = tensor-core kernels or an error where their alignment rules do
 * not hold, 3 = like 2 but never the CTA-pair kernel, 4 = automatic except that
 * convolution layers skip the tensor-memory (tcgen05) fused kernel and take the warp-level
 * fused kernels, 5 / 6 = like 2 with the CTA-pair GEMM kernel's tile width fixed at 192 / 256
 * columns (it is otherwise chosen from the problem's shape).  Returns the previous value.
 * Process-wide; also read once from the environment variable Q4_FORCE_VARIANT ("simt" / "tc" /
 * "tc1" / "fused1" / "tc192" / "tc256"). */
int q4_set_variant(int variant);
/* With Q4_LOG=1 in the environment every GEMM / convolution call prints one line to stderr
 * naming the kernel it was given. */

/*
 * Measurement helper (no counterpart in the paper): the tensor pipe's issue peak on
 * this device.  Launches num_ctas CTAs (one per SM is the intended use); each issues
 * 4 * iters back-to-back tcgen05.mma instructions of shape 128 x n x (32 bytes of
 * depth) on zero operands resident in shared memory and writes the elapsed SM clocks
 * to cycles_dev[cta] (device pointer, num_ctas entries).  kind: 0 = kind::i8
 * (u8 x u8 -> s32), 1 = kind::f16 (bf16 -> f32), 2 = kind::f8f6f4 (e4m3 -> f32),
 * 3 = kind::i8 issued by CTA pairs (cta_group::2, 256 x n per instruction; num_ctas
 * even, n a multiple of 32, one cycles_dev entry per pair, count 256 rows).
 * n: multiple of 16 in 16..256.  Multiply-accumulates per clock per SM =
 * 4 * iters * 128 * n * k / cycles, k = 32 for the 8-bit kinds and 16 for bf16.
 */
q4_status q4_measure_mma_peak(int kind, int n, int iters, unsigned long long* cycles_dev,
                              int num_ctas, void* stream);

/* Number of kernels this library has launched in this process (all streams). */
uint64_t q4_launch_count(void);

const char* q4_status_string(q4_status s);
int q4_version(void);

#ifdef __cplusplus
}
#endif
#endif
