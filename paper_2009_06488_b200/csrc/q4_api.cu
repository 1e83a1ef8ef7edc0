// C ABI of the q4 library (declared in q4.h): argument validation, kernel selection,
// launch.  No allocation, no synchronization except where the header says so.
#include <mutex>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "q4_common.cuh"

namespace q4 {

__device__ unsigned g_status_word = 0;

static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_variant{-1};   // -1 = not read from the environment yet

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// Q4_LOG=1 in the environment: one line on stderr per call saying which kernel it was given.
void log_choice(const char* call, const char* kernel)
{
    static int on = -1;
    if (on < 0) {
        const char* e = std::getenv("Q4_LOG");
        on = (e && e[0] == '1') ? 1 : 0;
    }
    if (on) std::fprintf(stderr, "[q4] %s -> %s\n", call, kernel);
}

static int variant()
{
    int v = g_variant.load(std::memory_order_relaxed);
    if (v < 0) {
        const char* e = std::getenv("Q4_FORCE_VARIANT");
        v = 0;
        if (e && !std::strcmp(e, "simt")) v = 1;
        if (e && !std::strcmp(e, "tc")) v = 2;
        if (e && !std::strcmp(e, "tc1")) v = 3;
        if (e && !std::strcmp(e, "fused1")) v = 4;
        if (e && !std::strcmp(e, "tc192")) v = 5;
        if (e && !std::strcmp(e, "tc256")) v = 6;
        g_variant.store(v, std::memory_order_relaxed);
    }
    return v;
}

// Variants 5 and 6 are variant 2 with the CTA-pair kernel's tile width fixed.
static int variant_kind() { const int v = variant(); return v >= 5 ? 2 : v; }
static int forced_pair_width() { const int v = variant(); return v == 5 ? 192 : v == 6 ? 256 : 0; }

static unsigned* status_ptr()
{
    // one address per device; looked up on first use with that device current
    static unsigned* ptrs[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        ptrs[dev] = static_cast<unsigned*>(p);
    }
    return ptrs[dev];
}

unsigned* device_status_ptr() { return status_ptr(); }

static q4_status check_gemm(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                            int32_t M, int32_t N, int32_t K, int32_t za, int32_t zb)
{
    if (M < 0 || N < 0 || K < 1) return Q4_ERR_INVALID_ARG;
    if (K > Q4_MAX_K) return Q4_ERR_RANGE;
    if ((M > 0 && !A) || (N > 0 && !Bt)) return Q4_ERR_INVALID_ARG;
    const int64_t kbytes = (K + 1) / 2;
    if (lda < kbytes || ldb < kbytes) return Q4_ERR_INVALID_ARG;
    if (za < 0 || za > 15 || zb < 0 || zb > 15) return Q4_ERR_RANGE;
    return Q4_OK;
}

static q4_status check_requant(const q4_requant* rq)
{
    if (!rq) return Q4_ERR_INVALID_ARG;
    if (rq->mult < (1 << 30)) return Q4_ERR_RANGE;
    if (rq->shift < 0 || rq->shift > 31) return Q4_ERR_RANGE;
    if (rq->zo < 0 || rq->zo > 15) return Q4_ERR_RANGE;
    if (rq->clamp_lo < 0 || rq->clamp_hi > 15 || rq->clamp_lo > rq->clamp_hi) return Q4_ERR_RANGE;
    return Q4_OK;
}

static size_t round256(size_t b) { return (b + 255) / 256 * 256; }

static q4_status run_gemm(GemmParams& p, bool rq, cudaStream_t st, void* ws = nullptr,
                          size_t ws_bytes = 0)
{
    p.status = status_ptr();
    if (!p.status) return Q4_ERR_CUDA;
    const int v = variant_kind();
    // The CTA-pair kernel pays off from about 64 of its 256 x 256 tiles (2048^3 is one wave of
    // 64: 12.1 us against 18.7 us), or from 32 where the depth is long enough to carry its
    // fixed costs -- prologue, pipeline fill, a last tile of 256 x 256 to drain; below that the
    // single-CTA kernel, with narrower tiles and its sums taken in the kernel, finishes sooner
    // (1024^3: 6.5 against 8.7 us; 1536^3, 36 tiles: 9.4 against 10.5 us; 8192 x 256 x 1024, 32
    // tiles: 7.8 against 9.3 us).  Variant 2 always takes the pair kernel where it applies.
    const long long pair_tiles = ((long long)p.M + 255) / 256 * (((long long)p.N + 255) / 256);
    const bool pair_pays = pair_tiles >= 64 || (pair_tiles >= 32 && p.K >= 2048);
    if (v != 1 && v != 3 && gemm_tc_pair_supported(p) && (v == 2 || pair_pays)) {
        // Large problems use the workspace, if given, for the depth sums where one pass over
        // an operand is cheaper than every output tile taking them again; without one the
        // kernel does everything itself.  The results are identical.
        // Layout of the workspace: [row sums of A][column sums of Bt].
        const size_t sums_bytes = round256(4 * (size_t)p.M) + round256(4 * (size_t)p.N);
        const bool ws_ok = ws && (uintptr_t)ws % 16 == 0;
        int32_t* wa = static_cast<int32_t*>(ws);
        int32_t* wb = ws ? reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + round256(4 * (size_t)p.M))
                         : nullptr;
        // The sums pre-pass is a launch of its own (about 3 us plus its pass over the operands).
        // Row sums alone the kernel takes as cheaply itself (they stay inside a CTA: 4096^3 51.7
        // against 54.4 us with the pre-pass, 8192^3 306 against 305 us); column sums need an
        // exchange between the CTAs of a pair, and from about 1e11 operations the pre-pass is
        // cheaper than that (8192^3: 305 against 320 us); below, the kernel takes both.
        const bool prepass_pays = !p.colsum_b && 2.0 * p.M * p.N * p.K >= 1e11;
        if ((!p.rowsum_a || !p.colsum_b) && ws_ok && ws_bytes >= sums_bytes && prepass_pays) {
            const bool do_a = !p.rowsum_a, do_b = !p.colsum_b;
            if (launch_operand_sums(p.A, p.lda, do_a ? p.M : 0, wa, p.Bt, p.ldb, do_b ? p.N : 0, wb,
                                    p.K, st) != cudaSuccess) return Q4_ERR_CUDA;
            if (do_a) p.rowsum_a = wa;
            if (do_b) p.colsum_b = wb;
        }
        log_choice(rq ? "q4_gemm_requant" : "q4_gemm", "CTA-pair tcgen05 kernel");
        return launch_gemm_tc_pair(p, rq, st, forced_pair_width());
    }
    if (v != 1 && gemm_tc_supported(p)) {
        log_choice(rq ? "q4_gemm_requant" : "q4_gemm", "single-CTA tcgen05 kernel");
        return launch_gemm_tc(p, rq, st);
    }
    if (v == 2 || v == 3) return Q4_ERR_ALIGNMENT;
    log_choice(rq ? "q4_gemm_requant" : "q4_gemm", "general kernel (operands not aligned for TMA)");
    return launch_gemm_simt(p, rq, st) == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

static q4_status check_conv(const q4_conv_desc* d, int32_t za)
{
    if (!d) return Q4_ERR_INVALID_ARG;
    if (d->N < 0 || d->H < 1 || d->W < 1 || d->C < 1) return Q4_ERR_INVALID_ARG;
    if (d->KH < 1 || d->KW < 1) return Q4_ERR_INVALID_ARG;
    if (d->stride_h < 1 || d->stride_w < 1 || d->pad_h < 0 || d->pad_w < 0) return Q4_ERR_INVALID_ARG;
    if (d->H + 2 * d->pad_h < d->KH || d->W + 2 * d->pad_w < d->KW) return Q4_ERR_INVALID_ARG;
    const int64_t K = (int64_t)d->KH * d->KW * d->C;
    if (K > Q4_MAX_K) return Q4_ERR_RANGE;
    const int64_t OH = (d->H + 2 * d->pad_h - d->KH) / d->stride_h + 1;
    const int64_t OW = (d->W + 2 * d->pad_w - d->KW) / d->stride_w + 1;
    if ((int64_t)d->N * OH * OW > INT32_MAX) return Q4_ERR_RANGE;
    if (za < 0 || za > 15) return Q4_ERR_RANGE;
    return Q4_OK;
}

struct ConvShape { int64_t M; int32_t K; int64_t lda; size_t off_rowsum, bytes; };

// Workspace of q4_conv2d: the unrolled matrix (pitch rounded up to 16 bytes so the
// tensor-core path applies) followed by its row sums.
static ConvShape conv_shape(const q4_conv_desc* d)
{
    ConvShape s;
    const int64_t OH = (d->H + 2 * d->pad_h - d->KH) / d->stride_h + 1;
    const int64_t OW = (d->W + 2 * d->pad_w - d->KW) / d->stride_w + 1;
    s.M = (int64_t)d->N * OH * OW;
    s.K = d->KH * d->KW * d->C;
    s.lda = (((int64_t)s.K + 1) / 2 + 15) / 16 * 16;
    s.off_rowsum = ((size_t)(s.M * s.lda) + 255) / 256 * 256;
    s.bytes = s.off_rowsum + ((size_t)s.M * 4 + 255) / 256 * 256;
    return s;
}

// Scratch of q4_conv2d_static: one fixed array per device, held from library load to
// process exit.  In host code this name is only a handle for cudaGetSymbolAddress,
// never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[Q4_STATIC_SCRATCH_BYTES];

// Device address of the static scratch on the current device (looked up once per
// device, with that device current); nullptr if the lookup fails.
static void* static_scratch_ptr()
{
    static void* ptrs[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) return nullptr;
        ptrs[dev] = p;
    }
    return ptrs[dev];
}

}  // namespace q4

using namespace q4;

extern "C" {

q4_status q4_gemm(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                  int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
                  int32_t za, int32_t zb, const int32_t* rowsum_a, const int32_t* colsum_b,
                  void* ws, size_t ws_bytes, void* stream)
{
    q4_status s = check_gemm(A, lda, Bt, ldb, M, N, K, za, zb);
    if (s != Q4_OK) return s;
    if (M == 0 || N == 0) return Q4_OK;
    if (!C || ldc < N) return Q4_ERR_INVALID_ARG;
    if ((uintptr_t)C % 4 != 0) return Q4_ERR_ALIGNMENT;
    GemmParams p{};
    p.A = A; p.Bt = Bt; p.lda = lda; p.ldb = ldb; p.M = M; p.N = N; p.K = K; p.za = za; p.zb = zb;
    p.rowsum_a = rowsum_a; p.colsum_b = colsum_b; p.C = C; p.ldc = ldc;
    return run_gemm(p, false, static_cast<cudaStream_t>(stream), ws, ws_bytes);
}

q4_status q4_gemm_requant(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                          int32_t M, int32_t N, int32_t K, int32_t za, int32_t zb,
                          const int32_t* rowsum_a, const int32_t* colsum_b,
                          const int32_t* bias, const q4_requant* rq,
                          uint8_t* Cq, int64_t ldcq, void* ws, size_t ws_bytes, void* stream)
{
    q4_status s = check_gemm(A, lda, Bt, ldb, M, N, K, za, zb);
    if (s != Q4_OK) return s;
    if ((s = check_requant(rq)) != Q4_OK) return s;
    if (N & 1) return Q4_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return Q4_OK;
    if (!Cq || ldcq < N / 2) return Q4_ERR_INVALID_ARG;
    GemmParams p{};
    p.A = A; p.Bt = Bt; p.lda = lda; p.ldb = ldb; p.M = M; p.N = N; p.K = K; p.za = za; p.zb = zb;
    p.rowsum_a = rowsum_a; p.colsum_b = colsum_b; p.bias = bias; p.Cq = Cq; p.ldcq = ldcq;
    p.rq = RequantParams{rq->mult, rq->shift, rq->zo, rq->clamp_lo, rq->clamp_hi};
    return run_gemm(p, true, static_cast<cudaStream_t>(stream), ws, ws_bytes);
}

q4_status q4_gemm_requant_channels(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                                   int32_t M, int32_t N, int32_t K, int32_t za, const int32_t* zb,
                                   const int32_t* rowsum_a, const int32_t* colsum_b,
                                   const int32_t* bias, const int32_t* mult, const int32_t* shift,
                                   int32_t zo, int32_t clamp_lo, int32_t clamp_hi,
                                   uint8_t* Cq, int64_t ldcq, void* ws, size_t ws_bytes, void* stream)
{
    q4_status s = check_gemm(A, lda, Bt, ldb, M, N, K, za, 0);
    if (s != Q4_OK) return s;
    if (zo < 0 || zo > 15 || clamp_lo < 0 || clamp_hi > 15 || clamp_lo > clamp_hi) return Q4_ERR_RANGE;
    if (N & 1) return Q4_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return Q4_OK;
    if (!Cq || ldcq < N / 2 || !mult || !shift) return Q4_ERR_INVALID_ARG;
    const void* words[] = {zb, rowsum_a, colsum_b, bias, mult, shift};
    for (const void* w : words)
        if ((uintptr_t)w % 4) return Q4_ERR_ALIGNMENT;
    GemmParams p{};
    p.A = A; p.Bt = Bt; p.lda = lda; p.ldb = ldb; p.M = M; p.N = N; p.K = K; p.za = za; p.zb = 0;
    p.rowsum_a = rowsum_a; p.colsum_b = colsum_b; p.bias = bias; p.Cq = Cq; p.ldcq = ldcq;
    p.rq = RequantParams{1 << 30, 2, zo, clamp_lo, clamp_hi};      // multiplier and shift come per channel
    p.zb_ch = zb; p.mult_ch = mult; p.shift_ch = shift;
    // the per-channel epilogue lives in the tensor-core kernels
    if (variant_kind() == 1) return Q4_ERR_UNSUPPORTED;
    if (!gemm_tc_supported(p)) return Q4_ERR_ALIGNMENT;
    return run_gemm(p, true, static_cast<cudaStream_t>(stream), ws, ws_bytes);
}

q4_status q4_im2col(const uint8_t* X, const q4_conv_desc* d, int32_t za,
                    uint8_t* A, int64_t lda, int32_t* rowsum_a, void* stream)
{
    q4_status s = check_conv(d, za);
    if (s != Q4_OK) return s;
    const ConvShape cs = conv_shape(d);
    if (lda < ((int64_t)cs.K + 1) / 2) return Q4_ERR_INVALID_ARG;
    if (cs.M == 0) return Q4_OK;
    if (!X || !A) return Q4_ERR_INVALID_ARG;
    if (rowsum_a && (uintptr_t)rowsum_a % 4 != 0) return Q4_ERR_ALIGNMENT;
    return launch_im2col(X, *d, za, A, lda, rowsum_a, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

size_t q4_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K)
{
    (void)K;
    if (M < 0 || N < 0) return 0;
    return round256(4 * (size_t)M) + round256(4 * (size_t)N);   // depth sums of both operands
}

size_t q4_conv2d_workspace_bytes(const q4_conv_desc* d)
{
    if (check_conv(d, 0) != Q4_OK) return 0;
    return conv_shape(d).bytes;
}

q4_status q4_conv2d(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                    const int32_t* colsum_w, const int32_t* bias,
                    const q4_conv_desc* d, int32_t za, int32_t zb, const q4_requant* rq,
                    uint8_t* Y, void* ws, size_t ws_bytes, void* stream)
{
    q4_status s = check_conv(d, za);
    if (s != Q4_OK) return s;
    if ((s = check_requant(rq)) != Q4_OK) return s;
    if (zb < 0 || zb > 15) return Q4_ERR_RANGE;
    if (d->OC < 0 || (d->OC & 1)) return Q4_ERR_INVALID_ARG;
    const ConvShape cs = conv_shape(d);
    if (ldw < ((int64_t)cs.K + 1) / 2) return Q4_ERR_INVALID_ARG;
    if (cs.M == 0 || d->OC == 0) return Q4_OK;
    if (!X || !Wt || !Y) return Q4_ERR_INVALID_ARG;
    if (!ws || ws_bytes < cs.bytes) return Q4_ERR_WORKSPACE;
    if ((uintptr_t)ws % 256 != 0) return Q4_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // Layers whose geometry allows it run as one fused kernel that never writes the
    // unrolled matrix (variants 1 and 3 keep the explicit unroll + GEMM path testable):
    // on the tensor-memory path where it has an instance for the layer (variant 4 skips
    // it), else on the warp-level kernels.
    const int v = variant_kind();
    if ((v == 0 || v == 2) && conv_tc_supported(*d, X, Wt, ldw, Y)) {
        const RequantParams rqp{rq->mult, rq->shift, rq->zo, rq->clamp_lo, rq->clamp_hi};
        return launch_conv_tc(X, Wt, ldw, colsum_w, bias, *d, za, zb, rqp, Y, st) == cudaSuccess
                   ? Q4_OK : Q4_ERR_CUDA;
    }
    if ((v == 0 || v == 2 || v == 4) && conv_fused_supported(*d, X, Wt, ldw, Y)) {
        const RequantParams rqp{rq->mult, rq->shift, rq->zo, rq->clamp_lo, rq->clamp_hi};
        return launch_conv_fused(X, Wt, ldw, colsum_w, bias, *d, za, zb, rqp, Y, st) == cudaSuccess
                   ? Q4_OK : Q4_ERR_CUDA;
    }

    GemmParams p{};
    // A layer whose unrolled matrix is the input itself -- a filter as large as the
    // unpadded image (a fully connected layer), or a 1x1 filter with stride 1 -- goes
    // straight to the GEMM; the workspace then only holds the depth sums.
    const bool whole_image = d->KH == d->H && d->KW == d->W;
    const bool pointwise = d->KH == 1 && d->KW == 1 && d->stride_h == 1 && d->stride_w == 1;
    if ((v == 0 || v == 4) && d->pad_h == 0 && d->pad_w == 0 && (whole_image || pointwise) &&
        cs.K % 2 == 0) {
        p.A = X; p.Bt = Wt; p.lda = cs.K / 2; p.ldb = ldw; p.M = (int32_t)cs.M; p.N = d->OC; p.K = cs.K;
        p.za = za; p.zb = zb; p.rowsum_a = nullptr; p.colsum_b = colsum_w; p.bias = bias;
        p.Cq = Y; p.ldcq = d->OC / 2;
        p.rq = RequantParams{rq->mult, rq->shift, rq->zo, rq->clamp_lo, rq->clamp_hi};
        return run_gemm(p, true, st, ws, ws_bytes);
    }

    log_choice("q4_conv2d", "explicit path: unroll into the workspace, then GEMM");
    uint8_t* A = static_cast<uint8_t*>(ws);
    int32_t* rowsum = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + cs.off_rowsum);
    if (launch_im2col(X, *d, za, A, cs.lda, rowsum, st) != cudaSuccess) return Q4_ERR_CUDA;

    p.A = A; p.Bt = Wt; p.lda = cs.lda; p.ldb = ldw; p.M = (int32_t)cs.M; p.N = d->OC; p.K = cs.K;
    p.za = za; p.zb = zb; p.rowsum_a = rowsum; p.colsum_b = colsum_w; p.bias = bias;
    p.Cq = Y; p.ldcq = d->OC / 2;
    p.rq = RequantParams{rq->mult, rq->shift, rq->zo, rq->clamp_lo, rq->clamp_hi};
    return run_gemm(p, true, st);
}

size_t q4_conv2d_weights_bytes(const q4_conv_desc* d)
{
    if (!d || check_conv(d, 0) != Q4_OK || d->OC <= 0 || (d->OC & 1)) return 0;
    return conv_tc_image_bytes(*d);
}

q4_status q4_conv2d_prepare_weights(const uint8_t* Wt, int64_t ldw, const int32_t* colsum_w,
                                    const int32_t* bias, const q4_conv_desc* d, int32_t za, int32_t zb,
                                    void* prepared, size_t prepared_bytes, void* stream)
{
    q4_status s = check_conv(d, za);
    if (s != Q4_OK) return s;
    if (zb < 0 || zb > 15) return Q4_ERR_RANGE;
    if (d->OC <= 0 || (d->OC & 1)) return Q4_ERR_INVALID_ARG;
    const ConvShape cs = conv_shape(d);
    if (ldw < ((int64_t)cs.K + 1) / 2) return Q4_ERR_INVALID_ARG;
    if (!Wt || !prepared) return Q4_ERR_INVALID_ARG;
    const size_t need = conv_tc_image_bytes(*d);
    if (need == 0) return Q4_ERR_UNSUPPORTED;
    if (prepared_bytes < need) return Q4_ERR_WORKSPACE;
    if ((uintptr_t)prepared % 16 != 0) return Q4_ERR_ALIGNMENT;
    const RequantParams rqp{1 << 30, 0, 0, 0, 15};       // not used by the preparation
    return launch_conv_tc(nullptr, Wt, ldw, colsum_w, bias, *d, za, zb, rqp, nullptr,
                          static_cast<cudaStream_t>(stream), nullptr, static_cast<uint8_t*>(prepared)) == cudaSuccess
               ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_conv2d_prepared(const uint8_t* X, const void* prepared, size_t prepared_bytes,
                             const q4_conv_desc* d, int32_t za, const q4_requant* rq, uint8_t* Y,
                             void* stream)
{
    q4_status s = check_conv(d, za);
    if (s != Q4_OK) return s;
    if ((s = check_requant(rq)) != Q4_OK) return s;
    if (d->OC <= 0 || (d->OC & 1)) return Q4_ERR_INVALID_ARG;
    if (!prepared) return Q4_ERR_INVALID_ARG;
    const size_t need = conv_tc_image_bytes(*d);
    if (need == 0) return Q4_ERR_UNSUPPORTED;
    if (prepared_bytes < need) return Q4_ERR_WORKSPACE;
    if ((uintptr_t)prepared % 16 != 0) return Q4_ERR_ALIGNMENT;
    const ConvShape cs = conv_shape(d);
    if (cs.M == 0) return Q4_OK;
    if (!X || !Y) return Q4_ERR_INVALID_ARG;
    const int v = variant_kind();
    if ((v != 0 && v != 2) || !conv_tc_supported(*d, X, nullptr, 0, Y)) return Q4_ERR_UNSUPPORTED;
    const RequantParams rqp{rq->mult, rq->shift, rq->zo, rq->clamp_lo, rq->clamp_hi};
    return launch_conv_tc(X, nullptr, 0, nullptr, nullptr, *d, za, 0, rqp, Y, static_cast<cudaStream_t>(stream),
                          static_cast<const uint8_t*>(prepared), nullptr) == cudaSuccess
               ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_conv2d_static(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                           const int32_t* colsum_w, const int32_t* bias,
                           const q4_conv_desc* d, int32_t za, int32_t zb, const q4_requant* rq,
                           uint8_t* Y, void* stream)
{
    // the same argument checks, in the same order, as q4_conv2d
    q4_status s = check_conv(d, za);
    if (s != Q4_OK) return s;
    if ((s = check_requant(rq)) != Q4_OK) return s;
    if (zb < 0 || zb > 15) return Q4_ERR_RANGE;
    if (d->OC < 0 || (d->OC & 1)) return Q4_ERR_INVALID_ARG;
    const ConvShape cs = conv_shape(d);
    if (ldw < ((int64_t)cs.K + 1) / 2) return Q4_ERR_INVALID_ARG;
    if (cs.M == 0 || d->OC == 0) return Q4_OK;
    if (!X || !Wt || !Y) return Q4_ERR_INVALID_ARG;
    // the layer must fit the built-in array; nothing is launched otherwise
    if (cs.bytes > (size_t)Q4_STATIC_SCRATCH_BYTES) return Q4_ERR_STATIC_SCRATCH;
    void* scratch = static_scratch_ptr();
    if (!scratch) return Q4_ERR_CUDA;
    // q4_conv2d rewrites the whole unrolled matrix (pad nibbles included) and every row
    // sum (written directly, or zeroed before accumulation), so stale contents cannot leak
    // through
    return q4_conv2d(X, Wt, ldw, colsum_w, bias, d, za, zb, rq, Y, scratch,
                     (size_t)Q4_STATIC_SCRATCH_BYTES, stream);
}

size_t q4_gemm_u8_workspace_bytes(int32_t M, int32_t N)
{
    if (M < 0 || N < 0) return 0;
    return round256(4 * (size_t)M) + round256(4 * (size_t)N);   // depth sums of both operands
}

q4_status q4_gemm_u8(const uint8_t* A, int64_t lda, const uint8_t* Bt, int64_t ldb,
                     int32_t* C, int64_t ldc, int32_t M, int32_t N, int32_t K,
                     int32_t za, int32_t zb, const int32_t* rowsum_a, const int32_t* colsum_b,
                     void* ws, size_t ws_bytes, void* stream)
{
    if (M < 0 || N < 0 || K < 1 || lda < K || ldb < K) return Q4_ERR_INVALID_ARG;
    if (za < 0 || za > 255 || zb < 0 || zb > 255 || K > 33024) return Q4_ERR_RANGE;
    if (M == 0 || N == 0) return Q4_OK;
    if (!A || !Bt || !C || ldc < N) return Q4_ERR_INVALID_ARG;
    if ((uintptr_t)A % 16 || (uintptr_t)Bt % 16 || lda % 16 || ldb % 16 || (uintptr_t)C % 4)
        return Q4_ERR_ALIGNMENT;
    if ((rowsum_a && (uintptr_t)rowsum_a % 4) || (colsum_b && (uintptr_t)colsum_b % 4))
        return Q4_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GemmParams p{};
    p.A = A; p.Bt = Bt; p.lda = lda; p.ldb = ldb; p.M = M; p.N = N; p.K = K; p.za = za; p.zb = zb;
    p.rowsum_a = rowsum_a; p.colsum_b = colsum_b; p.C = C; p.ldc = ldc;
    if ((!rowsum_a || !colsum_b) &&
        (!ws || (uintptr_t)ws % 4 || ws_bytes < q4_gemm_u8_workspace_bytes(M, N)))
        return Q4_ERR_WORKSPACE;
    p.status = device_status_ptr();
    if (!p.status) return Q4_ERR_CUDA;
    if (!rowsum_a || !colsum_b) {
        int32_t* sa = static_cast<int32_t*>(ws);
        int32_t* sb = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + round256(4 * (size_t)M));
        if (launch_byte_sums(A, lda, rowsum_a ? 0 : M, sa, Bt, ldb, colsum_b ? 0 : N, sb, K, st) != cudaSuccess)
            return Q4_ERR_CUDA;
        if (!rowsum_a) p.rowsum_a = sa;
        if (!colsum_b) p.colsum_b = sb;
    }
    return launch_gemm_u8(p, st);
}

q4_status q4_quant_params(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                          q4_qparams* qp, void* stream)
{
    if (rows < 0 || cols < 0 || ldx < cols || !qp) return Q4_ERR_INVALID_ARG;
    if ((int64_t)rows * cols > 0 && !X) return Q4_ERR_INVALID_ARG;
    if ((uintptr_t)X % 4 || (uintptr_t)qp % 4) return Q4_ERR_ALIGNMENT;
    return launch_quant_params(X, ldx, rows, cols, qp, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_quantize(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                      const q4_qparams* qp, uint8_t* Q, int64_t ldq, void* stream)
{
    if (rows < 0 || cols < 0 || ldx < cols || ldq < (cols + 1) / 2 || !qp) return Q4_ERR_INVALID_ARG;
    if ((int64_t)rows * cols == 0) return Q4_OK;
    if (!X || !Q) return Q4_ERR_INVALID_ARG;
    if ((uintptr_t)X % 4 || (uintptr_t)qp % 4) return Q4_ERR_ALIGNMENT;
    return launch_quantize(X, ldx, rows, cols, qp, Q, ldq, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_dequantize(const int32_t* C, int64_t ldc, int32_t rows, int32_t cols, float scale,
                        float* R, int64_t ldr, void* stream)
{
    if (rows < 0 || cols < 0 || ldc < cols || ldr < cols) return Q4_ERR_INVALID_ARG;
    if ((int64_t)rows * cols == 0) return Q4_OK;
    if (!C || !R) return Q4_ERR_INVALID_ARG;
    if ((uintptr_t)C % 4 || (uintptr_t)R % 4) return Q4_ERR_ALIGNMENT;
    return launch_dequantize(C, ldc, rows, cols, scale, R, ldr, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_selftest_wait_timeout(int* outcome_dev, void* stream)
{
    if (outcome_dev && (uintptr_t)outcome_dev % 4) return Q4_ERR_ALIGNMENT;
    return launch_wait_selftest(outcome_dev, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_conv2d_channels(const uint8_t* X, const uint8_t* Wt, int64_t ldw,
                             const int32_t* colsum_w, const int32_t* bias, const q4_conv_desc* d,
                             int32_t za, const int32_t* zb, const int32_t* mult, const int32_t* shift,
                             int32_t zo, int32_t clamp_lo, int32_t clamp_hi, uint8_t* Y, void* stream)
{
    q4_status s = check_conv(d, za);
    if (s != Q4_OK) return s;
    if (zo < 0 || zo > 15 || clamp_lo < 0 || clamp_hi > 15 || clamp_lo > clamp_hi) return Q4_ERR_RANGE;
    if (d->OC < 0 || (d->OC & 1)) return Q4_ERR_INVALID_ARG;
    const ConvShape cs = conv_shape(d);
    if (ldw < ((int64_t)cs.K + 1) / 2) return Q4_ERR_INVALID_ARG;
    if (cs.M == 0 || d->OC == 0) return Q4_OK;
    if (!X || !Wt || !Y || !zb || !mult || !shift) return Q4_ERR_INVALID_ARG;
    const void* words[] = {colsum_w, bias, zb, mult, shift};
    for (const void* w : words)
        if ((uintptr_t)w % 4) return Q4_ERR_ALIGNMENT;
    const RequantParams rqp{1 << 30, 2, zo, clamp_lo, clamp_hi};     // multiplier and shift come per channel
    // the tensor-memory kernels where they have an instance for the layer (variant 4 skips them)
    const int v = variant_kind();
    if ((v == 0 || v == 2) && conv_tc_supported(*d, X, Wt, ldw, Y))
        return launch_conv_tc(X, Wt, ldw, colsum_w, bias, *d, za, 0, rqp, Y, static_cast<cudaStream_t>(stream),
                              nullptr, nullptr, zb, mult, shift) == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
    if (!conv_fused_supported(*d, X, Wt, ldw, Y, true)) return Q4_ERR_UNSUPPORTED;
    return launch_conv_fused(X, Wt, ldw, colsum_w, bias, *d, za, 0, rqp, Y, static_cast<cudaStream_t>(stream),
                             zb, mult, shift) == cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_requant_channels(const int32_t* C0, int64_t ldc, int32_t M, int32_t N, int32_t K,
                              int32_t za, const int32_t* rowsum_a,
                              const int32_t* zb, const int32_t* bias,
                              const int32_t* mult, const int32_t* shift,
                              int32_t zo, int32_t clamp_lo, int32_t clamp_hi,
                              uint8_t* Cq, int64_t ldcq, void* stream)
{
    if (M < 0 || N < 0 || (N & 1) || K < 1 || ldc < N || ldcq < N / 2) return Q4_ERR_INVALID_ARG;
    if (K > Q4_MAX_K || za < 0 || za > 15 || zo < 0 || zo > 15 || clamp_lo < 0 || clamp_hi > 15 ||
        clamp_lo > clamp_hi)
        return Q4_ERR_RANGE;
    if (M == 0 || N == 0) return Q4_OK;
    if (!C0 || !rowsum_a || !mult || !shift || !Cq) return Q4_ERR_INVALID_ARG;
    const void* words[] = {C0, rowsum_a, zb, bias, mult, shift};
    for (const void* w : words)
        if ((uintptr_t)w % 4) return Q4_ERR_ALIGNMENT;
    return launch_requant_channels(C0, ldc, M, N, K, za, rowsum_a, zb, bias, mult, shift, zo, clamp_lo,
                                   clamp_hi, Cq, ldcq, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_pack_bt(const uint8_t* B_kn, int64_t ldb_kn, uint8_t* Bt, int64_t ldb,
                     int32_t K, int32_t N, void* stream)
{
    if (K < 1 || N < 0 || ldb_kn < (N + 1) / 2 || ldb < (K + 1) / 2) return Q4_ERR_INVALID_ARG;
    if (N == 0) return Q4_OK;
    if (!B_kn || !Bt) return Q4_ERR_INVALID_ARG;
    return launch_pack_bt(B_kn, ldb_kn, Bt, ldb, K, N, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

q4_status q4_row_sums(const uint8_t* P, int64_t ld, int32_t rows, int32_t K,
                      int32_t* sums, void* stream)
{
    if (rows < 0 || K < 1 || ld < (K + 1) / 2) return Q4_ERR_INVALID_ARG;
    if (rows == 0) return Q4_OK;
    if (!P || !sums) return Q4_ERR_INVALID_ARG;
    return launch_row_sums(P, ld, rows, K, sums, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? Q4_OK : Q4_ERR_CUDA;
}

size_t q4_gemm_host_staging_bytes(int32_t M, int32_t N, int32_t K,
                                  int64_t lda, int64_t ldb, int64_t ldc)
{
    (void)K;
    if (M < 0 || N < 0 || lda < 0 || ldb < 0 || ldc < 0) return 0;
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    return up((size_t)M * (size_t)lda) + up((size_t)N * (size_t)ldb) + up((size_t)M * (size_t)ldc * 4) +
           up((size_t)N * 4);      // the column sums of Bt, taken once for all row slices
}

// A second stream and two events per device for q4_gemm_host, created on first use and
// kept for the life of the process.
struct HostPipe { cudaStream_t side = nullptr; cudaEvent_t weights = nullptr, done = nullptr; bool ok = false; };
static HostPipe* host_pipe()
{
    static HostPipe pipes[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    HostPipe& h = pipes[dev];
    if (!h.ok) {
        if (cudaStreamCreateWithFlags(&h.side, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&h.weights, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&h.done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        h.ok = true;
    }
    return &h;
}

q4_status q4_gemm_host(const uint8_t* hA, int64_t lda, const uint8_t* hBt, int64_t ldb,
                       int32_t* hC, int64_t ldc, int32_t M, int32_t N, int32_t K,
                       int32_t za, int32_t zb, void* dev_staging, size_t dev_staging_bytes,
                       void* stream)
{
    q4_status s = check_gemm(hA, lda, hBt, ldb, M, N, K, za, zb);
    if (s != Q4_OK) return s;
    if (M == 0 || N == 0) return Q4_OK;
    if (!hC || ldc < N) return Q4_ERR_INVALID_ARG;
    if (!dev_staging || dev_staging_bytes < q4_gemm_host_staging_bytes(M, N, K, lda, ldb, ldc))
        return Q4_ERR_WORKSPACE;
    if ((uintptr_t)dev_staging % 256 != 0) return Q4_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    uint8_t* dA = static_cast<uint8_t*>(dev_staging);
    uint8_t* dB = dA + up((size_t)M * lda);
    int32_t* dC = reinterpret_cast<int32_t*>(dB + up((size_t)N * ldb));
    int32_t* dcb = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(dC) + up((size_t)M * ldc * 4));
    // only the bytes the header promises to touch: ceil(K / 2) of every operand row, N
    // elements of every output row (pitch padding is neither read nor written)
    const size_t kbytes = ((size_t)K + 1) / 2;
    // The int32 result is eight times the bytes of a packed operand, so the call is bound by
    // the copy back.  Rows go in slices that alternate between two streams: a slice's
    // download overlaps the next slice's upload and product (the two directions have their
    // own copy engines).  Bt and its column sums are needed by every slice and go first.
    HostPipe* hp = host_pipe();
    if (!hp) return Q4_ERR_CUDA;
    if (cudaMemcpy2DAsync(dB, (size_t)ldb, hBt, (size_t)ldb, kbytes, (size_t)N, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return Q4_ERR_CUDA;
    if (launch_row_sums(dB, ldb, N, K, dcb, st) != cudaSuccess) return Q4_ERR_CUDA;
    if (cudaEventRecord(hp->weights, st) != cudaSuccess ||
        cudaStreamWaitEvent(hp->side, hp->weights, 0) != cudaSuccess) return Q4_ERR_CUDA;
    int32_t slice = (M / 8 + 255) / 256 * 256;        // about eight slices, whole tiles of 256 rows
    if (slice < 1024) slice = 1024;
    int k = 0;
    for (int32_t m0 = 0; m0 < M; m0 += slice, ++k) {
        const int32_t rows = M - m0 < slice ? M - m0 : slice;
        cudaStream_t sk = (k & 1) ? hp->side : st;
        if (cudaMemcpy2DAsync(dA + (size_t)m0 * lda, (size_t)lda, hA + (size_t)m0 * lda, (size_t)lda, kbytes,
                              (size_t)rows, cudaMemcpyHostToDevice, sk) != cudaSuccess) return Q4_ERR_CUDA;
        s = q4_gemm(dA + (size_t)m0 * lda, lda, dB, ldb, dC + (size_t)m0 * ldc, ldc, rows, N, K, za, zb, nullptr,
                    dcb, nullptr, 0, sk);
        if (s != Q4_OK) break;
        if (cudaMemcpy2DAsync(hC + (size_t)m0 * ldc, (size_t)ldc * 4, dC + (size_t)m0 * ldc, (size_t)ldc * 4,
                              (size_t)N * 4, (size_t)rows, cudaMemcpyDeviceToHost, sk) != cudaSuccess) {
            s = Q4_ERR_CUDA;
            break;
        }
    }
    // the caller's stream ends behind the side stream, whatever happened above
    if (cudaEventRecord(hp->done, hp->side) != cudaSuccess ||
        cudaStreamWaitEvent(st, hp->done, 0) != cudaSuccess) return Q4_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return Q4_ERR_CUDA;
    return s;
}

q4_status q4_last_device_status(void* stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return Q4_ERR_CUDA;
    unsigned* dptr = status_ptr();
    if (!dptr) return Q4_ERR_CUDA;
    unsigned word = 0;
    if (cudaMemcpy(&word, dptr, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return Q4_ERR_CUDA;
    if (word) {
        if (cudaMemset(dptr, 0, sizeof(word)) != cudaSuccess) return Q4_ERR_CUDA;
        return (word & kStatusTimeout) ? Q4_ERR_DEVICE_TIMEOUT : Q4_ERR_WEIGHT_IMAGE;
    }
    return Q4_OK;
}

int q4_set_variant(int v)
{
    const int prev = variant();
    g_variant.store((v >= 1 && v <= 6) ? v : 0, std::memory_order_relaxed);
    return prev;
}

uint64_t q4_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* q4_status_string(q4_status s)
{
    switch (s) {
        case Q4_OK: return "ok";
        case Q4_ERR_INVALID_ARG: return "invalid argument";
        case Q4_ERR_ALIGNMENT: return "misaligned pointer or pitch";
        case Q4_ERR_RANGE: return "value out of range";
        case Q4_ERR_WORKSPACE: return "workspace missing or too small";
        case Q4_ERR_UNSUPPORTED: return "unsupported";
        case Q4_ERR_WEIGHT_IMAGE: return "weight image prepared for another layer";
        case Q4_ERR_CUDA: return "CUDA error";
        case Q4_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case Q4_ERR_STATIC_SCRATCH:
            return "layer needs more scratch than the library's built-in static array holds";
    }
    return "unknown status";
}

int q4_version(void) { return 100; }

}  // extern "C"
