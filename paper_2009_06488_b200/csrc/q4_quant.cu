// The float boundary of a quantized layer: Eq. 1's linear quantizer (Section II-A) at the
// input of a quantized layer that follows a floating-point one (F -> Q, Section III-B), and
// Eq. 4's conversion of an integer result back to floating point (Q -> F).
//
// Reading of Eq. 1 (its zero point is printed in real units, Eq. 2 uses it in steps of s):
//   s = (max(max w, 0) - min(min w, 0)) / 15   (1 for an all-zero tensor)
//   z = -floor(min(min w, 0) / s), clamped to 0..15
//   code = clamp(floor(w / s) + z, 0, 15)
// All of it in IEEE binary32 with correctly rounded operations (__fsub_rn, __fdiv_rn), so
// that a code -- an integer decided by floating-point arithmetic -- is reproducible.
//
// Three HBM-bound kernels:
//  * range_kernel    -- min and max over the tensor: 128-bit loads, a warp reduction, one
//                       pair of atomics per block on an order-preserving integer image of
//                       the floats (0.0f <-> 0, so a zeroed pair of words is the start value
//                       min = max = 0 that Eq. 1 asks for);
//  * finalize_kernel -- the two words become {scale, zero point} in place;
//  * quantize_kernel -- eight values per thread and 32-bit word of codes (aligned fast
//                       path), else one output byte per thread.
//  * dequantize_kernel -- r = s * r_hat, four values per thread.
#include "q4_common.cuh"

namespace q4 {

// Order-preserving map float -> int32 with 0.0f -> 0.
__device__ __forceinline__ int float_to_ordered(float f)
{
    const int b = __float_as_int(f);
    return b >= 0 ? b : b ^ 0x7FFFFFFF;
}
__device__ __forceinline__ float ordered_to_float(int i)
{
    return __int_as_float(i >= 0 ? i : i ^ 0x7FFFFFFF);
}

__global__ void __launch_bounds__(256)
range_kernel(const float* __restrict__ X, int64_t ldx, int32_t rows, int32_t cols, int* range, int vec)
{
    float lo = 0.0f, hi = 0.0f;
    const int64_t tid = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    if (vec) {
        // dense, 16-byte aligned: the matrix is one array of rows * cols floats
        const int64_t n4 = (int64_t)rows * cols / 4;
        const float4* X4 = reinterpret_cast<const float4*>(X);
        int64_t i = tid;
        for (; i + 3 * nthreads < n4; i += 4 * nthreads) {     // four loads in flight
            const float4 a = __ldcs(X4 + i), b = __ldcs(X4 + i + nthreads), c = __ldcs(X4 + i + 2 * nthreads),
                         d = __ldcs(X4 + i + 3 * nthreads);
            lo = fminf(lo, fminf(fminf(fminf(a.x, a.y), fminf(a.z, a.w)), fminf(fminf(b.x, b.y), fminf(b.z, b.w))));
            lo = fminf(lo, fminf(fminf(fminf(c.x, c.y), fminf(c.z, c.w)), fminf(fminf(d.x, d.y), fminf(d.z, d.w))));
            hi = fmaxf(hi, fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w))));
            hi = fmaxf(hi, fmaxf(fmaxf(fmaxf(c.x, c.y), fmaxf(c.z, c.w)), fmaxf(fmaxf(d.x, d.y), fmaxf(d.z, d.w))));
        }
        for (; i < n4; i += nthreads) {
            const float4 v = X4[i];
            lo = fminf(fminf(lo, v.x), fminf(v.y, fminf(v.z, v.w)));
            hi = fmaxf(fmaxf(hi, v.x), fmaxf(v.y, fmaxf(v.z, v.w)));
        }
        for (int64_t i = n4 * 4 + tid; i < (int64_t)rows * cols; i += nthreads) {
            lo = fminf(lo, X[i]);
            hi = fmaxf(hi, X[i]);
        }
    } else {
        for (int64_t i = tid; i < (int64_t)rows * cols; i += nthreads) {
            const float v = X[(i / cols) * ldx + i % cols];
            lo = fminf(lo, v);
            hi = fmaxf(hi, v);
        }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
        hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
    }
    __shared__ float slo[8], shi[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { slo[warp] = lo; shi[warp] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) { lo = fminf(lo, slo[w]); hi = fmaxf(hi, shi[w]); }
        if (lo < 0.0f) atomicMin(&range[0], float_to_ordered(lo));
        if (hi > 0.0f) atomicMax(&range[1], float_to_ordered(hi));
    }
}

__global__ void finalize_kernel(int* range)
{
    const float lo = ordered_to_float(range[0]), hi = ordered_to_float(range[1]);
    float s = __fdiv_rn(__fsub_rn(hi, lo), 15.0f);
    if (s == 0.0f) s = 1.0f;
    int z = -(int)floorf(__fdiv_rn(lo, s));
    z = min(max(z, 0), 15);
    range[0] = __float_as_int(s);
    range[1] = z;
}

// floor(fl(w / s)) -- the floor of the CORRECTLY ROUNDED binary32 quotient, which is what Eq. 1's
// code is defined by here -- without a division for almost every value.  With r = fl(1 / s)
// and x = fl(w * r): |x - fl(w / s)| <= (2^-23 + 2^-24) |w / s| (two roundings on one side, one
// on the other), so floor(x) is the wanted floor unless x lies within that distance of an
// integer; only then (and for a zero product, whose sign may have been lost to underflow) is
// the division carried out.  The test distance is 1e-6 |x|, five times the bound.  `fast` is
// false for scales so small or large that r would overflow or be subnormal.
__device__ __forceinline__ int floor_quotient(float w, float s, float r, bool fast)
{
    if (fast) {
        const float x = __fmul_rn(w, r);
        const float fx = floorf(x);
        const float d = __fsub_rn(x, fx);                      // exact, in [0, 1)
        const float thr = 1e-6f * fmaxf(fabsf(x), 1.0f);
        if (!(d < thr) && !(d > 1.0f - thr)) return __float2int_rd(fx);
    }
    return __float2int_rd(__fdiv_rn(w, s));
}

// Rows are walked by blockIdx.y, the 32-bit words of a row by blockIdx.x and the thread
// index: no divisions.  A dense matrix is passed as one row.
__global__ void __launch_bounds__(256)
quantize_vec_kernel(const float* __restrict__ X, int64_t ldx, int32_t rows, int64_t words_per_row,
                    const q4_qparams* __restrict__ qp, uint8_t* __restrict__ Q, int64_t ldq)
{
    const float s = qp->scale;
    const int z = qp->zero;
    const bool fast = s > 1e-30f && s < 1e30f;
    const float rs = __frcp_rn(s);
    for (int64_t r = blockIdx.y; r < rows; r += gridDim.y) {
        const float* xr = X + r * ldx;
        uint8_t* qr = Q + r * ldq;
        for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < words_per_row;
             j += (int64_t)gridDim.x * blockDim.x) {
            const float4* src = reinterpret_cast<const float4*>(xr + 8 * j);
            const float4 a = __ldcs(src), b = __ldcs(src + 1);
            const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
            uint32_t word = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                int q = floor_quotient(v[e], s, rs, fast);
                q = min(max(q, -z), 15 - z) + z;       // clamp before adding: no overflow
                word |= (uint32_t)q << (4 * e);
            }
            *reinterpret_cast<uint32_t*>(qr + 4 * j) = word;
        }
    }
}

__global__ void __launch_bounds__(256)
quantize_byte_kernel(const float* __restrict__ X, int64_t ldx, int32_t rows, int32_t cols,
                     const q4_qparams* __restrict__ qp, uint8_t* __restrict__ Q, int64_t ldq)
{
    const float s = qp->scale;
    const int z = qp->zero;
    const bool fast = s > 1e-30f && s < 1e30f;
    const float rs = __frcp_rn(s);
    const int kb = (cols + 1) / 2;
    const int64_t total = (int64_t)rows * kb;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / kb;
        const int j = (int)(i - r * kb);
        uint32_t byte = 0;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int c = 2 * j + e;
            if (c < cols) {
                int q = floor_quotient(X[r * ldx + c], s, rs, fast);
                q = min(max(q, -z), 15 - z) + z;
                byte |= (uint32_t)q << (4 * e);
            }
        }
        Q[r * ldq + j] = (uint8_t)byte;
    }
}

__global__ void __launch_bounds__(256)
dequantize_kernel(const int32_t* __restrict__ C, int64_t ldc, int32_t rows, int32_t cols, float scale,
                  float* __restrict__ R, int64_t ldr, int vec)
{
    if (vec) {
        const int qpr = cols / 4;
        const int64_t total = (int64_t)rows * qpr;
        for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
             i += (int64_t)gridDim.x * blockDim.x) {
            const int64_t r = i / qpr;
            const int j = (int)(i - r * qpr);
            const int4 c = *reinterpret_cast<const int4*>(C + r * ldc + 4 * j);
            float4 o;
            o.x = __fmul_rn(__int2float_rn(c.x), scale);
            o.y = __fmul_rn(__int2float_rn(c.y), scale);
            o.z = __fmul_rn(__int2float_rn(c.z), scale);
            o.w = __fmul_rn(__int2float_rn(c.w), scale);
            *reinterpret_cast<float4*>(R + r * ldr + 4 * j) = o;
        }
    } else {
        const int64_t total = (int64_t)rows * cols;
        for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
             i += (int64_t)gridDim.x * blockDim.x) {
            const int64_t r = i / cols;
            const int j = (int)(i - r * cols);
            R[r * ldr + j] = __fmul_rn(__int2float_rn(C[r * ldc + j]), scale);
        }
    }
}

static int grid_for(int64_t work_items)
{
    int64_t blocks = (work_items + 255) / 256;
    const int64_t cap = 148 * 16;
    if (blocks > cap) blocks = cap;
    return (int)(blocks < 1 ? 1 : blocks);
}

cudaError_t launch_quant_params(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                                q4_qparams* qp, cudaStream_t st)
{
    cudaError_t e = cudaMemsetAsync(qp, 0, sizeof(q4_qparams), st);    // min = max = 0
    if (e != cudaSuccess) return e;
    const int64_t n = (int64_t)rows * cols;
    if (n > 0) {
        const int vec = ldx == cols && (uintptr_t)X % 16 == 0;
        range_kernel<<<grid_for(vec ? n / 4 : n), 256, 0, st>>>(X, ldx, rows, cols, reinterpret_cast<int*>(qp), vec);
        count_launch();
    }
    finalize_kernel<<<1, 1, 0, st>>>(reinterpret_cast<int*>(qp));
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_quantize(const float* X, int64_t ldx, int32_t rows, int32_t cols,
                            const q4_qparams* qp, uint8_t* Q, int64_t ldq, cudaStream_t st)
{
    if ((int64_t)rows * cols == 0) return cudaSuccess;
    const bool vec = cols % 8 == 0 && ldx % 4 == 0 && ldq % 4 == 0 && (uintptr_t)X % 16 == 0 &&
                     (uintptr_t)Q % 4 == 0;
    if (vec) {
        // a dense matrix is one long row
        const bool dense = ldx == cols && ldq * 2 == cols;
        const int32_t r2 = dense ? 1 : rows;
        const int64_t wpr = dense ? (int64_t)rows * cols / 8 : cols / 8;
        int64_t gx = (wpr + 255) / 256, gy = r2;
        const int64_t cap = 148 * 16;
        if (gx > cap) gx = cap;
        if (gy > cap / gx) gy = cap / gx < 1 ? 1 : cap / gx;
        quantize_vec_kernel<<<dim3((unsigned)gx, (unsigned)gy), 256, 0, st>>>(X, ldx, r2, wpr, qp, Q, ldq);
    }
    else
        quantize_byte_kernel<<<grid_for((int64_t)rows * ((cols + 1) / 2)), 256, 0, st>>>(X, ldx, rows, cols, qp, Q, ldq);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_dequantize(const int32_t* C, int64_t ldc, int32_t rows, int32_t cols, float scale,
                              float* R, int64_t ldr, cudaStream_t st)
{
    if ((int64_t)rows * cols == 0) return cudaSuccess;
    const int vec = cols % 4 == 0 && ldc % 4 == 0 && ldr % 4 == 0 && (uintptr_t)C % 16 == 0 &&
                    (uintptr_t)R % 16 == 0;
    dequantize_kernel<<<grid_for(vec ? (int64_t)rows * (cols / 4) : (int64_t)rows * cols), 256, 0, st>>>(
        C, ldc, rows, cols, scale, R, ldr, vec);
    count_launch();
    return cudaGetLastError();
}

}  // namespace q4
