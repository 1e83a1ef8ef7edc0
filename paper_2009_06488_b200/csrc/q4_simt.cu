// General (SIMT) kernels of the q4 library: no alignment requirements, any shape.
// They are the slow-but-always-valid variants behind the tensor-core path, and the
// small helper kernels (weight transposition, depth sums, generic unrolling).
#include "q4_common.cuh"

namespace q4 {

// ------------------------------------------------------------------------------------
// Quantized GEMM (Eq. 2), 64 x 64 output tile per block, dp4a on unpacked bytes.
// ------------------------------------------------------------------------------------
constexpr int ST = 64;          // tile edge (rows of A / rows of Bt)
constexpr int SK = 64;          // depth slab in nibbles
constexpr int SPITCH = SK + 4;  // smem row pitch in bytes (17 words: conflict-free)

__device__ __forceinline__ void load_unpack_tile(const uint8_t* __restrict__ P, int64_t ld,
                                                 int row0, int rows, int kbyte0, int kbytes,
                                                 uint8_t (*s)[SPITCH], int tid)
{
#pragma unroll
    for (int i = 0; i < (ST * SK / 2) / 256; ++i) {
        int idx = tid + 256 * i;
        int r = idx / (SK / 2), kb = idx % (SK / 2);
        uint8_t byte = 0;
        if (row0 + r < rows && kbyte0 + kb < kbytes)
            byte = P[(int64_t)(row0 + r) * ld + kbyte0 + kb];
        *reinterpret_cast<uint16_t*>(&s[r][2 * kb]) =
            (uint16_t)((byte & 0x0F) | ((uint16_t)(byte >> 4) << 8));
    }
}

template <bool REQUANT>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmParams p)
{
    __shared__ __align__(16) uint8_t sA[ST][SPITCH];
    __shared__ __align__(16) uint8_t sB[ST][SPITCH];

    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int m0 = blockIdx.y * ST, n0 = blockIdx.x * ST;
    const int kbytes = (p.K + 1) / 2;

    int rows[4], cols[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) rows[i] = ty + 16 * i;
    cols[0] = 2 * tx; cols[1] = 2 * tx + 1; cols[2] = 2 * tx + 32; cols[3] = 2 * tx + 33;

    int acc[4][4] = {};
    int rsum[4] = {}, csum[4] = {};

    for (int kb0 = 0; kb0 < kbytes; kb0 += SK / 2) {
        load_unpack_tile(p.A, p.lda, m0, p.M, kb0, kbytes, sA, tid);
        load_unpack_tile(p.Bt, p.ldb, n0, p.N, kb0, kbytes, sB, tid);
        __syncthreads();
#pragma unroll
        for (int k4 = 0; k4 < SK / 4; ++k4) {
            uint32_t a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const uint32_t*>(&sA[rows[i]][4 * k4]);
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = *reinterpret_cast<const uint32_t*>(&sB[cols[j]][4 * k4]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                rsum[i] = dp4a_u8(a[i], 0x01010101u, rsum[i]);
                csum[i] = dp4a_u8(b[i], 0x01010101u, csum[i]);
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = dp4a_u8(a[i], b[j], acc[i][j]);
            }
        }
        __syncthreads();
    }

    const int kzz = p.K * p.za * p.zb;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + rows[i];
        if (m >= p.M) continue;
        const int ra = p.rowsum_a ? p.rowsum_a[m] : rsum[i];
        int v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + cols[j];
            int cb = 0, bias = 0;
            if (n < p.N) {
                cb = p.colsum_b ? p.colsum_b[n] : csum[j];
                if (REQUANT && p.bias) bias = p.bias[n];
            }
            v[j] = (int)((uint32_t)correct(acc[i][j], ra, cb, p.za, p.zb, kzz) + (uint32_t)bias);
        }
        if (!REQUANT) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (n0 + cols[j] < p.N) p.C[(int64_t)m * p.ldc + n0 + cols[j]] = v[j];
        } else {
#pragma unroll
            for (int j = 0; j < 4; j += 2) {
                const int n = n0 + cols[j];       // even; N is even, so n + 1 < N too
                if (n < p.N)
                    p.Cq[(int64_t)m * p.ldcq + (n >> 1)] =
                        (uint8_t)(requant(v[j], p.rq) | (requant(v[j + 1], p.rq) << 4));
            }
        }
    }
}

cudaError_t launch_gemm_simt(const GemmParams& p, bool rq, cudaStream_t st)
{
    dim3 grid((p.N + ST - 1) / ST, (p.M + ST - 1) / ST);
    if (grid.y > 65535) {
        // fold very tall problems: launch in row bands
        const int band = 65535 * ST;
        for (int64_t m0 = 0; m0 < p.M; m0 += band) {
            GemmParams q = p;
            q.A = p.A + m0 * p.lda;
            q.M = (int32_t)((p.M - m0 < band) ? (p.M - m0) : band);
            if (p.rowsum_a) q.rowsum_a = p.rowsum_a + m0;
            if (p.C) q.C = p.C + m0 * p.ldc;
            if (p.Cq) q.Cq = p.Cq + m0 * p.ldcq;
            cudaError_t e = launch_gemm_simt(q, rq, st);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    }
    if (rq) gemm_simt_kernel<true><<<grid, 256, 0, st>>>(p);
    else    gemm_simt_kernel<false><<<grid, 256, 0, st>>>(p);
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// K x N packed along n  ->  N x K packed along k (weights, once per matrix).
// One thread per output byte; pad bytes of the pitch are written 0.
// ------------------------------------------------------------------------------------
__global__ void pack_bt_kernel(const uint8_t* __restrict__ B_kn, int64_t ldb_kn,
                               uint8_t* __restrict__ Bt, int64_t ldb, int K, int N)
{
    const int64_t total = (int64_t)N * ldb;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i / ldb), kb = (int)(i % ldb);
        uint32_t out = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int k = 2 * kb + h;
            if (k < K) {
                const uint8_t byte = B_kn[(int64_t)k * ldb_kn + (n >> 1)];
                out |= ((n & 1) ? (byte >> 4) : (byte & 0x0F)) << (4 * h);
            }
        }
        Bt[i] = (uint8_t)out;
    }
}

cudaError_t launch_pack_bt(const uint8_t* B_kn, int64_t ldb_kn, uint8_t* Bt, int64_t ldb,
                           int32_t K, int32_t N, cudaStream_t st)
{
    const int64_t total = (int64_t)N * ldb;
    int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    if (blocks < 1) blocks = 1;
    pack_bt_kernel<<<blocks, 256, 0, st>>>(B_kn, ldb_kn, Bt, ldb, K, N);
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// Depth sums of a packed matrix: one warp per row.
// ------------------------------------------------------------------------------------
__global__ void row_sums_kernel(const uint8_t* __restrict__ P, int64_t ld, int rows, int K,
                                int32_t* __restrict__ sums)
{
    const int lane = threadIdx.x % 32;
    const int kbytes = (K + 1) / 2;
    for (int64_t r = blockIdx.x * (int64_t)(blockDim.x / 32) + threadIdx.x / 32; r < rows;
         r += (int64_t)gridDim.x * (blockDim.x / 32)) {
        const uint8_t* row = P + r * ld;
        int s = 0;
        for (int b = lane; b < kbytes; b += 32) {
            const uint8_t byte = row[b];
            s += (byte & 0x0F) + (byte >> 4);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (lane == 0) sums[r] = s;
    }
}

// Depth sums of both GEMM operands in one launch (the sums of Eq. 2's second and third
// terms), one warp per row, 128-bit loads when base and pitch allow.  HBM-bound: each
// packed byte is read once.
__global__ void __launch_bounds__(256) operand_sums_kernel(const uint8_t* __restrict__ A, int64_t lda,
                                                           int rows_a, int32_t* __restrict__ sums_a,
                                                           const uint8_t* __restrict__ B, int64_t ldb,
                                                           int rows_b, int32_t* __restrict__ sums_b,
                                                           int K, int vec)
{
    // Launched with programmatic stream serialization (its launch overlaps the previous kernel's
    // tail): nothing is read before that kernel has completed; the kernel after this one -- the
    // GEMM, which waits in the same way -- may begin its prologue at once.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x % 32;
    const int kbytes = (K + 1) / 2;
    const int total = rows_a + rows_b;
    for (int r = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32; r < total;
         r += gridDim.x * (blockDim.x / 32)) {
        const bool is_a = r < rows_a;
        const uint8_t* row = is_a ? A + (int64_t)r * lda : B + (int64_t)(r - rows_a) * ldb;
        int s = 0;
        int done = 0;
        if (vec) {
            const int nvec = kbytes / 16;
            const uint4* v = reinterpret_cast<const uint4*>(row);
            int i = lane;
            for (; i + 96 < nvec; i += 128) {          // four independent loads in flight
                const uint4 w0 = v[i], w1 = v[i + 32], w2 = v[i + 64], w3 = v[i + 96];
                s += nibble_sum(w0.x) + nibble_sum(w0.y) + nibble_sum(w0.z) + nibble_sum(w0.w);
                s += nibble_sum(w1.x) + nibble_sum(w1.y) + nibble_sum(w1.z) + nibble_sum(w1.w);
                s += nibble_sum(w2.x) + nibble_sum(w2.y) + nibble_sum(w2.z) + nibble_sum(w2.w);
                s += nibble_sum(w3.x) + nibble_sum(w3.y) + nibble_sum(w3.z) + nibble_sum(w3.w);
            }
            for (; i < nvec; i += 32) {
                const uint4 w = v[i];
                s += nibble_sum(w.x) + nibble_sum(w.y) + nibble_sum(w.z) + nibble_sum(w.w);
            }
            done = nvec * 16;
        }
        for (int b = done + lane; b < kbytes; b += 32) {
            const uint8_t byte = row[b];
            s += (byte & 0x0F) + (byte >> 4);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (lane == 0) {
            if (is_a) sums_a[r] = s; else sums_b[r - rows_a] = s;
        }
    }
}

cudaError_t launch_operand_sums(const uint8_t* A, int64_t lda, int32_t rows_a, int32_t* sums_a,
                                const uint8_t* B, int64_t ldb, int32_t rows_b, int32_t* sums_b,
                                int32_t K, cudaStream_t st)
{
    const int total = rows_a + rows_b;
    if (total <= 0) return cudaSuccess;
    const int vec = ((rows_a == 0 || ((uintptr_t)A % 16 == 0 && lda % 16 == 0)) &&
                     (rows_b == 0 || ((uintptr_t)B % 16 == 0 && ldb % 16 == 0))) ? 1 : 0;
    int blocks = (total + 7) / 8 < 148 * 16 ? (total + 7) / 8 : 148 * 16;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, operand_sums_kernel, A, (int64_t)lda, (int)rows_a, sums_a, B,
                                             (int64_t)ldb, (int)rows_b, sums_b, (int)K, vec);
    count_launch();
    return e;
}

cudaError_t launch_row_sums(const uint8_t* P, int64_t ld, int32_t rows, int32_t K,
                            int32_t* sums, cudaStream_t st)
{
    int blocks = (rows + 7) / 8 < 148 * 8 ? (rows + 7) / 8 : 148 * 8;
    if (blocks < 1) blocks = 1;
    row_sums_kernel<<<blocks, 256, 0, st>>>(P, ld, rows, K, sums);
    count_launch();
    return cudaGetLastError();
}

}  // namespace q4
