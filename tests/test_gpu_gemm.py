"""GPU parity: q4_gemm / q4_gemm_requant through the C ABI against the CPU oracle,
element by element, bit-exact (all work is integer)."""
import numpy as np
import pytest

import oracle
from paper_2009_06488_b200 import workloads as wl

pytestmark = pytest.mark.gpu

SIMT, TC, TC1 = 1, 2, 3      # general kernel / tensor-core (auto) / single-CTA tensor-core only
TC192, TC256 = 5, 6          # tensor-core with the CTA-pair kernel's tile width fixed


@pytest.fixture(scope="module")
def q4():
    from paper_2009_06488_b200 import binding
    yield binding
    binding.q4_set_variant(0)


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_gemm(q4, c, variant, ldc_pad=0, sums=False, use_ws=False):
    import torch
    q4.q4_set_variant(variant)
    A, Bt = dev(c.A), dev(c.Bt)
    C = torch.full((c.M, c.N + ldc_pad), -1515870811, dtype=torch.int32, device="cuda")  # 0xA5A5A5A5
    ra = cb = None
    if sums:
        ra = torch.empty(c.M, dtype=torch.int32, device="cuda")
        cb = torch.empty(c.N, dtype=torch.int32, device="cuda")
        q4.q4_row_sums(A, c.M, c.K, ra)
        q4.q4_row_sums(Bt, c.N, c.K, cb)
        if sums == "cols":      # the weights' sums only: the kernel takes the row sums of A
            ra = None
        if sums == "rows":
            cb = None
    ws = None
    if use_ws:     # scratch (poisoned): the depth sums
        ws = torch.full((q4.q4_gemm_workspace_bytes(c.M, c.N, c.K),), 0xA5, dtype=torch.uint8, device="cuda")
    q4.q4_gemm(A, Bt, C, c.M, c.N, c.K, c.za, c.zb, ra, cb, ws)
    assert q4.q4_last_device_status() == q4.Q4_OK
    out = C.cpu().numpy()
    if ldc_pad:
        assert (out[:, c.N:] == -1515870811).all()      # pitch padding untouched
    return out[:, :c.N], ra, cb


def run_requant(q4, c, variant, rq, bias=None, ld_pad=0, use_ws=False):
    import torch
    q4.q4_set_variant(variant)
    A, Bt = dev(c.A), dev(c.Bt)
    Cq = torch.full((c.M, c.N // 2 + ld_pad), 0xA5, dtype=torch.uint8, device="cuda")
    ws = None
    if use_ws:
        ws = torch.full((q4.q4_gemm_workspace_bytes(c.M, c.N, c.K),), 0xA5, dtype=torch.uint8, device="cuda")
    q4.q4_gemm_requant(A, Bt, Cq, c.M, c.N, c.K, c.za, c.zb,
                       q4.Requant(rq.mult, rq.shift, rq.zo, rq.clamp_lo, rq.clamp_hi),
                       None if bias is None else dev(bias), ws=ws)
    assert q4.q4_last_device_status() == q4.Q4_OK
    out = Cq.cpu().numpy()
    if ld_pad:
        assert (out[:, c.N // 2:] == 0xA5).all()
    return out[:, :c.N // 2]


TABLE1 = [(h, w, d) for h in (8, 24) for w in (100, 400, 1600) for d in (10, 40, 100)]
ODD = [(1, 1, 1), (3, 5, 7), (65, 33, 129), (130, 70, 255), (64, 64, 64)]


@pytest.mark.parametrize("shape", TABLE1 + ODD)
def test_simt_gemm_any_shape_any_pitch(q4, shape):
    M, N, K = shape
    kb = (K + 1) // 2
    c = wl.gemm_case("t", M, N, K, seed=M * 7919 + N * 31 + K, lda=kb + 3, ldb=kb + 1)
    got, _, _ = run_gemm(q4, c, SIMT, ldc_pad=3)
    want = oracle.gemm(c.A, c.Bt, M, N, K, c.za, c.zb)
    assert (got == want).all()


# aligned problems for the tensor-core path: tails in M, N and K, small N, tiny K
TC_SHAPES = [(64, 64, 256), (128, 256, 128), (128, 32, 32), (130, 260, 1000), (257, 40, 144),
             (300, 16, 72), (1000, 8, 9), (129, 130, 131), (384, 512, 1024), (5, 3, 1),
             (256, 96, 4096), (200, 200, 33)]


def aligned_case(M, N, K, seed, **kw):
    ld = ((K + 1) // 2 + 15) // 16 * 16
    return wl.gemm_case("t", M, N, K, seed=seed, lda=ld, ldb=ld, **kw)


@pytest.mark.parametrize("shape", TC_SHAPES)
def test_tc_gemm_matches_oracle(q4, shape):
    M, N, K = shape
    c = aligned_case(M, N, K, seed=M * 7919 + N * 31 + K)
    want = oracle.gemm(c.A, c.Bt, M, N, K, c.za, c.zb)
    got, _, _ = run_gemm(q4, c, TC, ldc_pad=4)
    assert (got == want).all()
    got2, _, _ = run_gemm(q4, c, TC, ldc_pad=1)      # unaligned int32 pitch: scalar stores
    assert (got2 == want).all()


# shapes that reach the CTA-pair kernel (M, N >= 256): tails in M, N, K; short depths
PAIR_SHAPES = [(256, 256, 128), (300, 260, 1000), (257, 514, 129), (1000, 300, 4096), (512, 768, 64),
               (384, 512, 33), (2048, 256, 640), (256, 192, 128), (700, 200, 257), (512, 400, 4096), (300, 200, 1000), (256, 192, 100), (640, 384, 31)]


@pytest.mark.parametrize("variant", [TC, TC1])
@pytest.mark.parametrize("shape", PAIR_SHAPES)
def test_pair_and_single_tensor_core_kernels_agree_with_oracle(q4, variant, shape):
    M, N, K = shape
    c = aligned_case(M, N, K, seed=M * 31 + N * 7 + K, with_bias=True)
    want = oracle.gemm(c.A, c.Bt, M, N, K, c.za, c.zb)
    got, _, _ = run_gemm(q4, c, variant, ldc_pad=4)
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, sums=True)
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, use_ws=True)     # sums taken by the pre-pass
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, sums="cols", use_ws=True)    # row sums of A inside the kernel
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, sums="rows")                 # column sums of Bt inside the kernel
    assert (got == want).all()
    rq = oracle.Requant(c.mult, 6, 4, 4, 15)
    wantq = oracle.requant_matrix(want, c.bias, rq)
    assert (run_requant(q4, c, variant, rq, c.bias, ld_pad=16) == wantq).all()
    assert (run_requant(q4, c, variant, rq, c.bias, ld_pad=3) == wantq).all()   # byte stores
    assert (run_requant(q4, c, variant, rq, c.bias, use_ws=True) == wantq).all()


# Both tile widths of the CTA-pair kernel on the same problems: column tails that leave the
# upper half of a 256-column tile empty or ragged, depths shorter than the operand rings, and
# enough tiles per CTA pair (four and more) for the accumulator buffers to go round.
WIDTH_SHAPES = [(256, 256, 128), (300, 320, 1000), (257, 200, 129), (512, 390, 64), (384, 512, 33),
                (4096, 4352, 256), (5000, 4100, 130), (2304, 2048, 640)]


@pytest.mark.parametrize("variant", [TC192, TC256])
@pytest.mark.parametrize("shape", WIDTH_SHAPES)
def test_pair_kernel_tile_widths_agree_with_oracle(q4, variant, shape):
    M, N, K = shape
    c = aligned_case(M, N, K, seed=M * 13 + N * 5 + K, with_bias=True)
    want = oracle.gemm(c.A, c.Bt, M, N, K, c.za, c.zb)
    got, _, _ = run_gemm(q4, c, variant, ldc_pad=4)           # depth sums taken inside the kernel
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, sums=True)
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, sums="cols")         # row sums alone: they stay inside a CTA
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, sums="rows", use_ws=True)
    assert (got == want).all()
    got, _, _ = run_gemm(q4, c, variant, ldc_pad=1)           # unaligned int32 pitch: scalar stores
    assert (got == want).all()
    rq = oracle.Requant(c.mult, 6, 4, 4, 15)
    wantq = oracle.requant_matrix(want, c.bias, rq)
    assert (run_requant(q4, c, variant, rq, c.bias, ld_pad=16) == wantq).all()
    assert (run_requant(q4, c, variant, rq, c.bias, ld_pad=3) == wantq).all()
    assert (run_requant(q4, c, variant, rq, c.bias, use_ws=True) == wantq).all()


def _random_shapes(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        M = int(rng.integers(1, 2600)) if rng.random() < 0.75 else int(rng.integers(3000, 7000))
        N = 2 * int(rng.integers(1, 700))
        K = int(rng.integers(1, 600)) if rng.random() < 0.6 else int(rng.integers(1, 48))   # many one-stage tiles
        out.append((M, N, K))
    return out


@pytest.mark.parametrize("shape", _random_shapes(36, 20260101))
def test_random_shapes_every_kernel_and_sums_combination(q4, shape):
    """Seeded random shapes (ragged in every dimension, a third of them with one or two
    depth stages per tile so that a CTA's tiles follow each other within a few thousand
    clocks) through the automatic choice and each forced kernel, with the depth sums given,
    given for the weights only, and taken through a workspace: int32 and re-quantized output
    against the oracle."""
    import torch
    M, N, K = shape
    c = aligned_case(M, N, K, seed=M * 131 + N * 17 + K, with_bias=True)
    want = oracle.gemm(c.A, c.Bt, M, N, K, c.za, c.zb)
    rq = oracle.Requant(c.mult, 7, 3, 1, 14)
    wantq = oracle.requant_matrix(want, c.bias, rq)
    for variant in (0, TC1, TC192, TC256):
        for kw in ({}, {"sums": True}, {"sums": "cols"}, {"use_ws": True}):
            try:
                got, _, _ = run_gemm(q4, c, variant, **kw)
            except q4.Q4Error as e:          # a forced kernel that does not take the shape
                assert e.status in (q4.Q4_ERR_ALIGNMENT, q4.Q4_ERR_UNSUPPORTED)
                continue
            assert (got == want).all(), (variant, kw)
        try:
            assert (run_requant(q4, c, variant, rq, c.bias) == wantq).all(), variant
        except q4.Q4Error as e:
            assert e.status in (q4.Q4_ERR_ALIGNMENT, q4.Q4_ERR_UNSUPPORTED)
    q4.q4_set_variant(0)


def test_odd_number_of_chunks_per_tile_with_short_depth(q4):
    """192-column tiles whose last column tile drains five of its six 32-column chunks
    (N = 1116), one depth stage per tile, depth sums taken in the kernel: the int32 staging
    slices of an epilogue warp alternate from store to store, and the next tile's first
    store follows the last one of this tile within a few hundred clocks.  Repeated, because
    what this guards against is a race (a slice refilled while its store still reads it)."""
    import torch
    M, N, K = 5415, 1116, 28
    c = aligned_case(M, N, K, seed=4242)
    want = torch.from_numpy(oracle.gemm(c.A, c.Bt, M, N, K, c.za, c.zb)).cuda()
    A, Bt = dev(c.A), dev(c.Bt)
    q4.q4_set_variant(TC192)
    try:
        for _ in range(60):
            C = torch.full((M, N), -1515870811, dtype=torch.int32, device="cuda")
            q4.q4_gemm(A, Bt, C, M, N, K, c.za, c.zb)
            assert torch.equal(C, want)
        assert q4.q4_last_device_status() == q4.Q4_OK
    finally:
        q4.q4_set_variant(0)


@pytest.mark.parametrize("variant", [SIMT, TC])
def test_precomputed_sums_give_the_same_result(q4, variant):
    c = aligned_case(200, 72, 300, seed=77)
    want, ra_want, cb_want = oracle.gemm_fourterm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb)
    got, ra, cb = run_gemm(q4, c, variant, sums=True)
    assert (ra.cpu().numpy() == ra_want).all() and (cb.cpu().numpy() == cb_want).all()
    assert (got == want).all()


@pytest.mark.parametrize("variant", [SIMT, TC])
@pytest.mark.parametrize("zz", [(0, 0), (15, 15), (0, 15), (15, 0)])
def test_extreme_zero_points(q4, variant, zz):
    c = aligned_case(140, 48, 520, seed=5, za=zz[0], zb=zz[1])
    got, _, _ = run_gemm(q4, c, variant)
    assert (got == oracle.gemm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb)).all()


@pytest.mark.parametrize("variant", [SIMT, TC])
def test_all_fifteen_inputs_reach_225K(q4, variant):
    K = 4096
    c = aligned_case(128, 32, K, seed=1, za=0, zb=0)
    c.A[:, :K // 2] = 0xFF
    c.Bt[:, :K // 2] = 0xFF
    got, _, _ = run_gemm(q4, c, variant)
    assert (got == 225 * K).all()


def test_c1_single_gemm(q4):
    c = wl.c1()
    want = oracle.gemm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb)
    for v in (SIMT, TC):
        got, _, _ = run_gemm(q4, c, v)
        assert (got == want).all()


@pytest.mark.parametrize("variant", [SIMT, TC])
@pytest.mark.parametrize("shape", [(64, 64, 256), (130, 260, 1000), (257, 40, 144), (300, 16, 72),
                                   (33, 2, 5), (128, 256, 512)])
def test_gemm_requant_matches_oracle(q4, variant, shape):
    M, N, K = shape
    c = aligned_case(M, N, K, seed=M + N + K, with_bias=True, za=8, zb=7)   # centred: outputs spread
    for i, (shift, zo, lo, hi) in enumerate([(c.shift, 0, 0, 15), (4, 3, 3, 15), (0, 8, 0, 9)]):
        rq = oracle.Requant(c.mult, shift, zo, lo, hi)
        bias = c.bias if i else None
        want = oracle.gemm_requant(c.A, c.Bt, M, N, K, c.za, c.zb, bias, rq)
        got = run_requant(q4, c, variant, rq, bias, ld_pad=0 if i == 0 else 16)
        assert (got == want).all()
        if shift == 4 and K >= 100:
            assert len(np.unique(oracle.unpack_rows(got, N))) > 3   # not saturated everywhere


@pytest.mark.parametrize("n", [512, 1024, 2048])
def test_c2_square_sweep_full_compare(q4, n):
    c = wl.c2(n)
    want = oracle.gemm(c.A, c.Bt, n, n, n, c.za, c.zb)
    got, _, _ = run_gemm(q4, c, TC)
    assert (got == want).all()
    rq = oracle.Requant(c.mult, c.shift, 0, 0, 15)
    wantq = oracle.requant_matrix(want, None, rq)
    gotq = run_requant(q4, c, TC, rq)
    assert (gotq == wantq).all()


def freivalds_check(c, C):
    """Exact integer Freivalds: C r == A' (B' r) and l C == (l A') B' in int64, with
    A' = A - za, B' = B - zb taken from the unpacked operands in row blocks."""
    rng = np.random.default_rng(c.seed + 1)
    r = rng.integers(1, 1 << 20, c.N).astype(np.int64)
    l = rng.integers(1, 1 << 20, c.M).astype(np.int64)
    blk = 512
    y = np.zeros(c.K, np.int64)                     # B' r
    for n0 in range(0, c.N, blk):
        b = oracle.unpack_rows(c.Bt[n0:n0 + blk], c.K).astype(np.int64) - c.zb
        y += b.T @ r[n0:n0 + blk]
    lA = np.zeros(c.K, np.int64)                    # l A'
    for m0 in range(0, c.M, blk):
        a = oracle.unpack_rows(c.A[m0:m0 + blk], c.K).astype(np.int64) - c.za
        assert (C[m0:m0 + blk].astype(np.int64) @ r == a @ y).all()
        lA += l[m0:m0 + blk] @ a
    lC = l @ C.astype(np.int64)
    for n0 in range(0, c.N, blk):
        b = oracle.unpack_rows(c.Bt[n0:n0 + blk], c.K).astype(np.int64) - c.zb
        assert (lC[n0:n0 + blk] == b @ lA).all()


def sampled_rows_check(c, C, rows):
    sub = np.ascontiguousarray(c.A[rows])
    want = oracle.gemm(sub, c.Bt, len(rows), c.N, c.K, c.za, c.zb)
    assert (C[rows] == want).all()


def test_c2_4096_sampled_rows_and_freivalds(q4):
    c = wl.c2(4096)
    got, _, _ = run_gemm(q4, c, TC)
    rows = np.unique(np.concatenate([np.arange(0, 4096, 97), [0, 127, 128, 4095]]))
    sampled_rows_check(c, got, rows)
    freivalds_check(c, got)
    # The int32 matrix is now known to equal the oracle's (sampled rows + exact Freivalds on
    # every entry), so the oracle's requantizer applied to it is the expected packed output
    # for the WHOLE matrix: every tile of every cluster, not a sample.
    rq = oracle.Requant(c.mult, c.shift, 0, 0, 15)
    gotq = run_requant(q4, c, TC, rq)
    assert (gotq == oracle.requant_matrix(got, None, rq)).all()
    # bias, a non-zero output zero point and a ReLU-style lower clamp on the same product
    # (the bias also re-centres the accumulators, whose mean follows the drawn zero points)
    bias = (wl.rand_ints(c.seed, 9, -512, 512, c.N) - int(got.mean())).astype(np.int32)
    span = max(1, int(np.abs(got.astype(np.int64) + bias[None, :]).max()))
    shift2 = min(31, max(0, int(np.ceil(np.log2(span / 8.0)))))       # outputs spread over the code range
    rq2 = oracle.Requant(c.mult, shift2, 8, 3, 14)
    gotq2 = run_requant(q4, c, TC, rq2, bias, use_ws=True)
    wantq2 = oracle.requant_matrix(got, bias, rq2)
    assert (gotq2 == wantq2).all()
    assert len(np.unique(oracle.unpack_rows(wantq2[:64], c.N))) > 3      # not saturated everywhere


def big_case_check(q4, c, nrows):
    """Full-size problems in the launch configuration the benchmark times: rows sampled
    across every row tile against the oracle, plus exact integer Freivalds on the whole
    matrix (any wrong entry breaks one of the two products)."""
    got, _, _ = run_gemm(q4, c, 0, use_ws=True)
    rng = np.random.default_rng(c.seed)
    rows = np.unique(np.concatenate([rng.integers(0, c.M, nrows), [0, 127, 128, 255, 256, c.M - 1]]))
    sampled_rows_check(c, got, rows)
    freivalds_check(c, got)
    return got, rows


def test_c2_8192_benchmark_shape(q4):
    c = wl.c2(8192)
    got, rows = big_case_check(q4, c, 40)
    rq = oracle.Requant(c.mult, c.shift, 0, 0, 15)
    gotq = run_requant(q4, c, 0, rq, use_ws=True)
    # whole packed matrix against the oracle's requantizer on the verified accumulators:
    # this is the only size at which a cluster of the fused-requant kernel owns several
    # tiles in a row
    assert (gotq == oracle.requant_matrix(got, None, rq)).all()


def test_c5_deep_k_worst_case_zero_points(q4):
    c = wl.c5()
    assert (c.za, c.zb) == (0, 15)
    got, _ = big_case_check(q4, c, 24)
    assert got.max() <= 0 and got.min() >= -225 * c.K     # sum a (b - 15) is never positive


def test_empty_problem_is_a_no_op(q4):
    import torch
    A = torch.zeros((0, 64), dtype=torch.uint8, device="cuda")
    Bt = torch.zeros((8, 64), dtype=torch.uint8, device="cuda")
    C = torch.zeros((0, 8), dtype=torch.int32, device="cuda")
    q4.q4_gemm(A, Bt, C, 0, 8, 128, 0, 0)
    assert q4.q4_last_device_status() == q4.Q4_OK


def test_pack_bt_matches_oracle(q4):
    import torch
    rng = np.random.default_rng(3)
    for K, N in [(7, 5), (32, 64), (33, 18), (300, 130)]:
        b_kn = oracle.pack_rows(rng.integers(0, 16, (K, N), dtype=np.uint8))
        ldb = (K + 1) // 2 + 2
        want = oracle.pack_bt(b_kn, K, N, ldb)
        Bt = torch.full((N, ldb), 0xA5, dtype=torch.uint8, device="cuda")
        q4.q4_pack_bt(dev(b_kn), Bt, K, N)
        assert (Bt.cpu().numpy() == want).all()


def test_host_entry_point(q4):
    import torch
    c = aligned_case(300, 200, 520, seed=12)
    hA, hBt = torch.from_numpy(c.A).pin_memory(), torch.from_numpy(c.Bt).pin_memory()
    hC = torch.zeros((c.M, c.N), dtype=torch.int32).pin_memory()
    need = q4.q4_gemm_host_staging_bytes(c.M, c.N, c.K, c.lda, c.ldb, c.N)
    staging = torch.empty(need, dtype=torch.uint8, device="cuda")
    q4.q4_set_variant(0)
    q4.q4_gemm_host(hA, hBt, hC, c.M, c.N, c.K, c.za, c.zb, staging)
    assert (hC.numpy() == oracle.gemm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb)).all()
    # several row slices over the two streams (slices of 1024 rows, a ragged last one), int32
    # pitch wider than a row: the padding on the host stays as it was
    c = aligned_case(2500, 264, 200, seed=13)
    hA, hBt = torch.from_numpy(c.A).pin_memory(), torch.from_numpy(c.Bt).pin_memory()
    hC = torch.full((c.M, c.N + 4), -7, dtype=torch.int32).pin_memory()
    staging = torch.full((q4.q4_gemm_host_staging_bytes(c.M, c.N, c.K, c.lda, c.ldb, c.N + 4),), 0xA5,
                         dtype=torch.uint8, device="cuda")
    for _ in range(2):          # the second call finds the first call's leftovers in the staging buffer
        q4.q4_gemm_host(hA, hBt, hC, c.M, c.N, c.K, c.za, c.zb, staging)
        assert q4.q4_last_device_status() == q4.Q4_OK
        assert (hC.numpy()[:, :c.N] == oracle.gemm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb)).all()
        assert (hC.numpy()[:, c.N:] == -7).all()
