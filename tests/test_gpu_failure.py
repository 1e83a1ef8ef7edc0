"""Failure reporting and ordering checks on the GPU, without any fault or hang: a bounded
device-side wait that runs out is reported once through q4_last_device_status and leaves the
context usable; calls issued on two streams at once give the oracle's results."""
import numpy as np
import pytest

import oracle
from paper_2009_06488_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q4():
    from paper_2009_06488_b200 import binding
    return binding


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def small_gemm_ok(q4):
    import torch
    c = wl.gemm_case("after", 200, 136, 520, seed=3, lda=272, ldb=272)
    C = torch.empty((c.M, c.N), dtype=torch.int32, device="cuda")
    q4.q4_gemm(dev(c.A), dev(c.Bt), C, c.M, c.N, c.K, c.za, c.zb)
    return (C.cpu().numpy() == oracle.gemm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb)).all()


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable(q4):
    import torch
    assert q4.q4_last_device_status() == q4.Q4_OK        # nothing pending from earlier tests
    outcome = torch.zeros(1, dtype=torch.int32, device="cuda")
    q4.q4_selftest_wait_timeout(outcome)
    assert q4.q4_last_device_status() == q4.Q4_ERR_DEVICE_TIMEOUT
    assert int(outcome.item()) == 2                      # the wait gave up; it did not complete
    assert q4.q4_last_device_status() == q4.Q4_OK        # the flag is cleared by reading it
    assert small_gemm_ok(q4)
    assert q4.q4_last_device_status() == q4.Q4_OK


def test_calls_on_two_streams_at_once(q4):
    import torch
    cases = [wl.gemm_case(f"s{i}", 640 + 128 * i, 448, 1536, seed=40 + i, lda=768, ldb=768) for i in range(2)]
    net = wl.c3(batch=8)
    L = net.layers[0]
    args = (L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
    d = q4.ConvDesc(*args)
    X, Wt = dev(net.X), dev(L.Wt)
    streams = [torch.cuda.Stream() for _ in range(2)]
    outs, convs = [], []
    torch.cuda.synchronize()
    for rep in range(3):                                  # repeat: ordering bugs show as differences between runs
        for c, st in zip(cases, streams):
            with torch.cuda.stream(st):
                A, Bt = dev(c.A), dev(c.Bt)
                C = torch.full((c.M, c.N), -1, dtype=torch.int32, device="cuda")
                ws = torch.empty(q4.q4_gemm_workspace_bytes(c.M, c.N, c.K), dtype=torch.uint8, device="cuda")
                q4.q4_gemm(A, Bt, C, c.M, c.N, c.K, c.za, c.zb, ws=ws)
                Y = torch.full((d.M, L.OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
                wsc = torch.empty(q4.q4_conv2d_workspace_bytes(d), dtype=torch.uint8, device="cuda")
                q4.q4_conv2d(X, Wt, d, L.za, L.zb, q4.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi), Y, wsc)
                outs.append((c, C, A, Bt, ws))
                convs.append((Y, wsc))
    torch.cuda.synchronize()
    wantY = oracle.conv2d(net.X, L.Wt, None, oracle.ConvDesc(*args), L.za, L.zb,
                          oracle.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi))
    want = {c.name: oracle.gemm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb) for c in cases}
    for c, C, *_ in outs:
        assert (C.cpu().numpy() == want[c.name]).all()
    for Y, _ in convs:
        assert (Y.cpu().numpy() == wantY).all()
    assert q4.q4_last_device_status() == q4.Q4_OK
