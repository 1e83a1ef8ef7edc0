"""q4_conv2d_static: the convolution entry point for callers that cannot allocate
device memory (no cudaMalloc available to them: a plugin without an allocator, a
fixed-pool process, a loop whose owner forbids allocator calls).  Its scratch is a
fixed array inside the library, shared by all calls, so the check is: same bytes as
q4_conv2d with a caller-provided workspace, on two calls in a row with different
layers (the second call finds the first call's leftovers in the array).

Collected last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest

from paper_2009_06488_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def layer(seed, N, H, W, C, OC, k, s, p):
    Wt = wl.rand_packed(seed, 2, OC, k * k * C)
    bias = wl.rand_ints(seed, 3, -512, 512, OC).astype(np.int32)
    return wl.ConvLayer("t", N, H, W, C, OC, k, k, s, p, 8, 7, Wt, bias, (1 << 30) + 77, 4, 3, 3, 15), \
        wl.rand_flat_nibbles(seed, 1, N * H * W * C)


def test_static_scratch_entry_point_matches_q4_conv2d_twice_in_a_row():
    import torch
    from paper_2009_06488_b200 import binding as q4
    q4.q4_set_variant(0)
    # second layer is smaller and has another pitch: stale bytes of the first call
    # lie beyond and between its rows
    for seed, geom in ((900, (4, 32, 32, 16, 32, 3, 1, 1)), (901, (3, 17, 13, 8, 16, 3, 2, 1))):
        L, X = layer(seed, *geom)
        d = q4.ConvDesc(L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
        rq = q4.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi)
        Xd, Wd, bd = dev(X), dev(L.Wt), dev(L.bias)
        assert q4.q4_conv2d_workspace_bytes(d) <= q4.Q4_STATIC_SCRATCH_BYTES
        ws = torch.empty(q4.q4_conv2d_workspace_bytes(d), dtype=torch.uint8, device="cuda")
        want = torch.full((d.M, L.OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
        q4.q4_conv2d(Xd, Wd, d, L.za, L.zb, rq, want, ws, bd)
        got = torch.full((d.M, L.OC // 2), 0x5A, dtype=torch.uint8, device="cuda")
        q4.q4_conv2d_static(Xd, Wd, d, L.za, L.zb, rq, got, bd)
        torch.cuda.synchronize()
        assert q4.q4_last_device_status() == q4.Q4_OK
        assert torch.equal(got, want)          # integer path: bit-exact
        assert len(torch.unique(got)) > 3


def test_static_scratch_rejects_layers_beyond_its_size():
    import torch
    from paper_2009_06488_b200 import binding as q4
    L, X = layer(902, 256, 32, 32, 16, 32, 3, 1, 1)       # needs ~21 MB of scratch
    d = q4.ConvDesc(L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
    assert q4.q4_conv2d_workspace_bytes(d) > q4.Q4_STATIC_SCRATCH_BYTES
    Y = torch.zeros((d.M, L.OC // 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_conv2d_static(dev(X), dev(L.Wt), d, L.za, L.zb,
                            q4.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi), Y)
    assert e.value.status == q4.Q4_ERR_STATIC_SCRATCH
    assert "static" in str(e.value)
    assert int(Y.sum()) == 0                   # nothing was launched
