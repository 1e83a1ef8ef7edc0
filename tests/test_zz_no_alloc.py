"""q4_conv2d_static: the convolution entry point for callers that cannot allocate
device memory (no cudaMalloc available to them: a plugin without an allocator, a
fixed-pool process, a loop whose owner forbids allocator calls).  Its scratch -- the
unrolled matrix and its row sums -- is a fixed array inside the library, shared by all
calls.  The layers here are ones the single-kernel fused path does not take (six and
seventy-two output channels, a 1x1 layer), so every call really unrolls into that array
and multiplies from it; the checks are the oracle's bytes and q4_conv2d's bytes with a
caller-provided workspace, on calls in a row with different layers (each later call
finds the earlier calls' leftovers in the array, beyond and between its own rows).

Collected last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest

import oracle
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


# N, H, W, C, OC, k, stride, pad -- a large layer first, then smaller ones with other
# pitches and row counts; the last is a 1x1 layer large enough for the big-GEMM kernel: its
# unrolled matrix is the input itself, and at this size the kernel takes the depth sums
# itself, so the call is a single launch that must leave the array alone and still agree
LAYERS = ((900, (6, 32, 32, 16, 72, 3, 1, 1)),
          (901, (3, 17, 13, 8, 6, 3, 2, 1)),
          (902, (2, 9, 11, 3, 6, 5, 1, 2)),
          (903, (74, 16, 16, 32, 400, 1, 1, 0)))


def test_static_scratch_entry_point_matches_oracle_and_q4_conv2d_on_calls_in_a_row():
    import torch
    from paper_2009_06488_b200 import binding as q4
    q4.q4_set_variant(0)
    for seed, geom in LAYERS:
        L, X = layer(seed, *geom)
        args = (L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
        d = q4.ConvDesc(*args)
        rq = q4.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi)
        Xd, Wd, bd = dev(X), dev(L.Wt), dev(L.bias)
        assert q4.q4_conv2d_workspace_bytes(d) <= q4.Q4_STATIC_SCRATCH_BYTES
        ws = torch.empty(q4.q4_conv2d_workspace_bytes(d), dtype=torch.uint8, device="cuda")
        other = torch.full((d.M, L.OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
        q4.q4_conv2d(Xd, Wd, d, L.za, L.zb, rq, other, ws, bd)
        got = torch.full((d.M, L.OC // 2), 0x5A, dtype=torch.uint8, device="cuda")
        n0 = q4.q4_launch_count()
        q4.q4_conv2d_static(Xd, Wd, d, L.za, L.zb, rq, got, bd)
        # more than one kernel: the scratch array was written (the unrolled matrix and its row
        # sums) and read back; a 1x1 layer has nothing to unroll
        assert q4.q4_launch_count() - n0 >= (1 if L.KH == 1 else 2)
        torch.cuda.synchronize()
        assert q4.q4_last_device_status() == q4.Q4_OK
        want = oracle.conv2d(X, L.Wt, L.bias, oracle.ConvDesc(*args), L.za, L.zb,
                             oracle.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi))
        assert (got.cpu().numpy() == want).all()      # integer path: bit-exact
        assert torch.equal(got, other)
        assert len(np.unique(want)) > 3


def test_static_scratch_rejects_layers_beyond_its_size():
    import torch
    from paper_2009_06488_b200 import binding as q4
    L, X = layer(904, 256, 32, 32, 16, 32, 3, 1, 1)       # needs ~21 MB of scratch
    d = q4.ConvDesc(L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
    assert q4.q4_conv2d_workspace_bytes(d) > q4.Q4_STATIC_SCRATCH_BYTES
    Y = torch.zeros((d.M, L.OC // 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_conv2d_static(dev(X), dev(L.Wt), d, L.za, L.zb,
                            q4.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi), Y)
    assert e.value.status == q4.Q4_ERR_STATIC_SCRATCH
    assert "static" in str(e.value)
    assert int(Y.sum()) == 0                   # nothing was launched
