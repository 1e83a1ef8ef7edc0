"""Writes paper_2009_06488_b200/requant_calibration.json (read by workloads.py): per-layer (mult, shift) for the conv
workloads c3 and c4, chosen from the CPU oracle's int32 accumulators on a small
batch so that the 4-bit outputs spread over their range instead of saturating.

The stored values are *inputs* of the workloads (the workload statement gives no
multipliers for these layers).  This script calls only the oracle and the input
generators; run it from the repository root:  python tests/golden/make_requant_calibration.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from oracle import ConvDesc, Requant  # noqa: E402
from paper_2009_06488_b200 import workloads as wl  # noqa: E402


def calibrate(net: wl.ConvNet) -> list[dict]:
    out = []
    X = net.X
    for L in net.layers:
        d = ConvDesc(L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
        acc = oracle.conv2d_direct(X, L.Wt, d, L.za, L.zb).astype(np.int64)
        if L.bias is not None:
            acc += L.bias.astype(np.int64)
        top = int(acc.max())
        span = max(1, 15 - L.zo)
        real = min(0.499, 0.8 * span / top) if top > 0 else 2.0 ** -8
        mult, shift = wl.requant_from_real(real)
        out.append({"layer": L.name, "mult": mult, "shift": shift, "acc_max": top,
                    "acc_min": int(acc.min())})
        rq = Requant(mult, shift, L.zo, L.clamp_lo, L.clamp_hi)
        X = oracle.conv2d(X, L.Wt, L.bias, d, L.za, L.zb, rq).reshape(-1)
    return out


def main():
    table = {"c3": calibrate(wl.c3(batch=4, requant=(1 << 30, 6)))}
    for seed in (4000, 4001, 4002):
        table[f"c4_seed{seed}"] = calibrate(wl.c4(batch=8, seed=seed, requant=[(1 << 30, 5)] * 5))
    table["c4_centred"] = calibrate(wl.c4(batch=8, seed=4000, centred=True,
                                          requant=[(1 << 30, 5)] * 5))
    path = os.path.join(ROOT, "paper_2009_06488_b200", "requant_calibration.json")
    with open(path, "w") as f:
        json.dump(table, f, indent=1)
        f.write("\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
