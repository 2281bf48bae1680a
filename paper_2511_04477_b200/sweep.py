"""Sparsity and format sweeps of the sparse GEMV against the same-layout dense GEMV.

    python -m paper_2511_04477_b200.sweep sparsity      # 0-90 % on 4096x14336 and 14336x4096, int4 g128
    python -m paper_2511_04477_b200.sweep formats       # Llama-2-70B-shaped linears x {int4,int3} x {g64,g128}, 50 %

Each case packs several distinct weight copies (together well above the 126 MB L2), visits them
round-robin inside one CUDA graph and times graph replays with CUDA events.  Printed per case: device
microseconds per call, effective GB/s over the bytes the method needs, percent of the measured HBM
peak, speed-up over the dense GEMV on the same packed buffers, and the ideal 1/(1 - sparsity).
Weights are random-init on the device; x and thresholds come from the seeded input module.
"""
from __future__ import annotations

import json
import math
import os
import sys

import numpy as np
import torch

from . import binding, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return 6650.0


def needed_bytes(m, n, count, bits, group):
    R, B = m // group, group * bits // 8
    return count * R * (B + 4) + 2 * n + 4 * count + 4 + 2 * m


def graph_us(fn, calls, replays=20):
    """Median device time per call of `calls` calls captured in one graph."""
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for i in range(min(calls, 4)):
            fn(i, s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        for i in range(calls):
            fn(i, s)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    with torch.cuda.stream(s):
        g.replay()
        for _ in range(replays):
            e0.record(s)
            g.replay()
            e1.record(s)
            e1.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3 / calls)
    return float(np.median(ts))


def make_copies(m, n, bits, group, copies):
    g = torch.Generator(device="cuda")
    out = []
    for c in range(copies):
        g.manual_seed(c)
        W = torch.empty((m, n), dtype=torch.float32, device="cuda").normal_(0.0, 0.02, generator=g).half()
        out.append(binding.spqt_pack(W, bits, group))
        del W
    return out


def run_case(m, n, bits, group, sparsities, x, copies, peak):
    packs = make_copies(m, n, bits, group, copies)
    xd = torch.from_numpy(x).cuda()
    ws = binding.new_workspace(m, n, bits, group)
    y = torch.empty(m, dtype=torch.float16, device="cuda")
    idx = torch.empty(n, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    calls = max(copies, 16)
    t_dense = graph_us(lambda i, s: binding.spqt_dense_gemv(packs[i % copies], xd, ws, y, stream=s), calls)
    rows = []
    for sp in sparsities:
        t = inputs.threshold_for_sparsity(x, sp)
        binding.spqt_sparsify(xd, t, idx, cnt)
        torch.cuda.synchronize()
        count = int(cnt.item())
        t_sparse = graph_us(lambda i, s: binding.spqt_sparse_gemv(packs[i % copies], xd, idx, cnt, ws, y, stream=s), calls)
        t_fused = graph_us(lambda i, s: binding.spqt_sparsify_gemv(packs[i % copies], xd, t, ws, idx, cnt, y, stream=s), calls)
        nb = needed_bytes(m, n, count, bits, group)
        rows.append({"m": m, "n": n, "bits": bits, "group": group, "sparsity": 1.0 - count / n, "count": count,
                     "sparse_us": t_sparse, "fused_us": t_fused, "dense_us": t_dense,
                     "sparse_gbs": nb / t_sparse * 1e-3, "pct_of_measured_peak": 100 * nb / t_sparse * 1e-3 / peak,
                     "dense_gbs": needed_bytes(m, n, n, bits, group) / t_dense * 1e-3,
                     "speedup_vs_dense": t_dense / t_sparse, "ideal": 1.0 / max(1e-9, count / n)})
    del packs
    torch.cuda.empty_cache()
    return rows


def show(rows):
    print("| m x n | fmt | sparsity | sparse us | +idx us | dense us | GB/s needed | % peak | x dense | ideal |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print("| %dx%d | int%d g%d | %.1f%% | %.2f | %.2f | %.2f | %.0f | %.1f | %.2f | %.2f |" % (
            r["m"], r["n"], r["bits"], r["group"], 100 * r["sparsity"], r["sparse_us"], r["fused_us"], r["dense_us"],
            r["sparse_gbs"], r["pct_of_measured_peak"], r["speedup_vs_dense"], r["ideal"]), flush=True)


def copies_for(m, n, bits, group):
    size = (m // group) * n * (group * bits // 8 + 4)
    return int(min(64, max(4, math.ceil(512e6 / size))))


def main(argv):
    which = argv[0] if argv else "sparsity"
    peak = _peak()
    binding.lib()
    out = []
    if which == "sparsity":
        for (m, n, dist) in [(4096, 14336, "gauss"), (14336, 4096, "laplace")]:
            x = inputs.activations(n, seed=3, dist=dist)
            sps = [i / 10 for i in range(10)]
            out += run_case(m, n, 4, 128, sps, x, copies_for(m, n, 4, 128), peak)
    elif which == "formats":
        for (name, m, n, dist) in inputs.LLAMA2_70B_LINEARS:
            x = inputs.activations(n, seed=5, dist=dist, outlier_frac=0.01, outlier_scale=20.0)
            for bits in (4, 3):
                for group in (128, 64):
                    out += run_case(m, n, bits, group, [0.5], x, copies_for(m, n, bits, group), peak)
    else:
        raise SystemExit("usage: python -m paper_2511_04477_b200.sweep [sparsity|formats]")
    show(out)
    print(json.dumps({"sweep": which, "hbm_peak_gbs": peak, "rows": out}))


if __name__ == "__main__":
    main(sys.argv[1:])
