"""Sparsity and format sweeps of the sparse GEMV against the same-layout dense GEMV.

    python -m paper_2511_04477_b200.sweep sparsity      # 0-90 % on 4096x14336 and 14336x4096, int4 g128
    python -m paper_2511_04477_b200.sweep formats       # Llama-2-70B-shaped linears x {int4,int3} x {g64,g128}, 50 %
    python -m paper_2511_04477_b200.sweep stack         # 32-layer Llama-3-8B-shaped stack, thresholds calibrated for 40 %

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


STACK_SITES = [  # (site, stacked matrix rows, n, distribution of the site's input)
    ("attn_in", 6144, 4096, "laplace"),    # q | k | v share x and idx
    ("attn_out", 4096, 4096, "laplace"),   # o
    ("mlp_in", 28672, 4096, "laplace"),    # gate | up
    ("mlp_mid", 4096, 14336, "gauss"),     # down
]


def build_stack(layers, tokens, sparsity=0.4, calib_vectors=64):
    """Packed weights of `layers` decoder layers (random-init on the device, one seed per matrix), per-site
    thresholds calibrated once on pooled calibration vectors, and `tokens` fresh inputs per site."""
    g = torch.Generator(device="cuda")
    packs, thr, xs = [], {}, {}
    for L in range(layers):
        row = {}
        for i, (site, m, n, _) in enumerate(STACK_SITES):
            g.manual_seed(L * 7 + i)
            W = torch.empty((m, n), dtype=torch.float32, device="cuda").normal_(0.0, 0.02, generator=g).half()
            row[site] = binding.spqt_pack(W, 4, 128)
            del W
        packs.append(row)
    for i, (site, m, n, dist) in enumerate(STACK_SITES):
        calib = [inputs.activations(n, seed=9000 + 100 * i + c, dist=dist) for c in range(calib_vectors)]
        thr[site] = inputs.pooled_threshold(calib, sparsity)
        host = np.stack([inputs.activations(n, seed=20000 + 1000 * i + t, dist=dist) for t in range(tokens)])
        xs[site] = (host, torch.from_numpy(host).cuda())
    return packs, thr, xs


def run_stack(layers=32, tokens=100, peak=None):
    """Per-token pass over the linear layers of the whole stack: 4 launches per layer (index collection
    inside the GEMV), one CUDA graph per token, device-timed; tokens/s of the linear layers."""
    packs, thr, xs = build_stack(layers, tokens)
    ws = {site: binding.new_workspace(m, n, 4, 128) for (site, m, n, _) in STACK_SITES}
    y = {site: torch.empty(m, dtype=torch.float16, device="cuda") for (site, m, n, _) in STACK_SITES}
    idx = {site: torch.empty(n, dtype=torch.int32, device="cuda") for (site, m, n, _) in STACK_SITES}
    cnt = {site: torch.zeros(1, dtype=torch.int32, device="cuda") for (site, m, n, _) in STACK_SITES}
    s = torch.cuda.Stream()

    def token_pass(t, stream):
        for L in range(layers):
            for (site, m, n, _) in STACK_SITES:
                binding.spqt_sparsify_gemv(packs[L][site], xs[site][1][t], thr[site], ws[site], idx[site], cnt[site],
                                           y[site], stream=stream)

    with torch.cuda.stream(s):
        token_pass(0, s)
    torch.cuda.synchronize()
    graphs = []
    for t in range(tokens):
        gph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gph, stream=s):
            token_pass(t, s)
        graphs.append(gph)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(s):
        for gph in graphs[:3]:
            gph.replay()
        e0.record(s)
        for gph in graphs:
            gph.replay()
        e1.record(s)
        e1.synchronize()
    ms_token = e0.elapsed_time(e1) / tokens
    sp = {site: [inputs.realised_sparsity(xs[site][0][t], thr[site]) for t in range(tokens)] for (site, _, _, _) in STACK_SITES}
    needed = 0
    for (site, m, n, _) in STACK_SITES:
        counts = [int(round((1.0 - v) * n)) for v in sp[site]]
        needed += layers * float(np.mean([needed_bytes(m, n, c, 4, 128) + 2 * n + 4 * c + 4 for c in counts]))
    status = max(binding.spqt_workspace_status(ws[site], m, 128) for (site, m, n, _) in STACK_SITES)
    out = {"layers": layers, "tokens": tokens, "ms_per_token": ms_token, "tokens_per_s": 1e3 / ms_token,
           "launches_per_token": 4 * layers, "needed_gb_per_token": needed * 1e-9,
           "needed_gbs": needed / ms_token * 1e-6, "pct_of_measured_peak": 100 * needed / ms_token * 1e-6 / (peak or _peak()),
           "thresholds": thr,
           "realised_sparsity": {k: {"mean": float(np.mean(v)), "min": float(np.min(v)), "max": float(np.max(v))} for k, v in sp.items()},
           "packed_gb": sum(p.nbytes for row in packs for p in row.values()) * 1e-9,
           "device_status": status}
    return out


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
    elif which == "stack":
        res = run_stack(peak=peak)
        print("32-layer stack: %.3f ms per token over the linear layers, %.0f tokens/s, %d launches per token, "
              "%.2f GB needed per token (%.0f GB/s, %.1f %% of the measured HBM peak); realised sparsity %s" % (
                  res["ms_per_token"], res["tokens_per_s"], res["launches_per_token"], res["needed_gb_per_token"],
                  res["needed_gbs"], res["pct_of_measured_peak"],
                  {k: "%.3f (%.3f-%.3f)" % (v["mean"], v["min"], v["max"]) for k, v in res["realised_sparsity"].items()}))
        print(json.dumps({"sweep": which, "hbm_peak_gbs": peak, "result": res}))
        return
    else:
        raise SystemExit("usage: python -m paper_2511_04477_b200.sweep [sparsity|formats|stack]")
    show(out)
    print(json.dumps({"sweep": which, "hbm_peak_gbs": peak, "rows": out}))


if __name__ == "__main__":
    main(sys.argv[1:])
