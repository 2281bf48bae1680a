"""The benchmark's other workloads: sparsity sweep, format sweep, dense shape sweep and the 32-layer stack.

Used by ``bench.py --config sweep|formats|dense|stack`` (and, in reduced form, by its default line).
Each case packs several distinct weight copies (together well above the 126 MB L2), visits them
round-robin inside one CUDA graph and times graph replays with CUDA events on the launching stream.
Weights are random-init on the device (their values do not affect timing); x and thresholds come
from the seeded input module.
"""
from __future__ import annotations

import json
import math
import os

import numpy as np
import torch

from . import binding, calibrate, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
L2_BYTES = 126e6


def hbm_peak():
    """(GB/s, "measured" | "fallback"): the measured copy bandwidth of this machine's B200s."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def needed_bytes(m, n, count, bits, group):
    """Algorithmic bytes of one GEMV: the active blocks with their scale and zero, x, the list, y."""
    R, B = m // group, group * bits // 8
    return count * R * (B + 4) + 2 * n + 4 * count + 4 + 2 * m


def graph_us(fn, calls, replays=20):
    """(median, min) device microseconds per call of `calls` calls captured in one graph."""
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
    return float(np.median(ts)), float(np.min(ts))


def make_copies(m, n, bits, group, copies, seed0=0):
    g = torch.Generator(device="cuda")
    out = []
    for c in range(copies):
        g.manual_seed(seed0 + c)
        W = torch.empty((m, n), dtype=torch.float32, device="cuda").normal_(0.0, 0.02, generator=g).half()
        out.append(binding.spqt_pack(W, bits, group))
        del W
    return out


def copies_for(m, n, bits, group, at_least=4, at_most=160):
    """Distinct packed copies so that the bytes between two visits of a copy exceed twice the L2."""
    size = (m // group) * n * (group * bits // 8 + 4)
    return int(min(at_most, max(at_least, math.ceil(2.4 * L2_BYTES / size))))


def run_case(m, n, bits, group, sparsities, x, copies, peak, unbalanced=False):
    """Sparse (given list), fused (list collected in the same launch) and dense GEMV on `copies` rotated
    packed matrices, for every sparsity."""
    packs = make_copies(m, n, bits, group, copies)
    xd = torch.from_numpy(x).cuda()
    ws = binding.new_workspace(m, n, bits, group)
    y = torch.empty(m, dtype=torch.float16, device="cuda")
    idx = torch.empty(n, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    calls = max(copies, 16)
    t_dense, _ = graph_us(lambda i, s: binding.spqt_dense_gemv(packs[i % copies], xd, ws, y, stream=s), calls)
    rows = []
    for sp in sparsities:
        t = inputs.threshold_for_sparsity(x, sp)
        binding.spqt_sparsify(xd, t, idx, cnt)
        torch.cuda.synchronize()
        count = int(cnt.item())
        t_sparse, _ = graph_us(lambda i, s: binding.spqt_sparse_gemv(packs[i % copies], xd, idx, cnt, ws, y, stream=s), calls)
        t_fused, _ = graph_us(lambda i, s: binding.spqt_sparsify_gemv(packs[i % copies], xd, t, ws, idx, cnt, y, stream=s), calls)
        nb = needed_bytes(m, n, count, bits, group)
        row = {"m": m, "n": n, "bits": bits, "group": group, "sparsity": 1.0 - count / n, "count": count,
               "copies": copies, "sparse_us": t_sparse, "fused_us": t_fused, "dense_us": t_dense,
               "sparse_gbs": nb / t_sparse * 1e-3, "frac_of_peak": nb / t_sparse * 1e-3 / peak,
               "fused_gbs": (nb + 2 * n + 4 * count + 4) / t_fused * 1e-3,
               "fused_frac_of_peak": (nb + 2 * n + 4 * count + 4) / t_fused * 1e-3 / peak,
               "dense_gbs": needed_bytes(m, n, n, bits, group) / t_dense * 1e-3,
               "dense_frac_of_peak": needed_bytes(m, n, n, bits, group) / t_dense * 1e-3 / peak,
               "speedup_vs_dense": t_dense / t_sparse, "fused_speedup_vs_dense": t_dense / t_fused,
               "ideal": 1.0 / max(1e-9, count / n)}
        if unbalanced:
            try:
                binding.spqt_set_tuning(0, 4)   # static column partition, no load balancing
                t_unb, _ = graph_us(lambda i, s: binding.spqt_sparsify_gemv(packs[i % copies], xd, t, ws, idx, cnt, y, stream=s), calls)
            finally:
                binding.spqt_set_tuning(0, 0)
            row["unbalanced_us"] = t_unb
            row["unbalanced_speedup_vs_dense"] = t_dense / t_unb
        rows.append(row)
    status = binding.spqt_workspace_status(ws, m, group)
    for r in rows:
        r["device_status"] = status
    del packs
    torch.cuda.empty_cache()
    return rows


def sparsity_sweep(peak, sparsities=None, copies=64, unbalanced=False):
    """0-90 % on a 14336 -> 4096 down-projection and a 4096 -> 14336 up-projection, int4 g128, 64 rotated copies."""
    sps = sparsities if sparsities is not None else [i / 10 for i in range(10)]
    out = []
    for (m, n, dist) in [(4096, 14336, "gauss"), (14336, 4096, "laplace")]:
        x = inputs.activations(n, seed=3, dist=dist)
        out += run_case(m, n, 4, 128, sps, x, copies, peak, unbalanced=unbalanced)
    return out


def format_sweep(peak, shapes=None, formats=None):
    """Llama-2-70B-shaped linears x {int4, int3} x {g128, g64} at 50 %, x with 1 % outliers x20."""
    out = []
    for (name, m, n, dist) in (shapes if shapes is not None else inputs.LLAMA2_70B_LINEARS):
        x = inputs.activations(n, seed=5, dist=dist, outlier_frac=0.01, outlier_scale=20.0)
        for (bits, group) in (formats if formats is not None else [(4, 128), (4, 64), (3, 128), (3, 64)]):
            out += run_case(m, n, bits, group, [0.5], x, copies_for(m, n, bits, group, at_least=4, at_most=16), peak)
    return out


def model_shapes_sweep(peak):
    """The GEMV shapes of three model sizes at the paper's three sparsity levels (its GEMV-level experiment,
    Sec. 6): Llama-3-8B-, Llama-2-13B- and Llama-2-70B-shaped linears, int4 g128, 25 / 40 / 50 %."""
    shapes = [("8b q,o", 4096, 4096, "laplace"), ("8b gate,up", 14336, 4096, "laplace"), ("8b down", 4096, 14336, "gauss"),
              ("13b q,k,v,o", 5120, 5120, "laplace"), ("13b gate,up", 13824, 5120, "laplace"), ("13b down", 5120, 13824, "gauss"),
              ("70b q,o", 8192, 8192, "laplace"), ("70b gate,up", 28672, 8192, "laplace"), ("70b down", 8192, 28672, "gauss")]
    out = []
    for (name, m, n, dist) in shapes:
        x = inputs.activations(n, seed=7, dist=dist)
        rows = run_case(m, n, 4, 128, [0.25, 0.4, 0.5], x, copies_for(m, n, 4, 128, at_least=4, at_most=40), peak)
        for r in rows:
            r["shape"] = name
        out += rows
    return out


def dense_shape_sweep(peak):
    """The dense zigzag GEMV on the paper's 15 shapes m in {2048, 4096, 8192} x k in {1024 ... 16384}
    (its hyper-parameter study, Sec. 6), int4 g128, over the CTA counts the autotuner would try, and the
    row-wise-layout baseline on the same shapes (the comparison the paper makes there)."""
    out = []
    for m in (2048, 4096, 8192):
        for n in (1024, 2048, 4096, 8192, 16384):
            copies = copies_for(m, n, 4, 128)
            packs = make_copies(m, n, 4, 128, copies)
            xd = torch.from_numpy(inputs.activations(n, seed=11)).cuda()
            ws = binding.new_workspace(m, n, 4, 128)
            y = torch.empty(m, dtype=torch.float16, device="cuda")
            calls = max(copies, 16)
            row = {"m": m, "n": n, "copies": copies}
            best = None
            for ctas in (0, 64, 96, 128, 148):
                try:
                    binding.spqt_set_tuning(ctas, 0)
                    us, _ = graph_us(lambda i, s: binding.spqt_dense_gemv(packs[i % copies], xd, ws, y, stream=s), calls, replays=10)
                finally:
                    binding.spqt_set_tuning(0, 0)
                row["us_ctas_%d" % ctas] = us
                if best is None or us < best[1]:
                    best = (ctas, us)
            row["best_ctas"], row["best_us"] = best
            row["dense_gbs"] = needed_bytes(m, n, n, 4, 128) / best[1] * 1e-3
            row["frac_of_peak"] = row["dense_gbs"] / peak
            del packs
            # the comparison baseline: the same weights' distribution in the row-wise layout, row-parallel kernel
            g = torch.Generator(device="cuda")
            rw = []
            for c in range(copies):
                g.manual_seed(c)
                W = torch.empty((m, n), dtype=torch.float32, device="cuda").normal_(0.0, 0.02, generator=g).half()
                rw.append(binding.spqt_rowwise_pack(W, 4, 128))
                del W
            us_rw, _ = graph_us(lambda i, s: binding.spqt_rowwise_dense_gemv(rw[i % copies], xd, y, stream=s), calls, replays=10)
            row["rowwise_us"] = us_rw
            row["rowwise_gbs"] = needed_bytes(m, n, n, 4, 128) / us_rw * 1e-3
            row["rowwise_frac_of_peak"] = row["rowwise_gbs"] / peak
            row["zigzag_dense_vs_rowwise"] = us_rw / row["us_ctas_0"]
            # activation sparsity on each layout at 50 %: the row-wise kernel with the inactive entries zeroed
            # (it reads every byte), the zigzag kernel over the list (collected in the same launch)
            x50 = inputs.activations(n, seed=11)
            t50 = inputs.threshold_for_sparsity(x50, 0.5)
            us_rw_t, _ = graph_us(lambda i, s: binding.spqt_rowwise_thresholded_gemv(rw[i % copies], xd, t50, y, stream=s), calls, replays=10)
            zz = make_copies(m, n, 4, 128, copies)
            idx = torch.empty(n, dtype=torch.int32, device="cuda")
            cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
            us_zz_s, _ = graph_us(lambda i, s: binding.spqt_sparsify_gemv(zz[i % copies], xd, t50, ws, idx, cnt, y, stream=s), calls, replays=10)
            del zz
            row["rowwise_thresholded_us"] = us_rw_t
            row["rowwise_sparse_speedup_over_its_dense"] = us_rw / us_rw_t
            row["zigzag_sparse_us"] = us_zz_s
            row["zigzag_sparse_speedup_over_its_dense"] = row["us_ctas_0"] / us_zz_s
            out.append(row)
            del rw
            torch.cuda.empty_cache()
    return out


def kq_sweep(peak):
    """The two-level format (one record per 256 rows of a column): the index collection followed by the sparse
    product over the list at 50 %, the product alone, and the dense product, on Llama-3-8B-shaped linears and one
    Llama-2-70B-shaped one with 4-bit codes, and with 2- and 8-bit codes on the two largest.  Needed bytes per
    active superblock: the record, 144 bytes (80, 176, 208 and 272 with 2-, 5-, 6- and 8-bit codes)."""
    out = []
    cases = [(4096, 4096, "laplace", 4), (6144, 4096, "laplace", 4), (28672, 4096, "laplace", 4), (4096, 14336, "gauss", 4),
             (28672, 8192, "laplace", 4),
             # the other code widths, on the two large shapes
             (28672, 4096, "laplace", 2), (28672, 4096, "laplace", 8), (28672, 8192, "laplace", 2), (28672, 8192, "laplace", 5),
             (28672, 8192, "laplace", 6), (28672, 8192, "laplace", 8)]
    for (m, n, dist, bits) in cases:
        R = m // 256
        rec = 256 * bits // 8 + 16
        copies = int(min(64, max(4, math.ceil(2.4 * L2_BYTES / (R * n * rec)))))
        g = torch.Generator(device="cuda")
        packs = []
        for c in range(copies):
            g.manual_seed(c)
            W = torch.empty((m, n), dtype=torch.float32, device="cuda").normal_(0.0, 0.02, generator=g).half()
            packs.append(binding.spqt_kqw_pack(W, bits))
            del W
        x = inputs.activations(n, seed=21, dist=dist)
        t = inputs.threshold_for_sparsity(x, 0.5)
        xd = torch.from_numpy(x).cuda()
        ws = binding.new_kq_workspace(packs[0])
        idx, cnt = binding.spqt_sparsify(xd, t)
        torch.cuda.synchronize()
        count = int(cnt.item())
        y = torch.empty(m, dtype=torch.float16, device="cuda")
        calls = max(copies, 16)

        def both(i, s):
            binding.spqt_sparsify(xd, t, idx, cnt, stream=s)
            binding.spqt_kqw_sparse_gemv(packs[i % copies], xd, idx, cnt, ws, y, stream=s)
        us_both, _ = graph_us(both, calls)
        us_sp, _ = graph_us(lambda i, s: binding.spqt_kqw_sparse_gemv(packs[i % copies], xd, idx, cnt, ws, y, stream=s), calls)
        us_de, _ = graph_us(lambda i, s: binding.spqt_kqw_dense_gemv(packs[i % copies], xd, ws, y, stream=s), calls)
        nb = lambda c: c * R * rec + 2 * n + 4 * c + 4 + 2 * m
        out.append({"m": m, "n": n, "bits": bits, "count": count, "copies": copies, "sparsify_plus_sparse_us": us_both, "sparse_us": us_sp,
                    "dense_us": us_de, "sparse_gbs": nb(count) / us_sp * 1e-3, "frac_of_peak": nb(count) / us_sp * 1e-3 / peak,
                    "dense_gbs": nb(n) / us_de * 1e-3, "dense_frac_of_peak": nb(n) / us_de * 1e-3 / peak,
                    "speedup_vs_dense": us_de / us_sp, "speedup_vs_dense_with_index_collection": us_de / us_both})
        del packs
        torch.cuda.empty_cache()
    return out


def batch_sweep(peak):
    """Small batches (1, 2, 4, 8 rows) on the stacked gate|up matrix and the down projection, int4 g128: rows that
    are independent draws (their union is 1 - 2^-B dense at 50 % each) and rows that share most of their
    hidden state, as beams do (a common vector plus 20 % individual noise).  Sparse over the union, and dense."""
    out = []
    for (m, n, dist) in [(28672, 4096, "laplace"), (4096, 14336, "gauss")]:
        copies = copies_for(m, n, 4, 128)
        packs = make_copies(m, n, 4, 128, copies)
        calls = max(copies, 16)
        ws1 = binding.new_workspace(m, n, 4, 128)
        wsb = binding.new_gemm_small_workspace(packs[0])
        idx = torch.empty(n, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
        base = inputs.activations(n, seed=31, dist=dist).astype(np.float32)
        for kind in ("independent", "beam-like"):
            for batch in (1, 2, 4, 8):
                if kind == "independent":
                    X = np.stack([inputs.activations(n, seed=40 + b, dist=dist) for b in range(batch)])
                else:
                    X = np.stack([(base + 0.2 * inputs.activations(n, seed=60 + b, dist=dist).astype(np.float32)).astype(np.float16)
                                  for b in range(batch)])
                t = inputs.threshold_for_sparsity(X[0], 0.5)
                Xd = torch.from_numpy(X).cuda()
                Y = torch.empty((batch, m), dtype=torch.float16, device="cuda")
                if batch == 1:
                    us, _ = graph_us(lambda i, s: binding.spqt_sparsify_gemv(packs[i % copies], Xd[0], t, ws1, idx, cnt, Y[0], stream=s), calls)
                    us_d, _ = graph_us(lambda i, s: binding.spqt_dense_gemv(packs[i % copies], Xd[0], ws1, Y[0], stream=s), calls)
                else:
                    us, _ = graph_us(lambda i, s: binding.spqt_sparse_gemm_small(packs[i % copies], Xd, t, wsb, idx, cnt, Y, stream=s), calls)
                    us_d, _ = graph_us(lambda i, s: binding.spqt_dense_gemm_small(packs[i % copies], Xd, wsb, Y, stream=s), calls)
                torch.cuda.synchronize()
                count = int(cnt.item())
                nb = needed_bytes(m, n, count, 4, 128) + (batch - 1) * (2 * n + 2 * m)
                out.append({"m": m, "n": n, "rows": kind, "batch": batch, "union_count": count, "union_sparsity": 1.0 - count / n,
                            "sparse_us": us, "sparse_us_per_row": us / batch, "dense_us": us_d, "dense_us_per_row": us_d / batch,
                            "sparse_gbs": nb / us * 1e-3, "frac_of_peak": nb / us * 1e-3 / peak,
                            "speedup_vs_dense": us_d / us})
        del packs
        torch.cuda.empty_cache()
    return out


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
    pools = {}
    for i, (site, m, n, dist) in enumerate(STACK_SITES):
        calib = np.concatenate([inputs.activations(n, seed=9000 + 100 * i + c, dist=dist) for c in range(calib_vectors)])
        pools[site] = torch.from_numpy(calib).cuda()
        host = np.stack([inputs.activations(n, seed=20000 + 1000 * i + t, dist=dist) for t in range(tokens)])
        xs[site] = (host, torch.from_numpy(host).cuda())
    thr = calibrate.unified(pools, sparsity)     # one global level: every site's threshold from its own pool
    return packs, thr, xs


def run_stack(layers=32, tokens=100, peak=None):
    """Per-token pass over the linear layers of the whole stack: 4 launches per layer (index collection
    inside the GEMV), one CUDA graph per token, device-timed; tokens/s of the linear layers."""
    peak = peak or hbm_peak()[0]
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
           "needed_gbs": needed / ms_token * 1e-6, "frac_of_peak": needed / ms_token * 1e-6 / peak,
           "thresholds": thr,
           "realised_sparsity": {k: {"mean": float(np.mean(v)), "min": float(np.min(v)), "max": float(np.max(v))} for k, v in sp.items()},
           "packed_gb": sum(p.nbytes for row in packs for p in row.values()) * 1e-9,
           "device_status": status}
    del packs, graphs
    torch.cuda.empty_cache()
    return out
