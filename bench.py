#!/usr/bin/env python
"""Benchmark of the SpQt hot path on B200: one line of JSON on stdout.

    python bench.py [--gpus N] [--steps K] [--warmup W]            the headline line (config "layer")
    python bench.py --config sweep | formats | dense | batch | kquant | models | stack   the other workloads, one JSON line each
    python bench.py --impl reference                               the fp64 CPU oracle on a bounded sample

Workload of the headline line (the configuration the metric is quoted on): the seven linear layers of
one Llama-3-8B-shaped decoder layer at batch 1 -- q, k, v, o (4096->4096, 4096->1024 x2, 4096->4096),
gate/up (4096->14336), down (14336->4096) -- INT4 codes, group 128, fp16 scale and zero, zigzag layout,
50 % activation sparsity.  A *step* is one pass over those seven matrices: four index collections
(attention input shared by q,k,v; attention output for o; MLP input shared by gate,up; MLP hidden for
down) and the products with all seven matrices -- in four launches: matrices that share an input are
packed as one (q|k|v, gate|up), and each launch collects its indices in its own prologue
(spqt_sparsify_gemv).  Eight distinct layer copies (about 1.5 GB of packed weights, far larger than the
126 MB L2) are visited round-robin so that weights really come from HBM.

value  = effective GB/s over the bytes the method needs
         (sum over GEMVs of count*R*(B+4) + 2n + 4count + 4 + 2m, plus 2n + 4count + 4 per index
         collection), whole job, inputs resident in HBM.  The K-step region is timed with CUDA events
         on the launching stream and repeated until a quarter of a second of device time has been
         timed; the value is that of the median region, the minimum is reported beside it.
e2e    = the same metric through spqt_host_step_launch (the step's four host-buffer linears recorded once and
         replayed with one call, one wait per step; four asynchronous calls, and a wait after every call, are
         reported beside it): x copied from pinned host memory,
         y written into pinned host memory by the kernel, the copy and the final wait of every
         call inside the timed region.
roofline.achieved = algorithmic bytes per launch of the dominant kernel (gemv_kernel, index collection
         inside: all four launches of a step are that kernel) / its mean duration in the timed region.

The other workloads: `sweep` = sparsity 0-90 % on the 14336->4096 and 4096->14336 projections against the
same-layout dense GEMV, 64 rotated weight copies, with the no-load-balancing ablation beside it;
`formats` = Llama-2-70B-shaped linears x {int4, int3} x {g128, g64} at 50 % with outlier activations;
`models` = the GEMV shapes of three model sizes at 25, 40 and 50 %; `dense` = the dense zigzag GEMV on the paper's 15 shapes over several grid sizes; `batch` = 1, 2, 4, 8 rows
over the union of their active sets; `stack` = a per-token
pass over a 32-layer Llama-3-8B-shaped stack with thresholds calibrated once for 40 % (tokens/s of the
linear layers).  The default line carries a short summary of each.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

BITS, GROUP = 4, 128
SPARSITY = 0.5
LAYER_COPIES = 8
X_POOL = 4            # distinct hidden states per site, rotated
MIN_TIMED_S = 0.25    # device time to accumulate over repeated K-step regions
METRIC = "sparse int4 GEMV effective HBM GB/s at 50% sparsity (Llama-3-8B-shaped decode-layer linears, batch 1)"

# ncu (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes of one launch of the fused kernel on the
# benchmark's stacked gate|up matrix (28672 x 4096, 50 %): traffic grows in proportion to the active blocks.
NCU_TRAFFIC_RATIO = 1.06


def needed_bytes_gemv(m, n, count, bits=BITS, group=GROUP):
    R, B = m // group, group * bits // 8
    return count * R * (B + 4) + 2 * n + 4 * count + 4 + 2 * m


def needed_bytes_sparsify(n, count):
    return 2 * n + 4 * count + 4


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc is not None:
            time.sleep(0.1)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for nm, v in zip(names, r[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time: all-reduce MAX when a process group is up, the value itself otherwise."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_rank: float, ms_local: float, world: int, device=None) -> float:
    """Replicas only: every rank moves bytes_per_rank; the job's rate is all ranks' bytes over the slowest rank's time."""
    ms = max_over_ranks(ms_local, device)
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


# --------------------------------------------------------------------------- reference arm (CPU oracle)

def oracle_sample(steps, warmup, threads=None, budget_s=None):
    """Time the oracle (index collection + fp64 sparse GEMV) on a bounded sample of the
    workload: ONE layer copy (all seven linears).  With a time budget, every step covers only the leading
    fraction of each matrix's block-rows that lets steps + warmup steps end inside it (one untimed full step
    measures the rate first); the bytes counted shrink with the rows."""
    import oracle
    from paper_2511_04477_b200 import inputs
    if threads:
        oracle.set_threads(threads)
    sample = inputs.LLAMA3_8B_LINEARS
    packed = []
    for i, (name, m, n, dist) in enumerate(sample):
        W = inputs.weights(m, n, seed=i)
        x = inputs.activations(n, seed=100 + i, dist=dist)
        t = inputs.threshold_for_sparsity(x, SPARSITY)
        packed.append((m, n, x, t) + oracle.pack(W, BITS, GROUP))

    def one_step(frac=1.0):
        nbytes = 0
        for (m, n, x, t, codes, s, z) in packed:
            idx, cnt = oracle.sparsify(x, t)
            keep = m if frac >= 1.0 else max(GROUP, int(math.ceil(frac * (m // GROUP))) * GROUP)
            oracle.sparse_gemv(codes, s, z, m, n, x, idx, BITS, GROUP, rows=None if keep == m else np.arange(keep, dtype=np.int32))
            nbytes += needed_bytes_gemv(keep, n, cnt) + needed_bytes_sparsify(n, cnt)
        return nbytes

    frac = 1.0
    if budget_s is not None:
        t0 = time.perf_counter()
        one_step()
        full = time.perf_counter() - t0
        frac = min(1.0, budget_s / max(1e-9, full * (steps + warmup)))
    for _ in range(warmup):
        one_step(frac)
    t0 = time.perf_counter()
    total = 0
    for _ in range(steps):
        total += one_step(frac)
    dt = time.perf_counter() - t0
    what = "one layer copy (q,k,v,o,gate,up,down)" if frac >= 1.0 else \
        "the leading %.1f %% of the block-rows of every linear of one layer copy (q,k,v,o,gate,up,down)" % (100 * frac)
    return {"value": total / dt / 1e9, "ms_per_step": dt / steps * 1e3, "cores": oracle.threads(),
            "sample": "%s, int4 g128, 50%% sparsity, index collection + fp64 sparse GEMV per linear, %d timed steps after "
                      "%d warm-up" % (what, steps, warmup)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    r = oracle_sample(steps, warmup, budget_s=60.0)   # exactly K timed steps after W warm-up steps, inside a minute
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": "GB/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama3-8b decode-layer linears, int4 g128, 50% sparsity (a bounded sample per step; see cpu_baseline.sample)"},
        "cpu_baseline": {"value": r["value"], "unit": "GB/s", "cores": r["cores"], "kind": "oracle", "sample": r["sample"]},
        "e2e": {"value": r["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- the other workloads

def roofline_obj(achieved, peak, peak_kind, bytes_per_launch, us_per_launch, kernel, traffic_ratio=NCU_TRAFFIC_RATIO):
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic_ratio * bytes_per_launch if traffic_ratio else None, "peak_kind": "of " + peak_kind,
            "kernel": kernel, "algorithmic_bytes_per_launch": bytes_per_launch, "avg_launch_us": us_per_launch}


def other_config_line(which, local, quick=False):
    """One of the other workloads as a dict in the same format as the headline line."""
    import torch
    from paper_2511_04477_b200 import sweep
    peak, kind = sweep.hbm_peak()
    base = {"n_gpus": 1, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int4/int3 codes, f32 accumulate, f16 in/out", "data": "synthetic", "unit": "GB/s"}
    with ClockSampler(local) as clk:
        if which == "sweep":
            rows = sweep.sparsity_sweep(peak, sparsities=[0.5] if quick else None, copies=64, unbalanced=True)
            at50 = [r for r in rows if abs(r["sparsity"] - 0.5) < 0.03]
            r0 = at50[0]
            nb = sweep.needed_bytes(r0["m"], r0["n"], r0["count"], 4, 128) + needed_bytes_sparsify(r0["n"], r0["count"])
            line = dict(base, metric="sparse int4 GEMV effective HBM GB/s at 50% sparsity on the 14336->4096 projection "
                                     "(sparsity sweep, 64 rotated weight copies)",
                        value=r0["fused_gbs"], ms_per_step=r0["fused_us"] * 1e-3, steps=20, warmup=4,
                        config={"workload": "sparsity sweep 0-90% on 4096x14336 and 14336x4096, int4 g128, sparse / index collection in "
                                            "the same launch / dense on the same packed buffers; 64 distinct weight copies rotated (2 GB, L2 is 126 MB)"},
                        roofline=roofline_obj(r0["fused_gbs"], peak, kind, nb, r0["fused_us"], "gemv_kernel<128,4,fused>"),
                        speedup_vs_dense_at_50pct={"%dx%d" % (r["m"], r["n"]): {"given_list": r["speedup_vs_dense"], "index_collection_inside": r["fused_speedup_vs_dense"],
                                                                                 "no_load_balancing": r.get("unbalanced_speedup_vs_dense")} for r in at50},
                        rows=rows)
        elif which == "formats":
            shapes = [s for s in __import__("paper_2511_04477_b200.inputs", fromlist=["x"]).LLAMA2_70B_LINEARS if (not quick or s[0] == "up")]
            rows = sweep.format_sweep(peak, shapes=shapes)
            r0 = [r for r in rows if r["m"] == 28672 and r["bits"] == 4 and r["group"] == 128][0]
            nb = sweep.needed_bytes(r0["m"], r0["n"], r0["count"], 4, 128) + needed_bytes_sparsify(r0["n"], r0["count"])
            line = dict(base, metric="sparse GEMV effective HBM GB/s at 50% sparsity on the 8192->28672 projection, int4 g128 "
                                     "(Llama-2-70B-shaped format sweep)",
                        value=r0["fused_gbs"], ms_per_step=r0["fused_us"] * 1e-3, steps=20, warmup=4,
                        config={"workload": "Llama-2-70B-shaped linears (8192x8192, 28672x8192, 8192x28672) x {int4,int3} x {g128,g64}, 50% sparsity, "
                                            "x ~ Laplace with 1% of entries x20; >= 4 rotated weight copies (> 2x L2)"},
                        roofline=roofline_obj(r0["fused_gbs"], peak, kind, nb, r0["fused_us"], "gemv_kernel<128,4,fused>", 1.13),
                        frac_of_peak={"%dx%d int%d g%d" % (r["m"], r["n"], r["bits"], r["group"]): {
                            "sparse": r["frac_of_peak"], "index_collection_inside": r["fused_frac_of_peak"], "dense": r["dense_frac_of_peak"],
                            "speedup_vs_dense": r["fused_speedup_vs_dense"]} for r in rows},
                        rows=rows)
        elif which == "dense":
            rows = sweep.dense_shape_sweep(peak)
            best = max(rows, key=lambda r: r["frac_of_peak"])
            nb = sweep.needed_bytes(best["m"], best["n"], best["n"], 4, 128)
            line = dict(base, metric="dense zigzag int4 GEMV effective HBM GB/s, best of the 15 shapes of the paper's hyper-parameter study",
                        value=best["dense_gbs"], ms_per_step=best["best_us"] * 1e-3, steps=10, warmup=4,
                        config={"workload": "dense same-layout GEMV, m in {2048,4096,8192} x n in {1024..16384}, int4 g128, grids of 64/96/128/148 CTAs "
                                            "and the built-in rule; beside it the row-wise-layout baseline (spqt_rowwise_dense_gemv) on the same shapes; rotated weight copies > 2x L2"},
                        roofline=roofline_obj(best["dense_gbs"], peak, kind, nb, best["best_us"], "gemv_kernel<128,4,dense>", 1.0),
                        zigzag_dense_vs_rowwise={"%dx%d" % (r["m"], r["n"]): r["zigzag_dense_vs_rowwise"] for r in rows},
                        speedup_from_50pct_sparsity={"%dx%d" % (r["m"], r["n"]): {"rowwise_layout": r["rowwise_sparse_speedup_over_its_dense"],
                                                                                    "zigzag_layout": r["zigzag_sparse_speedup_over_its_dense"]} for r in rows},
                        rows=rows)
        elif which == "models":
            rows = sweep.model_shapes_sweep(peak)
            r0 = [r for r in rows if r["shape"] == "70b gate,up" and abs(r["sparsity"] - 0.5) < 0.03][0]
            nb = sweep.needed_bytes(r0["m"], r0["n"], r0["count"], 4, 128)
            line = dict(base, metric="sparse int4 GEMV effective HBM GB/s at 50% sparsity, 28672x8192 (GEMV shapes of three model sizes at 25/40/50%)",
                        value=r0["sparse_gbs"], ms_per_step=r0["sparse_us"] * 1e-3, steps=20, warmup=4,
                        config={"workload": "Llama-3-8B-, Llama-2-13B- and Llama-2-70B-shaped linears, int4 g128, sparsity 25/40/50%, given list / index "
                                            "collection inside / dense; rotated weight copies > 2x L2"},
                        roofline=roofline_obj(r0["sparse_gbs"], peak, kind, nb, r0["sparse_us"], "gemv_kernel<128,4,list>"),
                        speedup_vs_dense={"%s @%d%%" % (r["shape"], round(100 * r["sparsity"])): {"given_list": r["speedup_vs_dense"],
                                                                                                 "index_collection_inside": r["fused_speedup_vs_dense"]} for r in rows},
                        rows=rows)
        elif which == "kquant":
            rows = sweep.kq_sweep(peak)
            r0 = [r for r in rows if r["m"] == 28672 and r["n"] == 8192 and r["bits"] == 4][0]
            nb = r0["sparse_gbs"] * r0["sparse_us"] * 1e3
            line = dict(base, metric="sparse GEMV over the two-level format (256-row superblocks, 6-bit block scales and minimums), effective HBM GB/s at 50% sparsity, 28672x8192",
                        value=r0["sparse_gbs"], ms_per_step=r0["sparse_us"] * 1e-3, steps=20, warmup=4,
                        config={"workload": "two-level format in the zigzag arrangement, 144-byte records; index list given (and, beside it, collected by a launch of its own); "
                                            "50% sparsity; Llama-3-8B-shaped linears and 28672x8192 with 4-bit codes, 28672x4096 and 28672x8192 also with 2- and 8-bit codes "
                                            "(80- and 272-byte records); rotated weight copies > 2x L2"},
                        roofline=roofline_obj(r0["sparse_gbs"], peak, kind, nb, r0["sparse_us"], "kq_gemv_kernel", None),
                        rows=rows)
        elif which == "batch":
            rows = sweep.batch_sweep(peak)
            r0 = [r for r in rows if r["m"] == 28672 and r["rows"] == "beam-like" and r["batch"] == 4][0]
            nb = r0["sparse_gbs"] * r0["sparse_us"] * 1e3
            line = dict(base, metric="sparse int4 GEMM effective HBM GB/s, 4 beam-like rows over the union of their active sets, "
                                     "stacked gate|up matrix 28672x4096",
                        value=r0["sparse_gbs"], ms_per_step=r0["sparse_us"] * 1e-3, steps=20, warmup=4,
                        config={"workload": "1, 2, 4, 8 rows on 28672x4096 and 4096x14336, int4 g128, threshold for 50% on the first row; rows independent "
                                            "or beam-like (a common hidden state plus 20% individual noise); union index collection + product, and dense"},
                        roofline=roofline_obj(r0["sparse_gbs"], peak, kind, nb, r0["sparse_us"], "gemm_small_kernel<128,4>", None),
                        rows=rows)
        elif which == "stack":
            res = sweep.run_stack(layers=32, tokens=40 if quick else 100, peak=peak)
            nb = res["needed_gb_per_token"] * 1e9 / res["launches_per_token"]
            line = dict(base, metric="tokens/s of the linear layers, 32-layer Llama-3-8B-shaped stack, int4 g128, thresholds calibrated for 40% sparsity",
                        unit="tokens/s", value=res["tokens_per_s"], ms_per_step=res["ms_per_token"], steps=res["tokens"], warmup=3,
                        config={"workload": "32 layers x (q|k|v, o, gate|up, down), 3.7 GB packed; per-site thresholds calibrated once on 64 pooled vectors; "
                                            "fresh x per token; one CUDA graph per token (128 launches, index collection inside)"},
                        roofline=roofline_obj(res["needed_gbs"], peak, kind, nb, res["ms_per_token"] * 1e3 / res["launches_per_token"],
                                              "gemv_kernel<128,4,fused>"),
                        result=res)
        else:
            raise SystemExit("unknown --config %r" % which)
    line["clocks"] = clk.summary()
    torch.cuda.empty_cache()
    return line


# --------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2511_04477_b200 import binding, inputs, sweep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()

    if args.config != "layer":
        if rank == 0:
            print(json.dumps(other_config_line(args.config, local, quick=args.quick)), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    linears = inputs.LLAMA3_8B_LINEARS
    sites = {"attn_in": ("laplace", 4096, ["q", "k", "v"]), "attn_out": ("laplace", 4096, ["o"]),
             "mlp_in": ("laplace", 4096, ["gate", "up"]), "mlp_mid": ("gauss", 14336, ["down"])}
    shape = {name: (m, n) for name, m, n, _ in linears}
    shape["qkv"] = (4096 + 1024 + 1024, 4096)
    shape["gateup"] = (2 * 14336, 4096)
    order = ["q", "k", "v", "o", "gate", "up", "down"]
    stacked = {"attn_in": "qkv", "attn_out": "o", "mlp_in": "gateup", "mlp_mid": "down"}   # the hot path's four GEMVs
    site_of = {nm: s for s, (_, _, names) in sites.items() for nm in names}
    site_of.update({"qkv": "attn_in", "gateup": "mlp_in"})

    # ---- weights: LAYER_COPIES x 7 matrices, random-init on the device, packed by spqt_pack
    layers = []
    g = torch.Generator(device=dev)
    for L in range(LAYER_COPIES):
        packs = {}
        Ws = {}
        for i, name in enumerate(order):
            m, n = shape[name]
            g.manual_seed(1000 * rank + L * 7 + i)
            Ws[name] = torch.empty((m, n), dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=g).half()
            packs[name] = binding.spqt_pack(Ws[name], BITS, GROUP)
        # the matrices that share an input, stacked by rows: one GEMV for q|k|v, one for gate|up
        packs["qkv"] = binding.spqt_pack(torch.cat([Ws["q"], Ws["k"], Ws["v"]], 0), BITS, GROUP)
        packs["gateup"] = binding.spqt_pack(torch.cat([Ws["gate"], Ws["up"]], 0), BITS, GROUP)
        del Ws
        layers.append(packs)
    torch.cuda.synchronize()
    weight_bytes = sum(p.nbytes for L in layers for p in L.values())

    # ---- activations: X_POOL hidden states per site (host, seeded), thresholds by nearest rank
    xs, ts = {}, {}
    for si, (s, (dname, n, _)) in enumerate(sites.items()):
        xs[s] = [inputs.activations(n, seed=10_000 + 97 * si + j, dist=dname) for j in range(X_POOL)]
        ts[s] = [inputs.threshold_for_sparsity(x, SPARSITY) for x in xs[s]]
    xd = {s: [torch.from_numpy(x).to(dev) for x in xs[s]] for s in sites}
    idx = {s: torch.empty(sites[s][1], dtype=torch.int32, device=dev) for s in sites}
    cnt = {s: torch.zeros(1, dtype=torch.int32, device=dev) for s in sites}
    ys = {nm: torch.empty(shape[nm][0], dtype=torch.float16, device=dev) for nm in shape}
    ws = {nm: binding.new_workspace(shape[nm][0], shape[nm][1], BITS, GROUP, dev) for nm in shape}

    stream = torch.cuda.Stream(device=dev)

    def hot_path_step(i):
        """The library's best route: matrices that share an input are packed as one (q|k|v, gate|up),
        and each of the four launches collects its indices itself (spqt_sparsify_gemv)."""
        L = layers[i % LAYER_COPIES]
        j = i % X_POOL
        for s, nm in stacked.items():
            binding.spqt_sparsify_gemv(L[nm], xd[s][j], ts[s][j], ws[nm], idx[s], cnt[s], ys[nm], stream=stream)

    def step(i, with_sparsify=True, gemv=True, dense=False, names=None):
        L = layers[i % LAYER_COPIES]
        j = i % X_POOL if with_sparsify else 0   # kernel-only regions keep the index lists of pool entry 0
        for s in sites:
            if with_sparsify:
                binding.spqt_sparsify(xd[s][j], ts[s][j], idx[s], cnt[s], stream=stream)
            if gemv:
                for nm in ([stacked[s]] if names == "stacked" else sites[s][2]):
                    if dense:
                        binding.spqt_dense_gemv(L[nm], xd[s][j], ws[nm], ys[nm], stream=stream)
                    else:
                        binding.spqt_sparse_gemv(L[nm], xd[s][j], idx[s], cnt[s], ws[nm], ys[nm], stream=stream)

    def counts_for(j):
        out = {}
        for s in sites:
            a = np.abs(xs[s][j].astype(np.float32))
            out[s] = int(np.count_nonzero(a > np.float32(ts[s][j])))
        return out

    counts = [counts_for(j) for j in range(X_POOL)]

    def step_bytes(i):
        c = counts[i % X_POOL]
        b = 0
        for s, nm in stacked.items():
            b += needed_bytes_sparsify(sites[s][1], c[s])
            b += needed_bytes_gemv(shape[nm][0], shape[nm][1], c[s])
        return b

    def gemv_bytes(dense=False):
        c = counts[0]
        return sum(needed_bytes_gemv(shape[nm][0], shape[nm][1], shape[nm][1] if dense else c[site_of[nm]])
                   for nm in stacked.values())

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def graph_len(K):
        """Steps captured per CUDA graph: the largest divisor of K not above 64 (so that exactly K run)."""
        return max(d for d in range(1, min(K, 64) + 1) if K % d == 0)

    def timed(fn, K, W, min_s=0.0, max_regions=4000):
        """W warm-up steps, then regions of EXACTLY K steps each between two events on the launching stream,
        launched as replays of a captured CUDA graph (so that the device, not the Python launch path, is
        timed), barrier + synchronize on both sides of every region; regions are repeated until min_s of
        device time has been timed.  Returns the list of region times (ms, max over ranks)."""
        g = graph_len(K)
        with torch.cuda.stream(stream):
            for i in range(W):
                fn(i)
        barrier()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(g):
                fn(W + i)
        with torch.cuda.stream(stream):
            graph.replay()          # one untimed replay: graph upload, instruction caches
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        regions, total = [], 0.0
        while True:
            with torch.cuda.stream(stream):
                e0.record(stream)
                for _ in range(K // g):
                    graph.replay()
                e1.record(stream)
            barrier()
            ms = max_over_ranks(e0.elapsed_time(e1), dev)
            regions.append(ms)
            total += ms * 1e-3
            if total >= min_s or len(regions) >= max_regions:
                break
        return regions

    K, W = args.steps, max(args.warmup, 3)
    med = lambda v: float(np.median(v))

    # ---- main timed region (whole hot path), with clocks sampled during it
    l0 = binding.spqt_launch_count()
    with ClockSampler(local) as clk:
        regions = timed(hot_path_step, K, W, min_s=args.min_seconds)
    launches = binding.spqt_launch_count() - l0
    ms, ms_min = med(regions), float(np.min(regions))
    g_len = graph_len(K)
    launches_timed = 4 * K
    bytes_K = (K // g_len) * sum(step_bytes(i) for i in range(W, W + g_len))
    value = world * bytes_K / (ms * 1e-3) / 1e9
    peak, peak_kind = sweep.hbm_peak()
    avg_launch_bytes = bytes_K / launches_timed
    avg_launch_us = ms * 1e3 / launches_timed
    achieved = avg_launch_bytes / avg_launch_us * 1e-3

    # ---- kernel-only regions: index lists given (pool entry 0), the dense comparison, index collection alone
    with torch.cuda.stream(stream):
        for s in sites:
            binding.spqt_sparsify(xd[s][0], ts[s][0], idx[s], cnt[s], stream=stream)
    ms_gemv = med(timed(lambda i: step(i, with_sparsify=False, names="stacked"), K, W, min_s=0.05))
    ms_dense = med(timed(lambda i: step(i, with_sparsify=False, dense=True, names="stacked"), K, W, min_s=0.05))
    ms_sparsify = med(timed(lambda i: step(i, gemv=False), K, W, min_s=0.02))
    ms_separate = med(timed(lambda i: step(i, names="stacked"), K, W, min_s=0.05))     # 4 index collections + 4 GEMVs
    with torch.cuda.stream(stream):
        for s in sites:
            binding.spqt_sparsify(xd[s][0], ts[s][0], idx[s], cnt[s], stream=stream)
    gb = K * gemv_bytes()
    gb_dense = K * gemv_bytes(dense=True)

    # ---- per shape, cold: enough distinct copies of every matrix that a copy has left L2 before its next visit
    per_shape = {}
    for nm in order + ["qkv", "gateup"]:
        s = site_of[nm]
        m, n = shape[nm]
        ncopy = sweep.copies_for(m, n, BITS, GROUP)
        packs = sweep.make_copies(m, n, BITS, GROUP, ncopy, seed0=500)
        reps = max(ncopy, 32)
        t_sp = med(timed(lambda i, nm=nm, s=s: binding.spqt_sparse_gemv(
            packs[i % ncopy], xd[s][0], idx[s], cnt[s], ws[nm], ys[nm], stream=stream), reps, 3, min_s=0.02))
        t_fu = med(timed(lambda i, nm=nm, s=s: binding.spqt_sparsify_gemv(
            packs[i % ncopy], xd[s][0], ts[s][0], ws[nm], idx[s], cnt[s], ys[nm], stream=stream), reps, 3, min_s=0.02))
        t_de = med(timed(lambda i, nm=nm, s=s: binding.spqt_dense_gemv(
            packs[i % ncopy], xd[s][0], ws[nm], ys[nm], stream=stream), reps, 3, min_s=0.02))
        c0 = counts[0][s]
        per_shape[nm] = {"m": m, "n": n, "count": c0, "copies": ncopy, "cold": True,
                         "sparse_us": t_sp * 1e3 / reps, "fused_us": t_fu * 1e3 / reps, "dense_us": t_de * 1e3 / reps,
                         "sparse_gbs": needed_bytes_gemv(m, n, c0) / (t_sp * 1e-3 / reps) / 1e9,
                         "fused_gbs": (needed_bytes_gemv(m, n, c0) + needed_bytes_sparsify(n, c0)) / (t_fu * 1e-3 / reps) / 1e9,
                         "dense_gbs": needed_bytes_gemv(m, n, n) / (t_de * 1e-3 / reps) / 1e9,
                         "speedup_vs_dense": t_de / t_sp, "fused_speedup_vs_dense": t_de / t_fu}
        per_shape[nm]["fused_frac_of_peak"] = per_shape[nm]["fused_gbs"] / peak
        del packs
        torch.cuda.empty_cache()

    # ---- achievable read and gather rates of this GPU with the GEMV's copy instruction (rank 0 only)
    probes = None
    if rank == 0:
        buf = torch.empty(2 << 30, dtype=torch.uint8, device=dev)   # 2 GB, far beyond L2
        buf.fill_(1)
        moved = torch.zeros(1, dtype=torch.int64, device=dev)
        probes = {}
        for pattern, key in ((0, "stream_read_gbs"), (1, "gather_64B_half_of_lines_gbs")):
            best = 0.0
            for _ in range(3):
                moved.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                binding.spqt_probe_read(buf, pattern, moved)
                e1.record()
                e1.synchronize()
                best = max(best, float(moved.item()) / (e0.elapsed_time(e1) * 1e-3) / 1e9)
            probes[key] = best
        del buf
        # the loop's arithmetic alone, operands in shared memory: the rate at which instruction issue saturates,
        # expressed as the bytes per second the same number of 2 KB chunks (2176 bytes with metadata) stands for
        sink = torch.empty(512 * torch.cuda.get_device_properties(dev).multi_processor_count, dtype=torch.float32,
                           device=dev)
        best = 0.0
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            chunks = binding.spqt_probe_arith(4000, sink)
            e1.record()
            e1.synchronize()
            best = max(best, chunks * 2176.0 / (e0.elapsed_time(e1) * 1e-3) / 1e9)
        probes["arithmetic_only_int4_g128_gbs_equivalent"] = best

    # ---- end to end from host buffers through the C ABI (copies + sync inside the timed region)
    e2e_names = list(stacked.values())
    hosts = [{nm: binding.HostLinear(layers[L][nm], ws[nm]) for nm in e2e_names} for L in range(LAYER_COPIES)]
    for L in range(LAYER_COPIES):
        for nm in e2e_names:
            hosts[L][nm].x_host.copy_(torch.from_numpy(xs[site_of[nm]][0]))

    steps_rec = [binding.HostStep([hosts[L][nm] for nm in e2e_names], [ts[site_of[nm]][0] for nm in e2e_names])
                 for L in range(LAYER_COPIES)]

    def e2e_step(i, how):
        if how == "recorded":
            # the step's four linears recorded once (spqt_host_step_create), replayed with one call; one wait
            steps_rec[i % LAYER_COPIES].launch(stream=stream)
            stream.synchronize()
            return
        for nm in e2e_names:
            binding.spqt_sparse_linear_host(hosts[i % LAYER_COPIES][nm], ts[site_of[nm]][0], stream=stream, wait=(how == "wait_per_call"))
        if how == "async_calls":
            stream.synchronize()       # one wait per step: the step's four results are then in pinned host memory

    e2e_K = min(K, 64)

    def e2e_time(how):
        for i in range(3):
            e2e_step(i, how)
        barrier()
        t0 = time.perf_counter()
        for i in range(3, 3 + e2e_K):
            e2e_step(i, how)
        torch.cuda.synchronize()
        return max_over_ranks(time.perf_counter() - t0, dev)

    e2e_s_per_call = e2e_time("wait_per_call")
    e2e_s_async = e2e_time("async_calls")
    e2e_s = e2e_time("recorded")
    for r in steps_rec:
        r.close()
    e2e_bytes = e2e_K * sum(needed_bytes_gemv(shape[nm][0], shape[nm][1], counts[0][site_of[nm]])
                            + needed_bytes_sparsify(shape[nm][1], counts[0][site_of[nm]]) for nm in e2e_names)
    h2d = sum(shape[nm][1] * 2 for nm in e2e_names)
    d2h = sum(shape[nm][0] * 2 for nm in e2e_names)

    status = max(binding.spqt_workspace_status(ws[nm], shape[nm][0], GROUP) for nm in shape)

    # ---- short forms of the other workloads (rank 0), so that one run covers them
    others = None
    if rank == 0 and not args.no_extra:
        del layers, hosts
        torch.cuda.empty_cache()
        others = {}
        sw = other_config_line("sweep", local, quick=True)
        others["sparsity_sweep_at_50pct"] = sw["speedup_vs_dense_at_50pct"]
        fm = other_config_line("formats", local, quick=True)
        others["formats_28672x8192_frac_of_peak"] = fm["frac_of_peak"]
        st = other_config_line("stack", local, quick=True)
        others["stack_32_layers"] = {k: st["result"][k] for k in ("tokens_per_s", "ms_per_token", "needed_gb_per_token", "needed_gbs",
                                                                    "frac_of_peak", "tokens", "device_status")}
        de = other_config_line("dense", local)
        others["rowwise_baseline_us_over_zigzag_dense_us"] = de["zigzag_dense_vs_rowwise"]
        ba = other_config_line("batch", local)
        others["small_batch_beam_like_28672x4096"] = {
            "B=%d" % r["batch"]: {"union_sparsity": r["union_sparsity"], "sparse_us_per_row": r["sparse_us_per_row"],
                                  "dense_us_per_row": r["dense_us_per_row"], "speedup_vs_dense": r["speedup_vs_dense"]}
            for r in ba["rows"] if r["m"] == 28672 and r["rows"] == "beam-like"}
        kq = other_config_line("kquant", local)
        others["two_level_format_at_50pct"] = {
            "%dx%d%s" % (r["m"], r["n"], "" if r["bits"] == 4 else " %d-bit codes" % r["bits"]):
                {"sparse_frac_of_peak": r["frac_of_peak"], "dense_frac_of_peak": r["dense_frac_of_peak"],
                 "speedup_vs_dense": r["speedup_vs_dense"]} for r in kq["rows"]}

    if rank == 0:
        cpu = oracle_sample(3, 1) if world >= 1 else None
        cpu_all = cpu["cores"]
        cpu1 = oracle_sample(1, 0, threads=1)      # the same sample on one core
        import oracle as _oracle
        _oracle.set_threads(cpu_all)
        clocks = clk.summary()
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "ms_per_step_min": ms_min / K, "regions_timed": len(regions),
            "device_seconds_timed": float(np.sum(regions)) * 1e-3,
            "us_x_mhz_per_step": (ms / K * 1e3) * clocks["sm_mhz"] if clocks["sm_mhz"] else None,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int4 codes, f32 accumulate, f16 in/out", "data": "synthetic",
            "config": {"workload": "llama3-8b decode-layer linears q,k,v,o,gate,up,down; int4 g128 zigzag; batch 1; "
                                   "50%% sparsity; q|k|v and gate|up packed as one matrix each (they share x and idx); per step "
                                   "4 launches, each collecting its indices and multiplying, one stream, "
                                   "replayed from a CUDA graph of %d steps" % g_len,
                       "l2_defeat": "%d distinct layer copies rotated, %.2f GB of packed weights (> 126 MB L2); per-shape numbers use "
                                    "enough copies of each matrix that the bytes between two visits exceed twice the L2" % (
                                        LAYER_COPIES, weight_bytes / 1e9),
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "us_per_launch": avg_launch_us,
            "us_per_step": {"hot_path": ms * 1e3 / K, "gemv_only_given_lists": ms_gemv * 1e3 / K,
                            "dense_gemv_only": ms_dense * 1e3 / K, "sparsify_only": ms_sparsify * 1e3 / K,
                            "four_sparsify_plus_four_gemv_launches": ms_separate * 1e3 / K},
            "speedup_vs_dense_same_layout": ms_dense / ms,
            "speedup_vs_dense_same_layout_given_lists": ms_dense / ms_gemv,
            "dense_gbs": gb_dense / (ms_dense * 1e-3) / 1e9,
            "gemv_only_gbs": gb / (ms_gemv * 1e-3) / 1e9,
            "pct_of_peak": {"of_measured_%.0f" % peak: 100 * achieved / peak, "of_nominal_8000": 100 * achieved / 8000,
                            "of_probed_gather": 100 * achieved / probes["gather_64B_half_of_lines_gbs"]},
            "probed_rooflines": probes,
            "per_shape": per_shape,
            "roofline": roofline_obj(achieved, peak, peak_kind, avg_launch_bytes, avg_launch_us, "gemv_kernel<128,4,fused>"),
            "cpu_baseline": {"value": cpu["value"], "unit": "GB/s", "cores": cpu["cores"], "kind": "oracle",
                             "sample": cpu["sample"], "single_thread_value": cpu1["value"]},
            "e2e": {"value": world * e2e_bytes / e2e_s / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s / e2e_K * 1e3,
                    "calls": "one spqt_host_step_launch per step (the step's four linears recorded once: per linear the copy of x from "
                             "pinned host memory, one launch, y written into pinned host memory) and one stream synchronisation",
                    "ms_per_step_four_async_calls_one_wait": e2e_s_async / e2e_K * 1e3,
                    "value_four_async_calls_one_wait": world * e2e_bytes / e2e_s_async / 1e9,
                    "ms_per_step_waiting_after_every_call": e2e_s_per_call / e2e_K * 1e3,
                    "value_waiting_after_every_call": world * e2e_bytes / e2e_s_per_call / 1e9},
            "gpu_launches": launches_timed, "launches_counted_incl_warmup_capture_and_repeats": launches,
            "clocks": clocks,
            "device_status": status,
            "other_configs": others,
            "paper_context": "paper reports up to 1.55x end-to-end decode speedup and up to 1.78x sparse-GEMV "
                             "speedup at 50% sparsity on Apple GPUs (Q4_K); other hardware, context only",
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="layer", choices=["layer", "sweep", "formats", "dense", "batch", "kquant", "models", "stack"])
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_S,
                    help="device time to accumulate over repeated K-step regions of the headline measurement")
    ap.add_argument("--quick", action="store_true", help="reduced form of --config sweep/formats/stack")
    ap.add_argument("--no-extra", action="store_true", help="headline line without the summaries of the other workloads")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
