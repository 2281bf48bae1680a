"""Run one sparse and one dense GEMV a few times on a single packed matrix, with L2 flushed
before every call -- a small, self-terminating case for `ncu` captures.

    python -m paper_2511_04477_b200.profile_case M N SPARSITY [GROUP] [REPEATS] [fused|pack|sparsify|rowwise|kq|kq2|kq5|kq6|kq8|batch4]

With `fused` the sparse call is the one that collects the indices in the same launch; with `pack` only the
offline conversion is repeated, with `sparsify` only the index collection (L2 flushed before each as well);
`rowwise` = the row-wise baseline's dense GEMV, `kq` = the two-level format's sparse and dense GEMV (`kq2`, `kq5`, `kq6`, `kq8`: with codes of that width), `batch4` = four
beam-like rows over the union of their active sets and the dense batch call.

Weights are random-init on the device (values do not affect timing); x and the threshold come
from the seeded input module.  Prints the active count and the workspace status word.
"""
from __future__ import annotations

import sys

import torch

from . import binding, inputs


def main(argv):
    m, n, sp = int(argv[0]), int(argv[1]), float(argv[2])
    group = int(argv[3]) if len(argv) > 3 else 128
    repeats = int(argv[4]) if len(argv) > 4 else 3
    mode = argv[5] if len(argv) > 5 else ""
    fused = mode == "fused"
    torch.manual_seed(0)
    W = (torch.randn(m, n, device="cuda", dtype=torch.float32) * 0.02).half()
    if mode == "rowwise" or mode.startswith("kq"):
        x = inputs.activations(n, seed=1)
        xd = torch.from_numpy(x).cuda()
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        if mode == "rowwise":
            p = binding.spqt_rowwise_pack(W, 4, group)
            del W
            for _ in range(repeats):
                flush.zero_()
                binding.spqt_rowwise_dense_gemv(p, xd)
            torch.cuda.synchronize()
            print("ok rowwise")
            return
        p = binding.spqt_kqw_pack(W, int(mode[2:] or 4))
        del W
        ws = binding.new_kq_workspace(p)
        idx, cnt = binding.spqt_sparsify(xd, inputs.threshold_for_sparsity(x, sp))
        for _ in range(repeats):
            flush.zero_()
            binding.spqt_kqw_sparse_gemv(p, xd, idx, cnt, ws)
            flush.zero_()
            binding.spqt_kqw_dense_gemv(p, xd, ws)
        torch.cuda.synchronize()
        print("ok kq count=%d" % int(cnt.item()))
        return
    p = binding.spqt_pack(W, 4, group)
    if mode == "batch4":
        import numpy as np
        del W
        base = inputs.activations(n, seed=31).astype(np.float32)
        X = np.stack([(base + 0.2 * inputs.activations(n, seed=60 + b).astype(np.float32)).astype(np.float16) for b in range(4)])
        Xd = torch.from_numpy(X).cuda()
        t = inputs.threshold_for_sparsity(X[0], sp)
        ws = binding.new_gemm_small_workspace(p)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        for _ in range(repeats):
            flush.zero_()
            Y, idx, cnt = binding.spqt_sparse_gemm_small(p, Xd, t, ws)
            flush.zero_()
            binding.spqt_dense_gemm_small(p, Xd, ws)
        torch.cuda.synchronize()
        print("ok batch4 union count=%d" % int(cnt.item()))
        return
    if mode == "pack":
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        for _ in range(repeats):
            flush.zero_()
            binding.spqt_pack(W, 4, group)
        torch.cuda.synchronize()
        print("ok pack")
        return
    del W
    x = inputs.activations(n, seed=1)
    t = inputs.threshold_for_sparsity(x, sp)
    xd = torch.from_numpy(x).cuda()
    ws = binding.new_workspace(m, n, 4, group)
    idx, cnt = binding.spqt_sparsify(xd, t)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # larger than the 126 MB L2
    if mode == "sparsify":
        for _ in range(repeats):
            flush.zero_()
            binding.spqt_sparsify(xd, t, idx, cnt)
        torch.cuda.synchronize()
        print("ok sparsify count=%d" % int(cnt.item()))
        return
    for _ in range(repeats):
        flush.zero_()
        if fused:
            binding.spqt_sparsify_gemv(p, xd, t, ws, idx, cnt)
        else:
            binding.spqt_sparse_gemv(p, xd, idx, cnt, ws)
        flush.zero_()
        binding.spqt_dense_gemv(p, xd, ws)
    torch.cuda.synchronize()
    print("ok count=%d status=%d" % (int(cnt.item()), binding.spqt_workspace_status(ws, m, group)))


if __name__ == "__main__":
    main(sys.argv[1:])
