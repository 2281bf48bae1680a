"""Run one sparse and one dense GEMV a few times on a single packed matrix, with L2 flushed
before every call -- a small, self-terminating case for `ncu` captures.

    python -m paper_2511_04477_b200.profile_case M N SPARSITY [GROUP] [REPEATS] [fused|pack|sparsify]

With `fused` the sparse call is the one that collects the indices in the same launch; with `pack` only the
offline conversion is repeated, with `sparsify` only the index collection (L2 flushed before each as well).

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
    p = binding.spqt_pack(W, 4, group)
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
