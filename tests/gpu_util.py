"""Helpers shared by the GPU parity tests (not collected as tests)."""
import numpy as np
import torch

import oracle
from paper_2511_04477_b200 import binding

TOL = 2e-3   # |y - y_ref| <= TOL * sum_k |What_jk| |x_k| over the active columns, per row


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def pack_on_gpu(W, bits, group):
    return binding.spqt_pack(dev(W), bits, group)


def packed_to_host(p):
    torch.cuda.synchronize()
    return (p.codes.cpu().numpy(), p.scales.cpu().numpy().reshape(p.m // p.group, p.n),
            p.zeros.cpu().numpy().reshape(p.m // p.group, p.n))


def check_y(y_gpu, y_ref, bound, what=""):
    """Per-row tolerance check; returns the worst err/bound ratio."""
    y = y_gpu.astype(np.float64)
    err = np.abs(y - y_ref)
    lim = TOL * bound
    bad = np.nonzero(err > lim)[0]
    assert bad.size == 0, "%s: %d rows out of tolerance, first %d: got %r want %r bound %r" % (
        what, bad.size, bad[0], y[bad[0]], y_ref[bad[0]], bound[bad[0]])
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(bound > 0, err / bound, 0.0)
    return float(ratio.max()) if ratio.size else 0.0


def run_sparse(p, x, t, ws, shuffle_seed=None):
    """sparsify + sparse GEMV on the GPU; returns (y, idx, count) as numpy."""
    xd = dev(x)
    idx, cnt = binding.spqt_sparsify(xd, t)
    if shuffle_seed is not None:
        torch.cuda.synchronize()
        c = int(cnt.item())
        perm = np.random.Generator(np.random.PCG64(shuffle_seed)).permutation(c)
        idx[:c] = idx[:c][torch.from_numpy(perm).cuda()]
    y = binding.spqt_sparse_gemv(p, xd, idx, cnt, ws)
    torch.cuda.synchronize()
    c = int(cnt.item())
    return y.cpu().numpy(), idx.cpu().numpy()[:c], c
