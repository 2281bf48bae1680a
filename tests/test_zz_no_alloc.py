"""The entry point that allocates nothing (spqt_sparse_gemv_static).

Hosts that may not obtain device memory themselves -- an operator inside a framework whose
allocator owns the device, a serving loop with a frozen memory map -- get the sparse GEMV on a
1 MiB scratch compiled into the library.  It must give the bits of spqt_sparse_gemv, on a first
call (which also looks up the scratch's device address) and on the calls after it, whatever the
scratch held before.  Collected last on purpose: a run that stops at the first failure has then
already run every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04477_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _case(m, n, group, seed, sparsity):
    W = inputs.weights(m, n, seed=seed)
    x = inputs.activations(n, seed=seed + 1)
    t = inputs.threshold_for_sparsity(x, sparsity)
    p = binding.spqt_pack(torch.from_numpy(W).cuda(), 4, group)
    xd = torch.from_numpy(x).cuda()
    idx, cnt = binding.spqt_sparsify(xd, t)
    return p, xd, idx, cnt


def test_static_scratch_entry_point_matches_the_workspace_entry_point_on_consecutive_calls():
    assert torch.cuda.is_available()
    # two different problems back to back, then the first again: the shared scratch always holds
    # another call's leftovers when a call starts
    cases = [_case(4096, 4096, 128, 11, 0.5), _case(1024, 1500, 64, 13, 0.25), _case(4096, 4096, 128, 11, 0.5)]
    for (p, xd, idx, cnt) in cases:
        ws = binding.new_workspace(p.m, p.n, p.bits, p.group)
        y_ref = binding.spqt_sparse_gemv(p, xd, idx, cnt, ws)
        y = torch.full((p.m,), float("nan"), dtype=torch.float16, device="cuda")
        before = torch.cuda.memory_allocated()
        binding.spqt_sparse_gemv_static(p, xd, idx, cnt, y)
        binding.spqt_sparse_gemv_static(p, xd, idx, cnt, y)       # and once more on the warm scratch
        assert torch.cuda.memory_allocated() == before             # nothing taken from torch's allocator
        torch.cuda.synchronize()
        a, b = y.cpu().numpy(), y_ref.cpu().numpy()
        assert np.isfinite(a.astype(np.float32)).all()
        # same kernel, same fixed summation order: the bits agree (well inside the 2e-3 tolerance)
        assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
        assert binding.spqt_static_status(p.m, p.group) == 0       # the last call ran to completion


def test_static_scratch_entry_point_matches_the_oracle():
    """Not only the sibling entry point: every row against the fp64 oracle, within the tolerance the
    other GEMV tests use (2e-3 * sum_k |What_jk||x_k| over the active columns)."""
    for (m, n, group, seed, sparsity) in [(1024, 4096, 128, 21, 0.5), (512, 1500, 64, 23, 0.25)]:
        p, xd, idx, cnt = _case(m, n, group, seed, sparsity)
        y = torch.full((m,), float("nan"), dtype=torch.float16, device="cuda")
        binding.spqt_sparse_gemv_static(p, xd, idx, cnt, y)
        torch.cuda.synchronize()
        c = int(cnt.item())
        x = xd.cpu().numpy()
        codes = p.codes.cpu().numpy()
        s = p.scales.cpu().numpy().reshape(m // group, n)
        z = p.zeros.cpu().numpy().reshape(m // group, n)
        ref_idx, ref_cnt = oracle.sparsify(x, inputs.threshold_for_sparsity(x, sparsity))
        assert c == ref_cnt and np.array_equal(idx.cpu().numpy()[:c], ref_idx)
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, 4, group)
        err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
        assert np.all(err <= 2e-3 * bound)


def test_static_scratch_entry_point_refuses_what_does_not_fit_or_is_malformed():
    L = binding.lib()
    p, xd, idx, cnt = _case(128, 64, 128, 3, 0.5)
    y = torch.empty(128, dtype=torch.float16, device="cuda")
    args = lambda m, n, bits, group: (p.codes.data_ptr(), p.scale_zero.data_ptr(), m, n, bits, group,
                                      xd.data_ptr(), idx.data_ptr(), cnt.data_ptr(), y.data_ptr(), None)
    before = binding.spqt_launch_count()
    assert L.spqt_sparse_gemv_static(*args(128, 64, 5, 128)) == 2          # unsupported format
    assert L.spqt_sparse_gemv_static(*args(100, 64, 4, 128)) == 2          # m not a multiple of the group
    huge = 128 * 4096                                                      # R = 4096 block-rows: > 1 MiB of scratch
    assert binding.spqt_packed_sizes(huge, 64, 4, 128).gemv_workspace_bytes > (1 << 20)
    assert L.spqt_sparse_gemv_static(*args(huge, 64, 4, 128)) == 4         # refused, nothing launched
    # a null or misaligned pointer is refused before the scratch is cleared or anything is launched
    good = args(128, 64, 4, 128)
    assert L.spqt_sparse_gemv_static(*(good[:6] + (None,) + good[7:])) == 1                    # x missing
    assert L.spqt_sparse_gemv_static(*(good[:6] + (xd.data_ptr() + 1,) + good[7:])) == 3       # x misaligned
    assert L.spqt_sparse_gemv_static(*((p.codes.data_ptr() + 8,) + good[1:])) == 3             # codes misaligned
    assert binding.spqt_launch_count() == before
