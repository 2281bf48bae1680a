"""Parity of the CUDA path (through the C ABI) with the CPU oracle.

Bit-exact for packed bytes, indices and counts; y within
2e-3 * sum_k |What_jk||x_k| per row (exact where the arithmetic is exact)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04477_b200 import binding, inputs
from gpu_util import TOL, check_y, dev, pack_on_gpu, packed_to_host, run_sparse

pytestmark = pytest.mark.gpu

FORMATS = [(4, 128), (4, 64), (3, 128), (3, 64)]
GEMV_FORMATS = FORMATS


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.lib()


# ------------------------------------------------------------------ a1: quantize + zigzag pack

@pytest.mark.parametrize("bits,group", FORMATS)
@pytest.mark.parametrize("m_blocks,n", [(1, 1), (2, 37), (3, 300), (8, 1030)])
def test_pack_is_byte_identical_to_the_oracle(bits, group, m_blocks, n):
    m = m_blocks * group
    W = inputs.weights(m, n, seed=bits * 100 + group + n)
    if n > 30:
        W[:group, 5] = np.float16(0.0123)          # constant group -> scale 0
        W[:, 7] = (W[:, 7].astype(np.float32) * 2.0**-12).astype(np.float16)   # fp16-subnormal scale
        W[3, 9] = np.float16(60000.0)              # huge range
    codes, s, z = oracle.pack(W, bits, group)
    p = pack_on_gpu(W, bits, group)
    gc, gs, gz = packed_to_host(p)
    assert np.array_equal(gs.view(np.uint16), s.view(np.uint16))
    assert np.array_equal(gz.view(np.uint16), z.view(np.uint16))
    assert np.array_equal(gc, codes)
    q = binding.spqt_unpack(p)
    torch.cuda.synchronize()
    assert np.array_equal(q.cpu().numpy(), oracle.unpack_codes(codes, m, n, bits, group))


def test_pack_honours_the_leading_dimension():
    m, n, ldw = 256, 100, 164
    big = inputs.weights(m, ldw, seed=77)
    Wd = dev(big)[:, :n]
    p = binding.spqt_pack(Wd, 4, 128)
    codes, s, z = oracle.pack(np.ascontiguousarray(big[:, :n]), 4, 128)
    gc, gs, gz = packed_to_host(p)
    assert np.array_equal(gc, codes) and np.array_equal(gs, s) and np.array_equal(gz, z)


def test_group_sizes_outside_64_and_128_are_refused(hand_example):
    # the library supports G in {64,128} only; the hand example (G=4) pins the oracle
    with pytest.raises(binding.SpqtError):
        binding.spqt_pack(dev(hand_example["W"]), 4, 4)


# ------------------------------------------------------------------ a2: index collection

@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 1023, 1024, 1025, 4096, 8192, 14336, 28672, 40000, 65536, 65537, 100000])
def test_index_list_is_bit_exact(n):
    x = inputs.activations(n, seed=1000 + n, dist="laplace" if n % 2 == 0 else "gauss")
    if n > 100:
        x[17] = np.float16(np.nan)
        x[18] = np.float16(np.inf)
        x[19] = np.float16(-np.inf)
        x[20] = np.float16(-0.0)
    ts = [-1.0, 0.0, inputs.threshold_for_sparsity(x, 0.25), inputs.threshold_for_sparsity(x, 0.5),
          inputs.threshold_for_sparsity(x, 0.9), 1e9, float("inf")]
    xd = dev(x)
    for t in ts:
        idx = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        binding.spqt_sparsify(xd, t, idx, cnt)
        torch.cuda.synchronize()
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        assert int(cnt.item()) == ref_cnt
        assert np.array_equal(idx.cpu().numpy()[:ref_cnt], ref_idx)
        assert np.all(idx.cpu().numpy()[ref_cnt:] == -7)       # nothing written past count


def test_empty_input_gives_count_zero():
    x = torch.empty(0, dtype=torch.float16, device="cuda")
    idx = torch.empty(1, dtype=torch.int32, device="cuda")
    cnt = torch.full((1,), 5, dtype=torch.int32, device="cuda")
    binding.spqt_sparsify(x, 0.5, idx, cnt)
    torch.cuda.synchronize()
    assert int(cnt.item()) == 0


# ------------------------------------------------------------------ a3-a5: sparse GEMV

@pytest.mark.parametrize("bits,group", GEMV_FORMATS)
@pytest.mark.parametrize("m_blocks,n,dist", [(2, 300, "laplace"), (8, 4096, "laplace"), (3, 1111, "gauss")])
def test_sparse_gemv_matches_oracle_across_sparsities(bits, group, m_blocks, n, dist):
    m = m_blocks * group
    W = inputs.weights(m, n, seed=m + n + bits)
    x = inputs.activations(n, seed=5 + n, dist=dist)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    for sp in (0.0, 0.25, 0.5, 0.9, 0.999):
        t = inputs.threshold_for_sparsity(x, sp)
        y, idx, cnt = run_sparse(p, x, t, ws)
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        assert cnt == ref_cnt and np.array_equal(idx, ref_idx)
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group)
        check_y(y, y_ref, bound, "sparsity %.3f" % sp)
    assert not ws[: 4 * (m // group + 1)].any()                # arrival counters and status word are zero
    assert binding.spqt_workspace_status(ws, m, group) == 0


@pytest.mark.parametrize("bits,group", GEMV_FORMATS)
def test_degenerate_counts(bits, group):
    m, n = 2 * group, 500
    W = inputs.weights(m, n, seed=3)
    x = inputs.activations(n, seed=4)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    # nothing active -> exactly zero
    y, idx, cnt = run_sparse(p, x, float("inf"), ws)
    assert cnt == 0 and not y.any()
    # exactly one active entry (the largest magnitude)
    a = np.abs(x.astype(np.float32))
    t = float(np.sort(a)[-2])
    y, idx, cnt = run_sparse(p, x, t, ws)
    assert cnt == 1 and idx[0] == int(a.argmax())
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    check_y(y, y_ref, bound, "one active column")


@pytest.mark.parametrize("bits,group", GEMV_FORMATS)
def test_one_hot_probes_return_the_dequantized_column(bits, group):
    """x = c e_k: y = c * What[:,k]; one product per row, so the result is the fp16
    rounding of the exact value (catches any layout / row-permutation slip)."""
    m, n = 3 * group, 140
    W = inputs.weights(m, n, seed=8)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    for k in (0, 1, 7, 8, 31, 32, 33, 139):
        x = np.zeros(n, np.float16)
        x[k] = np.float16(-1.5)
        y, idx, cnt = run_sparse(p, x, 0.5, ws)
        assert cnt == 1 and idx[0] == k
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
        check_y(y, y_ref, bound, "one-hot k=%d" % k)
        # stronger: a single product per row, so y is within half an fp16 ulp (plus fp32 dust)
        assert np.all(np.abs(y.astype(np.float64) - y_ref) <= (2.0**-11 + 2.0**-20) * np.abs(y_ref) + 2.0**-25)


@pytest.mark.parametrize("bits,group", GEMV_FORMATS)
def test_lossless_family_is_bit_exact(bits, group):
    """W = ((5j + 3k) mod 2^bits) / 2^bits quantizes without loss, x in {+-1, +-2, +-1/2}: every partial sum
    is exact in fp32, so the sparse, fused and dense results must equal the oracle's bit for bit.  (The kernel
    sums the cumulative values of four codes, which carry 12 bits more than a single code: with these 700
    columns the largest partial sum is 4.1e6 times the smallest term, a quarter of the 2^24 that fp32 holds
    exactly.)"""
    m, n = 4 * group, 700
    W = inputs.lossless_weights(m, n, levels=1 << bits)
    x = inputs.small_rational_activations(n, seed=12)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    for t in (0.25, 0.75, 1.5):
        y, idx, cnt = run_sparse(p, x, t, ws)
        y_ref, _ = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
        assert np.array_equal(y.astype(np.float64), y_ref.astype(np.float16).astype(np.float64))
        y2, _, _ = run_sparse(p, x, t, ws, shuffle_seed=3)       # any index order
        assert np.array_equal(y2, y)
        yf, _, _ = binding.spqt_sparsify_gemv(p, dev(x), t, ws)
        torch.cuda.synchronize()
        assert np.array_equal(yf.cpu().numpy(), y)
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    yd_ref, _ = oracle.dense_gemv(codes, s, z, m, n, x, bits, group)
    assert np.array_equal(yd.cpu().numpy().astype(np.float64), yd_ref.astype(np.float16).astype(np.float64))


@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64)])
def test_accumulation_error_is_far_inside_the_tolerance(bits, group):
    """A guard on the kernel's own arithmetic, tighter than the stated tolerance: with 2048 active columns the
    fp32 sums stay within 1e-4 of the bound (the tolerance is 2e-3), and all but a few rows round to the same
    fp16 value as the fp64 result."""
    m, n = 2048, 4096
    W = inputs.weights(m, n, seed=5)
    x = inputs.activations(n, seed=6)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    y, idx, cnt = run_sparse(p, x, inputs.threshold_for_sparsity(x, 0.5), ws)
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    assert check_y(y, y_ref, bound, "accumulation") < 1e-4
    same = np.count_nonzero(y.astype(np.float64) == y_ref.astype(np.float16).astype(np.float64))
    assert same >= 0.97 * m
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    yd_ref, dbound = oracle.dense_gemv(codes, s, z, m, n, x, bits, group)
    assert check_y(yd.cpu().numpy(), yd_ref, dbound, "accumulation, dense") < 1e-4


def test_index_order_does_not_matter_beyond_rounding_and_calls_are_reproducible():
    m, n, bits, group = 1024, 4096, 4, 128
    W = inputs.weights(m, n, seed=1)
    x = inputs.activations(n, seed=2)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    t = inputs.threshold_for_sparsity(x, 0.5)
    y1, idx, cnt = run_sparse(p, x, t, ws)
    y2, _, _ = run_sparse(p, x, t, ws)
    assert np.array_equal(y1.view(np.uint16), y2.view(np.uint16))  # fixed combination order
    y3, idx3, _ = run_sparse(p, x, t, ws, shuffle_seed=9)
    assert sorted(idx3.tolist()) == idx.tolist()
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    check_y(y3, y_ref, bound, "shuffled idx")


@pytest.mark.parametrize("splits", [1, 2, 3, 7, 16, 33, 148, 301, 1024])
def test_any_number_of_workers(splits):
    m, n, bits, group = 512, 1500, 4, 128
    W = inputs.weights(m, n, seed=31)
    x = inputs.activations(n, seed=32)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    t = inputs.threshold_for_sparsity(x, 0.4)
    try:
        binding.spqt_set_tuning(splits)
        y, idx, cnt = run_sparse(p, x, t, ws)
    finally:
        binding.spqt_set_tuning(0)
    assert binding.spqt_workspace_status(ws, m, group) == 0
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    check_y(y, y_ref, bound, "S=%d" % splits)


def test_one_workspace_serves_changing_shapes_and_worker_counts():
    """The workspace cleans itself: calls of different shapes, formats and CTA counts (so that block-rows
    have one, two to four and many contributing CTAs in turn) share one workspace; every result stays
    right, and the second round repeats the first bit for bit."""
    cases = [(1024, 2048, 4, 128, 0), (4096, 1024, 4, 128, 0), (28672, 512, 4, 128, 0), (512, 3000, 3, 64, 7),
             (1024, 2048, 4, 64, 0), (2048, 1024, 3, 128, 40), (1024, 2048, 4, 128, 300)]
    nbytes = max(binding.new_workspace(m, n, b, g).numel() for (m, n, b, g, _) in cases)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    prepared, first_round = [], []
    for ci, (m, n, bits, group, ctas) in enumerate(cases):
        p = pack_on_gpu(inputs.weights(m, n, seed=700 + ci), bits, group)
        prepared.append((p, packed_to_host(p), inputs.activations(n, seed=800 + ci)))
    for rep in range(2):
        for ci, (m, n, bits, group, ctas) in enumerate(cases):
            p, (codes, s, z), x = prepared[ci]
            t = inputs.threshold_for_sparsity(x, 0.5)
            try:
                binding.spqt_set_tuning(ctas)
                y, idx, cnt = run_sparse(p, x, t, ws)
            finally:
                binding.spqt_set_tuning(0)
            assert binding.spqt_workspace_status(ws, m, group) == 0
            if rep == 0:
                y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
                check_y(y, y_ref, bound, "case %d" % ci)
                first_round.append(y.copy())
            else:
                assert np.array_equal(y.view(np.uint16), first_round[ci].view(np.uint16)), "case %d changed" % ci


def test_checked_mode_refuses_bad_index_lists():
    """Checked mode: a well-formed list gives the same bits as the normal path and status 0; a list with an
    index out of range, a negative index, a repeated index or a count outside [0, n] gives status 2 and
    y = 0, and nothing is read through the bad indices."""
    m, n, bits, group = 256, 1000, 4, 128
    p = pack_on_gpu(inputs.weights(m, n, seed=91), bits, group)
    x = inputs.activations(n, seed=92)
    xd = dev(x)
    idx, cnt = binding.spqt_sparsify(xd, inputs.threshold_for_sparsity(x, 0.5))
    torch.cuda.synchronize()
    c = int(cnt.item())
    y_plain = binding.spqt_sparse_gemv(p, xd, idx, cnt, binding.new_workspace(m, n, bits, group)).cpu().numpy()

    def run_checked(idx_t, count_value):
        ws = binding.new_workspace(m, n, bits, group)
        cnt_t = torch.tensor([count_value], dtype=torch.int32, device="cuda")
        try:
            binding.spqt_set_debug(True)
            y = binding.spqt_sparse_gemv(p, xd, idx_t, cnt_t, ws)
        finally:
            binding.spqt_set_debug(False)
        return y.cpu().numpy(), binding.spqt_workspace_status(ws, m, group)

    y, status = run_checked(idx, c)
    assert status == 0 and np.array_equal(y.view(np.uint16), y_plain.view(np.uint16))
    bad = {}
    t = idx.clone(); t[3] = n; bad["index == n"] = (t, c)
    t = idx.clone(); t[c - 1] = 2 ** 31 - 1; bad["huge index"] = (t, c)
    t = idx.clone(); t[0] = -5; bad["negative index"] = (t, c)
    t = idx.clone(); t[7] = t[8]; bad["repeated index"] = (t, c)
    bad["count > n"] = (idx, n + 1)
    bad["count < 0"] = (idx, -1)
    for what, (idx_t, count_value) in bad.items():
        y, status = run_checked(idx_t, count_value)
        assert status == 2, what
        assert not y.any(), what
    # and the next well-formed call on a fresh workspace is untouched by all that
    y, status = run_checked(idx, c)
    assert status == 0 and np.array_equal(y.view(np.uint16), y_plain.view(np.uint16))
    # the verdict is per call: after a refusal the same workspace serves a well-formed list normally,
    # while its status word stays set until the caller zeroes the workspace
    ws = binding.new_workspace(m, n, bits, group)
    try:
        binding.spqt_set_debug(True)
        bad_idx = idx.clone(); bad_idx[0] = n
        y_bad = binding.spqt_sparse_gemv(p, xd, bad_idx, cnt, ws).cpu().numpy()
        y_good = binding.spqt_sparse_gemv(p, xd, idx, cnt, ws).cpu().numpy()
    finally:
        binding.spqt_set_debug(False)
    assert not y_bad.any()
    assert np.array_equal(y_good.view(np.uint16), y_plain.view(np.uint16))
    assert binding.spqt_workspace_status(ws, m, group) == 2


@pytest.mark.parametrize("m,group", [(4096, 128), (8192, 128), (2048, 64)])
def test_cluster_and_global_memory_combination_give_the_same_bits(m, group):
    """With 2 or 4 CTAs per block-row the partial sums are combined through a thread-block cluster's
    shared memory when the device can hold all clusters; switched off, through global memory.  Both add
    in the same order, so y must not change by a bit (and both must match the oracle)."""
    n, bits = 2048, 4
    p = pack_on_gpu(inputs.weights(m, n, seed=61), bits, group)
    codes, s, z = packed_to_host(p)
    x = inputs.activations(n, seed=62)
    t = inputs.threshold_for_sparsity(x, 0.5)
    ys = []
    for flags in (0, 2):
        ws = binding.new_workspace(m, n, bits, group)
        try:
            binding.spqt_set_tuning(0, flags)
            y, idx, cnt = run_sparse(p, x, t, ws)
        finally:
            binding.spqt_set_tuning(0, 0)
        assert binding.spqt_workspace_status(ws, m, group) == 0
        ys.append(y)
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    check_y(ys[0], y_ref, bound, "cluster")
    assert np.array_equal(ys[0].view(np.uint16), ys[1].view(np.uint16))


def test_seeded_random_shapes_formats_worker_counts_and_launch_modes():
    """Sixty seeded draws of (format, m, n, sparsity, number of CTAs, launch flags, fused or not): every
    y row against the oracle, index lists bit-exact, status word clean."""
    rng = np.random.Generator(np.random.PCG64(20251125))
    for case in range(60):
        bits, group = FORMATS[int(rng.integers(0, 4))]
        m = group * int(rng.choice([1, 2, 3, 5, 8, 16, 24, 32, 48, 64]))
        n = int(rng.choice([1, 2, 7, 33, 64, 255, 1000, 1024, 2049, 4096, 5000]))
        sp = float(rng.choice([0.0, 0.3, 0.5, 0.9, 1.0]))
        ctas = int(rng.choice([0, 0, 0, 1, 5, 37, 96, 148, 300]))
        flags = int(rng.integers(0, 4))
        fused = bool(rng.integers(0, 2))
        W = inputs.weights(m, n, seed=1000 + case)
        x = inputs.activations(n, seed=2000 + case, dist="laplace" if case % 2 else "gauss")
        t = inputs.threshold_for_sparsity(x, sp) if sp < 1.0 else float("inf")
        p = pack_on_gpu(W, bits, group)
        codes, s, z = packed_to_host(p)
        ws = binding.new_workspace(m, n, bits, group)
        what = "case %d: int%d g%d %dx%d sp %.1f ctas %d flags %d fused %d" % (case, bits, group, m, n, sp, ctas, flags, fused)
        try:
            binding.spqt_set_tuning(ctas, flags)
            if fused:
                idx_t = torch.full((n,), -1, dtype=torch.int32, device="cuda")
                cnt_t = torch.zeros(1, dtype=torch.int32, device="cuda")
                y_t, _, _ = binding.spqt_sparsify_gemv(p, dev(x), t, ws, idx_t, cnt_t)
                torch.cuda.synchronize()
                cnt = int(cnt_t.item())
                y, idx = y_t.cpu().numpy(), idx_t.cpu().numpy()[:cnt]
            else:
                y, idx, cnt = run_sparse(p, x, t, ws)
        finally:
            binding.spqt_set_tuning(0, 0)
        assert binding.spqt_workspace_status(ws, m, group) == 0, what
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        assert cnt == ref_cnt and np.array_equal(idx, ref_idx), what
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group)
        check_y(y, y_ref, bound, what)


def test_heavy_tailed_outliers():
    m, n, bits, group = 1024, 8192, 4, 128
    W = inputs.weights(m, n, seed=51)
    x = inputs.activations(n, seed=52, outlier_frac=0.01, outlier_scale=20.0)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    t = inputs.threshold_for_sparsity(x, 0.5)
    y, idx, cnt = run_sparse(p, x, t, ws)
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    check_y(y, y_ref, bound, "outliers")


# ------------------------------------------------------------------ a2 + a3-a5 in one launch

@pytest.mark.parametrize("bits,group", GEMV_FORMATS)
@pytest.mark.parametrize("m_blocks,n", [(2, 300), (8, 4096), (3, 1111), (32, 4096), (1, 1), (2, 33000)])
def test_fused_index_collection_and_gemv_equals_the_two_calls(bits, group, m_blocks, n):
    m = m_blocks * group
    W = inputs.weights(m, n, seed=m + n + 7)
    x = inputs.activations(n, seed=9 + n)
    if n > 100:
        x[3] = np.float16(np.nan)
        x[4] = np.float16(-np.inf)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    xd = dev(x)
    for sp in (0.0, 0.5, 0.97, None):
        t = float("inf") if sp is None else inputs.threshold_for_sparsity(x, sp)
        idx = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        y, _, _ = binding.spqt_sparsify_gemv(p, xd, t, ws, idx, cnt)
        torch.cuda.synchronize()
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        assert int(cnt.item()) == ref_cnt
        got = idx.cpu().numpy()
        assert np.array_equal(got[:ref_cnt], ref_idx) and np.all(got[ref_cnt:] == -7)
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group)
        check_y(y.cpu().numpy(), y_ref, bound, "fused, sparsity %r" % sp)
        y2, _, _ = run_sparse(p, x, t, ws)
        assert np.array_equal(y.cpu().numpy().view(np.uint16), y2.view(np.uint16))
    assert binding.spqt_workspace_status(ws, m, group) == 0


# ------------------------------------------------------------------ a6: dense GEMV

@pytest.mark.parametrize("bits,group", GEMV_FORMATS)
@pytest.mark.parametrize("m_blocks,n", [(2, 300), (8, 4096), (1, 1)])
def test_dense_gemv_matches_oracle_and_the_sparse_path_at_threshold_below_zero(bits, group, m_blocks, n):
    m = m_blocks * group
    W = inputs.weights(m, n, seed=61 + n)
    x = inputs.activations(n, seed=62 + n)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    y_ref, bound = oracle.dense_gemv(codes, s, z, m, n, x, bits, group)
    check_y(yd.cpu().numpy(), y_ref, bound, "dense")
    ys, idx, cnt = run_sparse(p, x, -1.0, ws)
    assert cnt == n
    check_y(ys, y_ref, bound, "sparse at t<0")


def test_config_single_gemv_4096x4096_seed0_every_row():
    """The single-GEMV configuration, every output row: W 4096x4096 ~ N(0, 0.02^2) int4 g128,
    x ~ Laplace(0,1), threshold = nearest-rank median of |x|, seed 0."""
    m = n = 4096
    W = inputs.weights(m, n, seed=0)
    x = inputs.activations(n, seed=0, dist="laplace")
    t = inputs.threshold_for_sparsity(x, 0.5)
    assert abs(t - 0.693) < 0.03                       # ln 2 for |Laplace|
    p = pack_on_gpu(W, 4, 128)
    codes, s, z = packed_to_host(p)
    c_ref, s_ref, z_ref = oracle.pack(W, 4, 128)
    assert np.array_equal(codes, c_ref) and np.array_equal(s, s_ref) and np.array_equal(z, z_ref)
    ws = binding.new_workspace(m, n, 4, 128)
    y, idx, cnt = run_sparse(p, x, t, ws)
    ref_idx, ref_cnt = oracle.sparsify(x, t)
    assert cnt == ref_cnt and np.array_equal(idx, ref_idx)
    assert abs(inputs.realised_sparsity(x, t) - 0.5) < 2e-3
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, 4, 128)
    worst = check_y(y, y_ref, bound, "config 0")
    assert worst < 5e-4                                # an order of magnitude inside the tolerance
    yf, _, _ = binding.spqt_sparsify_gemv(p, dev(x), t, ws)
    torch.cuda.synchronize()
    assert np.array_equal(yf.cpu().numpy().view(np.uint16), y.view(np.uint16))
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    yd_ref, dbound = oracle.dense_gemv(codes, s, z, m, n, x, 4, 128)
    check_y(yd.cpu().numpy(), yd_ref, dbound, "config 0 dense")


# ------------------------------------------------------------------ full-size shapes, sampled rows

@pytest.mark.parametrize("name,m,n,dist", [l for l in inputs.LLAMA3_8B_LINEARS if l[0] in ("q", "k", "gate", "down")])
def test_llama3_8b_shapes_on_sampled_rows(name, m, n, dist):
    bits, group = 4, 128
    W = inputs.weights(m, n, seed={"q": 401, "k": 402, "gate": 403, "down": 404}[name])
    x = inputs.activations(n, seed=7, dist=dist)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    rows = np.unique(np.concatenate([
        np.random.Generator(np.random.PCG64(5)).integers(0, m, size=192),
        [0, 63, 64, 127, 128, m - 129, m - 128, m - 1]])).astype(np.int32)
    for sp in (0.25, 0.4, 0.5):
        t = inputs.threshold_for_sparsity(x, sp)
        y, idx, cnt = run_sparse(p, x, t, ws)
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        assert cnt == ref_cnt and np.array_equal(idx, ref_idx)
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group, rows=rows)
        check_y(y[rows], y_ref, bound, "%s at %.2f" % (name, sp))
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    y_ref, bound = oracle.dense_gemv(codes, s, z, m, n, x, bits, group, rows=rows)
    check_y(yd.cpu().numpy()[rows], y_ref, bound, "%s dense" % name)
    # spot-check the packed bytes of a few blocks against the oracle's pack of those rows
    r = (m // group) - 1
    sub = np.ascontiguousarray(W[r * group:(r + 1) * group])
    c_ref, s_ref, z_ref = oracle.pack(sub, bits, group)
    B = oracle.block_bytes(bits, group)
    assert np.array_equal(codes[r * n * B:(r + 1) * n * B], c_ref)
    assert np.array_equal(s[r], s_ref[0]) and np.array_equal(z[r], z_ref[0])


def test_32_layer_stack_token_pass_on_sampled_layers_sites_and_rows():
    """The 32-layer Llama-3-8B-shaped stack as the sweep tool runs it (3.7 GB of packed weights, thresholds
    calibrated once per site for 40 % on pooled vectors, fresh x per token, index collection inside the GEMV
    launch): index lists bit-exact and y on sampled rows against the oracle, for three layers, all four
    sites and two tokens."""
    from paper_2511_04477_b200 import sweep
    layers, tokens = 32, 3
    packs, thr, xs = sweep.build_stack(layers, tokens)
    rng = np.random.Generator(np.random.PCG64(77))
    for L in (0, 17, 31):
        for (site, m, n, _) in sweep.STACK_SITES:
            p = packs[L][site]
            codes, s, z = packed_to_host(p)
            ws = binding.new_workspace(m, n, 4, 128)
            rows = np.unique(np.concatenate([rng.integers(0, m, size=48), [0, 127, 128, m - 1]])).astype(np.int32)
            for t in (0, tokens - 1):
                x = xs[site][0][t]
                y, idx, cnt = binding.spqt_sparsify_gemv(p, xs[site][1][t], thr[site], ws)
                torch.cuda.synchronize()
                ref_idx, ref_cnt = oracle.sparsify(x, thr[site])
                assert int(cnt.item()) == ref_cnt and np.array_equal(idx.cpu().numpy()[:ref_cnt], ref_idx)
                assert 0.3 < 1.0 - ref_cnt / n < 0.5   # calibrated for 40 %, fluctuates per token
                y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, 4, 128, rows=rows)
                check_y(y.cpu().numpy()[rows], y_ref, bound, "layer %d %s token %d" % (L, site, t))
            assert binding.spqt_workspace_status(ws, m, 128) == 0


@pytest.mark.parametrize("bits,group", FORMATS)
def test_llama2_70b_attention_shape_with_heavy_tailed_outliers(bits, group):
    """8192 -> 8192, every format, x ~ Laplace with 1 % of the entries multiplied by 20, 50 % sparsity."""
    m = n = 8192
    W = inputs.weights(m, n, seed=70 + bits + group)
    x = inputs.activations(n, seed=71, outlier_frac=0.01, outlier_scale=20.0)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    rows = np.unique(np.concatenate([np.random.Generator(np.random.PCG64(6)).integers(0, m, size=160),
                                     [0, group - 1, group, m - group, m - 1]])).astype(np.int32)
    t = inputs.threshold_for_sparsity(x, 0.5)
    y, idx, cnt = run_sparse(p, x, t, ws)
    ref_idx, ref_cnt = oracle.sparsify(x, t)
    assert cnt == ref_cnt and np.array_equal(idx, ref_idx)
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group, rows=rows)
    check_y(y[rows], y_ref, bound, "70B attention shape")
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    yd_ref, dbound = oracle.dense_gemv(codes, s, z, m, n, x, bits, group, rows=rows)
    check_y(yd.cpu().numpy()[rows], yd_ref, dbound, "70B attention shape, dense")


# ------------------------------------------------------------------ host-buffer entry point

def test_host_entry_point_matches_the_device_path():
    m, n, bits, group = 1024, 4096, 4, 128
    W = inputs.weights(m, n, seed=71)
    x = inputs.activations(n, seed=72)
    p = pack_on_gpu(W, bits, group)
    h = binding.HostLinear(p)
    t = inputs.threshold_for_sparsity(x, 0.5)
    h.x_host.copy_(torch.from_numpy(x))
    y_host = binding.spqt_sparse_linear_host(h, t).numpy().copy()
    y_dev, idx, cnt = run_sparse(p, x, t, binding.new_workspace(m, n, bits, group))
    assert np.array_equal(y_host.view(np.uint16), y_dev.view(np.uint16))
    assert int(h.count.item()) == cnt
    # the variant that does not wait: two linears enqueued one after the other, one synchronisation
    h2 = binding.HostLinear(p)
    x2 = inputs.activations(n, seed=73)
    h.y_host.zero_()
    h2.x_host.copy_(torch.from_numpy(x2))
    s = torch.cuda.Stream()
    binding.spqt_sparse_linear_host(h, t, stream=s, wait=False)
    binding.spqt_sparse_linear_host(h2, t, stream=s, wait=False)
    s.synchronize()
    assert np.array_equal(h.y_host.numpy().view(np.uint16), y_dev.view(np.uint16))
    y2, _, _ = run_sparse(p, x2, t, binding.new_workspace(m, n, bits, group))
    assert np.array_equal(h2.y_host.numpy().view(np.uint16), y2.view(np.uint16))
    # and both recorded once as a step, replayed twice with different contents of the x buffers
    step = binding.HostStep([h, h2], [t, t])
    for (xa, xb, ya, yb) in ((x, x2, y_dev, y2), (x2, x, y2, y_dev)):
        h.x_host.copy_(torch.from_numpy(xa))
        h2.x_host.copy_(torch.from_numpy(xb))
        h.y_host.zero_()
        h2.y_host.zero_()
        step.launch(stream=s)
        s.synchronize()
        assert np.array_equal(h.y_host.numpy().view(np.uint16), ya.view(np.uint16))
        assert np.array_equal(h2.y_host.numpy().view(np.uint16), yb.view(np.uint16))
    step.close()


def test_read_and_gather_probes_fetch_what_they_report():
    """The roofline probes of the benchmark: every 64-byte block of the region, or half of them."""
    buf = torch.ones(256 << 20, dtype=torch.uint8, device="cuda")
    moved = torch.zeros(1, dtype=torch.int64, device="cuda")
    binding.spqt_probe_read(buf, 0, moved)
    torch.cuda.synchronize()
    all_blocks = int(moved.item())
    assert 0.98 * buf.numel() <= all_blocks <= buf.numel()
    moved.zero_()
    binding.spqt_probe_read(buf, 1, moved)
    torch.cuda.synchronize()
    assert abs(int(moved.item()) - all_blocks // 2) <= all_blocks // 100


def test_arithmetic_probe_does_the_work_it_reports():
    """The arithmetic-only probe: chunk count as documented, sums that grow with the chunks (the arithmetic is not
    optimised away), and a sink that is too small is refused."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    sink = torch.zeros(512 * sms, dtype=torch.float32, device="cuda")
    assert binding.spqt_probe_arith(30, sink) == sms * 16 * 30
    torch.cuda.synchronize()
    a = sink.double().cpu().numpy().copy()
    assert binding.spqt_probe_arith(60, sink) == sms * 16 * 60
    torch.cuda.synchronize()
    b = sink.double().cpu().numpy()
    assert np.all(np.isfinite(a)) and np.all(a > 0)
    assert np.allclose(b, 2 * a, rtol=1e-4)       # whole rounds of the three stages: twice the sums
    with pytest.raises(binding.SpqtError):
        binding.spqt_probe_arith(30, sink[: 512 * sms - 1])


def test_kernels_are_counted():
    before = binding.spqt_launch_count()
    x = dev(inputs.activations(256, seed=1))
    binding.spqt_sparsify(x, 0.5)
    assert binding.spqt_launch_count() == before + 1


# ------------------------------------------------------------------ a1: zeros of both signs in a group

@pytest.mark.parametrize("bits,group", FORMATS)
def test_pack_of_groups_with_zeros_of_both_signs_is_byte_identical(bits, group):
    """Pruned weights: groups whose minimum (or maximum) is zero with -0.0 and +0.0 both present, in either
    order, and all-zero groups of either sign.  The stored offset is +0.0 whatever the order."""
    m, n = 2 * group, 136                      # 136 columns: the 4-bit G=64 kernel's vector path too
    W = np.abs(inputs.weights(m, n, seed=5))
    W[::3] = np.float16(0.0)
    W[1::7] = np.float16(-0.0)
    W[:, 5] = -W[:, 5]                         # maximum zero
    W[:group, 9] = np.float16(-0.0)            # a whole group of -0.0
    W[group:, 9] = np.float16(0.0)
    W[0, 11], W[1, 11] = np.float16(0.0), np.float16(-0.0)
    W[0, 12], W[1, 12] = np.float16(-0.0), np.float16(0.0)
    codes, s, z = oracle.pack(W, bits, group)
    assert not z[:, [0, 9, 11, 12]].view(np.uint16).any()          # +0.0 offsets
    gc, gs, gz = packed_to_host(pack_on_gpu(W, bits, group))
    assert np.array_equal(gs.view(np.uint16), s.view(np.uint16))
    assert np.array_equal(gz.view(np.uint16), z.view(np.uint16))
    assert np.array_equal(gc, codes)


# ------------------------------------------------------------------ lists longer than the shared-memory window

@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64)])
@pytest.mark.parametrize("m_blocks,n", [(300, 20000), (2, 20000), (5, 32768), (160, 32768)])
def test_lists_longer_than_the_shared_memory_window(bits, group, m_blocks, n):
    """A CTA keeps 12288 list entries in shared memory at a time; with more active entries than that in
    its slices the window is rebuilt between spans -- in the sparse call, in the call that collects the
    indices itself (which then also writes the returned list span by span) and in the dense call over an
    odd number of columns.  Index list bit-exact, y on sampled rows against the oracle, and the one-launch
    and two-launch routes agree bit for bit."""
    m = m_blocks * group
    nn = n - 1 if n == 20000 else n            # 19999 columns: the dense call takes the list path as well
    W = inputs.weights(m, nn, seed=m_blocks + n)
    x = inputs.activations(nn, seed=77 + n)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, nn, bits, group)
    rows = np.unique(np.concatenate([np.random.Generator(np.random.PCG64(3)).integers(0, m, size=64),
                                     [0, group - 1, group, m - group, m - 1]])).astype(np.int32)
    xd = dev(x)
    for sp in (0.0, 0.1):
        t = inputs.threshold_for_sparsity(x, sp)
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        assert ref_cnt > 12288
        y, idx, cnt = run_sparse(p, x, t, ws)
        assert cnt == ref_cnt and np.array_equal(idx, ref_idx)
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, nn, x, ref_idx, bits, group, rows=rows)
        check_y(y[rows], y_ref, bound, "sparse, long list, sparsity %.1f" % sp)
        idx_t = torch.full((nn,), -7, dtype=torch.int32, device="cuda")
        cnt_t = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        yf, _, _ = binding.spqt_sparsify_gemv(p, xd, t, ws, idx_t, cnt_t)
        torch.cuda.synchronize()
        got = idx_t.cpu().numpy()
        assert int(cnt_t.item()) == ref_cnt
        assert np.array_equal(got[:ref_cnt], ref_idx) and np.all(got[ref_cnt:] == -7)
        assert np.array_equal(yf.cpu().numpy().view(np.uint16), y.view(np.uint16))
    yd = binding.spqt_dense_gemv(p, xd, ws)
    torch.cuda.synchronize()
    yd_ref, dbound = oracle.dense_gemv(codes, s, z, m, nn, x, bits, group, rows=rows)
    check_y(yd.cpu().numpy()[rows], yd_ref, dbound, "dense, long x")
    assert binding.spqt_workspace_status(ws, m, group) == 0


# ------------------------------------------------------------------ Llama-2-70B-shaped linears at full size

@pytest.mark.parametrize("bits,group", FORMATS)
@pytest.mark.parametrize("name,m,n", [("up", 28672, 8192), ("down", 8192, 28672)])
def test_llama2_70b_mlp_shapes_at_full_size_on_sampled_rows(bits, group, name, m, n):
    """8192 -> 28672 and 28672 -> 8192 in every format, x ~ Laplace with 1 % of the entries multiplied by 20,
    50 % sparsity, in the launch configuration the benchmark times: sparse, index collection in the same
    launch, and dense, on sampled rows; packed bytes of two block-rows against the oracle's pack."""
    W = inputs.weights(m, n, seed=900 + bits + group + (0 if name == "up" else 1))
    x = inputs.activations(n, seed=901, outlier_frac=0.01, outlier_scale=20.0)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    B = oracle.block_bytes(bits, group)
    for r in (0, m // group - 1):
        c_ref, s_ref, z_ref = oracle.pack(np.ascontiguousarray(W[r * group:(r + 1) * group]), bits, group)
        assert np.array_equal(codes[r * n * B:(r + 1) * n * B], c_ref)
        assert np.array_equal(s[r], s_ref[0]) and np.array_equal(z[r], z_ref[0])
    del W
    ws = binding.new_workspace(m, n, bits, group)
    rows = np.unique(np.concatenate([np.random.Generator(np.random.PCG64(8)).integers(0, m, size=96),
                                     [0, group - 1, group, m - group, m - 1]])).astype(np.int32)
    t = inputs.threshold_for_sparsity(x, 0.5)
    y, idx, cnt = run_sparse(p, x, t, ws)
    ref_idx, ref_cnt = oracle.sparsify(x, t)
    assert cnt == ref_cnt and np.array_equal(idx, ref_idx)
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group, rows=rows)
    check_y(y[rows], y_ref, bound, "%s sparse" % name)
    idx_t = torch.full((n,), -7, dtype=torch.int32, device="cuda")
    cnt_t = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    yf, _, _ = binding.spqt_sparsify_gemv(p, dev(x), t, ws, idx_t, cnt_t)
    torch.cuda.synchronize()
    assert int(cnt_t.item()) == ref_cnt and np.array_equal(idx_t.cpu().numpy()[:ref_cnt], ref_idx)
    assert np.array_equal(yf.cpu().numpy().view(np.uint16), y.view(np.uint16))
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    yd_ref, dbound = oracle.dense_gemv(codes, s, z, m, n, x, bits, group, rows=rows)
    check_y(yd.cpu().numpy()[rows], yd_ref, dbound, "%s dense" % name)
    assert binding.spqt_workspace_status(ws, m, group) == 0


# ------------------------------------------------------------------ ablation: no load balancing

@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64)])
@pytest.mark.parametrize("m_blocks,n", [(2, 300), (32, 4096), (48, 4096), (224, 4096), (3, 1111)])
def test_static_column_partition_ablation_matches_the_oracle(bits, group, m_blocks, n):
    """The paper's "sparse without load balancing": CTAs and warps take fixed ranges of the matrix columns.
    Same index list and, up to the order of the partial sums, the same y -- also when the active entries
    are all in one part of x (the case the static partition balances worst)."""
    m = m_blocks * group
    W = inputs.weights(m, n, seed=m + n + 11)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    spread = inputs.activations(n, seed=13 + n)
    clustered = spread.copy()
    clustered[n // 3:] = (clustered[n // 3:].astype(np.float32) * 1e-3).astype(np.float16)   # active entries in the first third
    for x, sp in ((spread, 0.5), (spread, 0.0), (clustered, 0.7)):
        t = inputs.threshold_for_sparsity(x, sp)
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group)
        idx = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        try:
            binding.spqt_set_tuning(0, 4)
            y, _, _ = binding.spqt_sparsify_gemv(p, dev(x), t, ws, idx, cnt)
            torch.cuda.synchronize()
        finally:
            binding.spqt_set_tuning(0, 0)
        got = idx.cpu().numpy()
        assert int(cnt.item()) == ref_cnt
        assert np.array_equal(got[:ref_cnt], ref_idx) and np.all(got[ref_cnt:] == -7)
        check_y(y.cpu().numpy(), y_ref, bound, "static partition, sparsity %.1f" % sp)
    assert binding.spqt_workspace_status(ws, m, group) == 0


# ------------------------------------------------------------------ per-shape profiling

def test_autotune_picks_a_grid_and_results_stay_right():
    """spqt_autotune times the candidate grids for a shape and later calls use its choice; the results
    still match the oracle, and a small matrix is not spread over every SM."""
    m, n, bits, group = 1024, 4096, 4, 128
    W = inputs.weights(m, n, seed=301)
    x = inputs.activations(n, seed=302)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_workspace(m, n, bits, group)
    t = inputs.threshold_for_sparsity(x, 0.5)
    flush = torch.empty(192 << 20, dtype=torch.uint8, device="cuda")
    before = binding.spqt_launch_count()
    ctas_sparse, ctas_dense = binding.spqt_autotune(p, dev(x), t, ws, flush)
    assert binding.spqt_launch_count() > before + 20          # it really timed launches
    R = m // group
    valid = {148} | {k * R for k in range(1, 9)}
    assert ctas_sparse in valid and ctas_dense in valid
    y, idx, cnt = run_sparse(p, x, t, ws)
    ref_idx, ref_cnt = oracle.sparsify(x, t)
    assert cnt == ref_cnt and np.array_equal(idx, ref_idx)
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group)
    check_y(y, y_ref, bound, "after autotune, sparse")
    yf, _, _ = binding.spqt_sparsify_gemv(p, dev(x), t, ws)
    yd = binding.spqt_dense_gemv(p, dev(x), ws)
    torch.cuda.synchronize()
    check_y(yf.cpu().numpy(), y_ref, bound, "after autotune, fused")
    yd_ref, dbound = oracle.dense_gemv(codes, s, z, m, n, x, bits, group)
    check_y(yd.cpu().numpy(), yd_ref, dbound, "after autotune, dense")
    assert binding.spqt_workspace_status(ws, m, group) == 0


# ------------------------------------------------------------------ threshold calibration

def test_calibration_threshold_is_the_exact_order_statistic():
    from paper_2511_04477_b200 import calibrate
    g = np.random.Generator(np.random.PCG64(9))
    pools = {"laplace": g.laplace(0.0, 1.0, size=64 * 4096).astype(np.float16),
             "gauss": g.standard_normal(32 * 14336).astype(np.float16),
             "ties": (g.integers(0, 5, size=1000) * 0.25).astype(np.float16),
             "one": np.array([-3.0], np.float16)}
    pools["laplace"][:7] = [np.nan, np.inf, -np.inf, 0.0, -0.0, 65504.0, 6e-8]
    ws = binding.new_calibration_workspace()
    for name, pool in pools.items():
        for sp in (0.0, 1e-6, 0.25, 0.4, 0.5, 0.9, 1.0):
            t = float(binding.spqt_calibrate_threshold(dev(pool), sp, ws).item())
            assert t == oracle.calibrate_threshold(pool, sp), (name, sp)
        assert not ws.any()                                       # the histogram is left zeroed
    assert float(binding.spqt_calibrate_threshold(torch.empty(0, dtype=torch.float16, device="cuda"), 0.5, ws).item()) == -1.0
    # the two modes of the tool: one global level; per-matrix levels averaged over the matrices that share an input
    sites = {"attn_in": dev(pools["laplace"]), "attn_out": dev(pools["laplace"][::2].copy()),
             "mlp_in": dev(pools["laplace"][1::2].copy()), "mlp_mid": dev(pools["gauss"])}
    host = {k: v.cpu().numpy() for k, v in sites.items()}
    uni = calibrate.unified(sites, 0.4)
    assert uni == {k: oracle.calibrate_threshold(host[k], 0.4) for k in sites}
    levels = {"q": 0.3, "k": 0.5, "v": 0.4, "o": 0.25, "gate": 0.6, "up": 0.5, "down": 0.45}
    grp = calibrate.grouped(sites, levels)
    for site, names in calibrate.LLAMA_GROUPS.items():
        assert grp[site] == oracle.calibrate_threshold(host[site], oracle.group_sparsity([levels[nm] for nm in names]))


# ------------------------------------------------------------------ small batch over the union of active sets

@pytest.mark.parametrize("bits,group", GEMV_FORMATS)
@pytest.mark.parametrize("m_blocks,n,batch", [(2, 300, 2), (8, 4096, 4), (3, 1111, 3), (32, 4096, 8), (1, 1, 1), (224, 1024, 5),
                                                  (4, 14336, 4), (2, 20001, 3), (1, 65535, 2)])
def test_small_batch_over_the_union_matches_the_oracle(bits, group, m_blocks, n, batch):
    m = m_blocks * group
    W = inputs.weights(m, n, seed=m + n + batch)
    X = np.stack([inputs.activations(n, seed=500 + 10 * batch + b, dist="laplace" if b % 2 == 0 else "gauss") for b in range(batch)])
    if n > 100:
        X[0, 3] = np.float16(np.nan)
        X[batch - 1, 4] = np.float16(-np.inf)
    p = pack_on_gpu(W, bits, group)
    codes, s, z = packed_to_host(p)
    ws = binding.new_gemm_small_workspace(p)
    big = torch.full((batch, n + 8), 7.0, dtype=torch.float16, device="cuda")        # rows with a leading dimension
    big[:, :n] = dev(X)
    Xd = big[:, :n]
    rows = None if m <= 4096 else np.unique(np.random.Generator(np.random.PCG64(4)).integers(0, m, size=128)).astype(np.int32)
    for sp in (0.5, 0.9, 0.0, None):
        t = float("inf") if sp is None else inputs.threshold_for_sparsity(X[0], sp)
        idx = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        Y = torch.full((batch, m), float("nan"), dtype=torch.float16, device="cuda")
        binding.spqt_sparse_gemm_small(p, Xd, t, ws, idx, cnt, Y)
        torch.cuda.synchronize()
        ref_idx, ref_cnt = oracle.union_sparsify(X, t)
        got = idx.cpu().numpy()
        assert int(cnt.item()) == ref_cnt
        assert np.array_equal(got[:ref_cnt], ref_idx) and np.all(got[ref_cnt:] == -7)
        Y_ref, bound = oracle.sparse_gemm_small(codes, s, z, m, n, X, ref_idx, bits, group, rows=rows)
        Yh = Y.cpu().numpy()
        for b in range(batch):
            if n > 100 and b == 0 and 3 in ref_idx:
                continue                                         # the NaN entry is in the union through another row
            check_y(Yh[b] if rows is None else Yh[b][rows], Y_ref[b], bound[b], "batch row %d, sparsity %r" % (b, sp))
        Y2 = torch.empty_like(Y)
        binding.spqt_sparse_gemm_small(p, Xd, t, ws, idx, cnt, Y2)
        torch.cuda.synchronize()
        assert torch.equal(Y.view(torch.int16), Y2.view(torch.int16))        # fixed order of sums
    Xc = X.copy()
    if n > 100:
        Xc[0, 3] = np.float16(0.5)
        Xc[batch - 1, 4] = np.float16(-0.5)
    Yd = binding.spqt_dense_gemm_small(p, dev(Xc), ws)
    torch.cuda.synchronize()
    for b in range(batch):
        yd_ref, dbound = oracle.dense_gemv(codes, s, z, m, n, Xc[b], bits, group, rows=rows)
        yb = Yd.cpu().numpy()[b]
        check_y(yb if rows is None else yb[rows], yd_ref, dbound, "dense batch row %d" % b)
    assert not ws[: 4 * (m // group)].any()                      # arrival counters back at zero


def test_small_batch_of_identical_rows_equals_the_single_row_call():
    m, n, bits, group = 1024, 4096, 4, 128
    W = inputs.weights(m, n, seed=44)
    x = inputs.activations(n, seed=45)
    p = pack_on_gpu(W, bits, group)
    t = inputs.threshold_for_sparsity(x, 0.5)
    y1, idx1, cnt1 = run_sparse(p, x, t, binding.new_workspace(m, n, bits, group))
    X = np.repeat(x[None, :], 6, axis=0)
    Y, idx, cnt = binding.spqt_sparse_gemm_small(p, dev(X), t, binding.new_gemm_small_workspace(p))
    torch.cuda.synchronize()
    assert int(cnt.item()) == cnt1 and np.array_equal(idx.cpu().numpy()[:cnt1], idx1)
    Yh = Y.cpu().numpy().astype(np.float64)
    codes, s, z = packed_to_host(p)
    y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx1, bits, group)
    for b in range(6):
        check_y(Y.cpu().numpy()[b], y_ref, bound, "row %d" % b)
        assert np.array_equal(Yh[b], Yh[0])


# ---------------------------------------------------------------- row-wise comparison baseline

@pytest.mark.parametrize("group", [128, 64])
@pytest.mark.parametrize("m,n", [(8, 128), (1000, 1152), (333, 1024), (1024, 4096), (4096, 4096), (2051, 14336), (64, 16384), (5000, 2048)])
def test_rowwise_baseline_pack_and_dense_gemv_match_the_oracle(group, m, n):
    W = inputs.weights(m, n, seed=3 * m + n + group)
    W[0, :group] = np.float16(0.25)                      # a constant group: scale 0
    W[m - 1, n - group:n - group + 2] = np.array([0.0, -0.0], dtype=np.float16)
    x = inputs.activations(n, seed=m + 7, dist="gauss" if n > 8192 else "laplace")
    q, s, z = oracle.rowwise_quantize(W, 4, group)
    p = binding.spqt_rowwise_pack(dev(W), 4, group)
    torch.cuda.synchronize()
    assert np.array_equal(p.codes.cpu().numpy(), oracle.rowwise_pack_codes(q, 4, group))
    assert np.array_equal(p.scales.cpu().numpy().view(np.uint16).reshape(m, n // group), s.view(np.uint16))
    assert np.array_equal(p.zeros.cpu().numpy().view(np.uint16).reshape(m, n // group), z.view(np.uint16))
    y = torch.full((m,), float("nan"), dtype=torch.float16, device="cuda")
    binding.spqt_rowwise_dense_gemv(p, dev(x), y)
    torch.cuda.synchronize()
    y_ref, bound = oracle.rowwise_dense_gemv(q, s, z, x, group)
    check_y(y.cpu().numpy(), y_ref, bound, "row-wise dense %dx%d g%d" % (m, n, group))
    y2 = binding.spqt_rowwise_dense_gemv(p, dev(x))
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))             # fixed order of sums
    # thresholded: the inactive entries (and a NaN) contribute nothing
    xs = x.copy()
    if n > 100:
        xs[5] = np.float16(np.nan)
    for sp in (0.5, 0.0):
        t = inputs.threshold_for_sparsity(x, sp)
        yt = binding.spqt_rowwise_thresholded_gemv(p, dev(xs), t)
        torch.cuda.synchronize()
        yt_ref, tb = oracle.rowwise_thresholded_gemv(q, s, z, xs, t, group)
        check_y(yt.cpu().numpy(), yt_ref, tb, "row-wise thresholded %dx%d g%d sparsity %r" % (m, n, group, sp))


@pytest.mark.parametrize("group", [128, 64])
def test_rowwise_baseline_is_exact_on_lossless_weights(group):
    # codes along a row take every value 0..15 inside every group (the column coefficient is odd), so
    # scale = 1/16 and zero = 0: the product is an exact small rational
    m, n = 515, 3072
    j, k = np.meshgrid(np.arange(m), np.arange(n), indexing="ij")
    W = (((3 * j + 5 * k) % 16) / 16.0).astype(np.float16)
    x = np.random.Generator(np.random.PCG64(8)).choice(np.array([1, -1, 2, -2, 0.5, -0.5], dtype=np.float16), n)
    p = binding.spqt_rowwise_pack(dev(W), 4, group)
    y = binding.spqt_rowwise_dense_gemv(p, dev(x))
    torch.cuda.synchronize()
    exact = W.astype(np.float64) @ x.astype(np.float64)
    assert np.array_equal(y.cpu().numpy(), exact.astype(np.float16))
    assert np.array_equal(exact.astype(np.float16).astype(np.float64), exact)   # the exact result is an fp16 value


def test_rowwise_baseline_refuses_what_it_does_not_cover():
    L = binding.lib()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    a = buf.data_ptr()
    assert L.spqt_rowwise_pack(a, 8, 100, 100, 4, 128, a, a, None) == 2          # n not a multiple of the group
    assert L.spqt_rowwise_pack(a, 8, 128, 128, 3, 128, a, a, None) == 2          # 4-bit only
    assert L.spqt_rowwise_dense_gemv(a, a, 8, 16384 + 128, 4, 128, a, a, None) == 2
    assert L.spqt_rowwise_dense_gemv(a, a, 8, 128, 4, 128, None, a, None) == 1
    assert L.spqt_rowwise_dense_gemv(a + 4, a, 8, 128, 4, 128, a, a, None) == 3


# ---------------------------------------------------------------- two-level format (6-bit block scales and minimums)

@pytest.mark.parametrize("m_blocks,n", [(1, 1), (1, 300), (2, 1111), (16, 4096), (4, 14336), (56, 1024)])
def test_kq_pack_bytes_and_products_match_the_oracle(m_blocks, n):
    m = 256 * m_blocks
    W = inputs.weights(m, n, seed=9 * m_blocks + n)
    if n >= 300:
        W[:32, 0] = np.abs(W[:32, 0])                     # a block without negative weights: minimum field 0
        W[:256, 1] = np.float16(0.0)                      # an all-zero superblock
        W[:256, 2] = np.float16(-0.0)
        W[32:64, 3] = np.float16(0.125)                   # a constant block
    x = inputs.activations(n, seed=m_blocks + 70, dist="gauss" if n > 8192 else "laplace")
    q, sc, mn, d, dmin = oracle.kq_quantize(W)
    p = binding.spqt_kq_pack(dev(W))
    torch.cuda.synchronize()
    got = p.records.cpu().numpy()
    want = oracle.kq_pack(q, sc, mn, d, dmin)
    assert np.array_equal(got, want), "first differing byte %d" % int(np.nonzero(got != want)[0][0])
    ws = binding.new_kq_workspace(p)
    xd = dev(x)
    for sp in (0.5, 0.9, 0.0, None):
        t = float("inf") if sp is None else inputs.threshold_for_sparsity(x, sp)
        idx, cnt = binding.spqt_sparsify(xd, t)
        y = torch.full((m,), float("nan"), dtype=torch.float16, device="cuda")
        binding.spqt_kq_sparse_gemv(p, xd, idx, cnt, ws, y)
        torch.cuda.synchronize()
        c = int(cnt.item())
        y_ref, bound = oracle.kq_gemv(q, sc, mn, d, dmin, x, idx.cpu().numpy()[:c])
        check_y(y.cpu().numpy(), y_ref, bound, "two-level sparse, sparsity %r" % sp)
        y2 = binding.spqt_kq_sparse_gemv(p, xd, idx, cnt, ws)
        torch.cuda.synchronize()
        assert torch.equal(y.view(torch.int16), y2.view(torch.int16))           # fixed order of sums
    yd = binding.spqt_kq_dense_gemv(p, xd, ws)
    torch.cuda.synchronize()
    y_ref, bound = oracle.kq_gemv(q, sc, mn, d, dmin, x)
    check_y(yd.cpu().numpy(), y_ref, bound, "two-level dense")
    assert not ws[: 4 * m_blocks].any()                                        # arrival counters back at zero


def test_kq_llama_shape_on_sampled_rows_and_a_shuffled_list():
    m, n = 14336, 4096
    W = inputs.weights(m, n, seed=77)
    x = inputs.activations(n, seed=78)
    q, sc, mn, d, dmin = oracle.kq_quantize(W)
    p = binding.spqt_kq_pack(dev(W))
    ws = binding.new_kq_workspace(p)
    t = inputs.threshold_for_sparsity(x, 0.5)
    xd = dev(x)
    idx, cnt = binding.spqt_sparsify(xd, t)
    torch.cuda.synchronize()
    c = int(cnt.item())
    perm = np.random.Generator(np.random.PCG64(5)).permutation(c)
    idx[:c] = idx[:c][torch.from_numpy(perm).cuda()]
    y = binding.spqt_kq_sparse_gemv(p, xd, idx, cnt, ws)
    torch.cuda.synchronize()
    rows = np.unique(np.random.Generator(np.random.PCG64(6)).integers(0, m, size=256))
    y_ref, bound = oracle.kq_gemv(q, sc, mn, d, dmin, x, idx.cpu().numpy()[:c], rows=rows)
    check_y(y.cpu().numpy()[rows], y_ref, bound, "two-level 14336x4096")


def test_kq_refuses_what_it_does_not_cover():
    L = binding.lib()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    a = buf.data_ptr()
    assert L.spqt_kq_pack(a, 128, 8, 8, a, None) == 2                        # m not a multiple of 256
    assert L.spqt_kq_dense_gemv(a, 256, 8, a, a, a, 16, None) == 4           # workspace too small
    assert L.spqt_kq_sparse_gemv(a, 256, 8, a, None, a, a, a, 1 << 16, None) == 1
    assert L.spqt_kq_dense_gemv(a + 8, 256, 8, a, a, a, 1 << 16, None) == 3


@pytest.mark.parametrize("bits", [2, 5, 6, 8])
@pytest.mark.parametrize("m_blocks,n", [(1, 1), (2, 1111), (16, 4096), (4, 14336)])
def test_kq_other_code_widths_match_the_oracle(bits, m_blocks, n):
    """The two-level format with 2-, 5-, 6- and 8-bit codes: record bytes identical to the oracle's, sparse and dense
    products within the tolerance, repeated calls bit-identical."""
    m = 256 * m_blocks
    W = inputs.weights(m, n, seed=5 * m_blocks + n + bits)
    if n >= 300:
        W[:32, 0] = np.abs(W[:32, 0])
        W[:256, 1] = np.float16(0.0)
        W[:256, 2] = np.float16(-0.0)
        W[32:64, 3] = np.float16(0.125)
    x = inputs.activations(n, seed=m_blocks + 90, dist="gauss" if n > 8192 else "laplace")
    q, sc, mn, d, dmin = oracle.kq_quantize(W, bits=bits)
    p = binding.spqt_kqw_pack(dev(W), bits)
    torch.cuda.synchronize()
    got = p.records.cpu().numpy()
    want = oracle.kq_pack(q, sc, mn, d, dmin, bits=bits)
    assert got.size == want.size == m_blocks * n * oracle.kq_record_bytes(bits=bits)
    assert np.array_equal(got, want), "first differing byte %d" % int(np.nonzero(got != want)[0][0])
    ws = binding.new_kq_workspace(p)
    xd = dev(x)
    for sp in (0.5, 0.9, 0.0, None):
        t = float("inf") if sp is None else inputs.threshold_for_sparsity(x, sp)
        idx, cnt = binding.spqt_sparsify(xd, t)
        y = torch.full((m,), float("nan"), dtype=torch.float16, device="cuda")
        binding.spqt_kqw_sparse_gemv(p, xd, idx, cnt, ws, y)
        torch.cuda.synchronize()
        c = int(cnt.item())
        y_ref, bound = oracle.kq_gemv(q, sc, mn, d, dmin, x, idx.cpu().numpy()[:c])
        check_y(y.cpu().numpy(), y_ref, bound, "two-level %d-bit sparse, sparsity %r" % (bits, sp))
        y2 = binding.spqt_kqw_sparse_gemv(p, xd, idx, cnt, ws)
        torch.cuda.synchronize()
        assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    yd = binding.spqt_kqw_dense_gemv(p, xd, ws)
    torch.cuda.synchronize()
    y_ref, bound = oracle.kq_gemv(q, sc, mn, d, dmin, x)
    check_y(yd.cpu().numpy(), y_ref, bound, "two-level %d-bit dense" % bits)
    assert not ws[: 4 * m_blocks].any()


def test_kq_width_four_is_the_plain_format_and_other_widths_are_refused():
    W = inputs.weights(512, 300, seed=3)
    a = binding.spqt_kq_pack(dev(W))
    b = binding.spqt_kqw_pack(dev(W), 4)
    torch.cuda.synchronize()
    assert torch.equal(a.records, b.records)
    L = binding.lib()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    p = buf.data_ptr()
    for bits in (1, 3, 7, 16):
        assert L.spqt_kqw_pack(p, 256, 8, 8, bits, p, None) == 2
        assert L.spqt_kqw_dense_gemv(p, 256, 8, bits, p, p, p, 1 << 16, None) == 2
    assert binding.spqt_kqw_packed_sizes(512, 10, 2)[0] == 2 * 10 * 80
    assert binding.spqt_kqw_packed_sizes(512, 10, 8)[0] == 2 * 10 * 272
    assert binding.spqt_kqw_packed_sizes(512, 10, 5)[0] == 2 * 10 * 176
    assert binding.spqt_kqw_packed_sizes(512, 10, 6)[0] == 2 * 10 * 208


@pytest.mark.parametrize("seed", [1, 2])
def test_random_shapes_across_the_partition_regimes(seed):
    """Seeded random cases over the regimes of the work map -- block-rows far below, near and above the SM count,
    lists that fit the shared-memory window and lists that do not, every format, thresholds from 0 to 99 % -- through
    the given-list, index-collecting and dense calls: lists bit-exact, the two sparse routes bit-identical, sampled
    rows against the oracle."""
    rng = np.random.default_rng(seed)
    for it in range(12):
        bits, group = GEMV_FORMATS[it % 4]
        R = int(rng.choice([1, 2, 7, 31, 74, 147, 148, 149, 160, 223, 296, 300, 451, 1000]))
        n = int(rng.choice([64, 777, 4096, 5000, 12288, 12289, 20001, 32768]))
        if R * group * n > 3e8:
            n = 4096
        m = R * group
        sp = float(rng.choice([0.0, 0.1, 0.5, 0.9, 0.99]))
        torch.manual_seed(100 * seed + it)
        Wd = (torch.randn(m, n, device="cuda") * 0.02).half()
        x = inputs.activations(n, seed=1000 * seed + it)
        t = inputs.threshold_for_sparsity(x, sp)
        p = binding.spqt_pack(Wd, bits, group)
        del Wd
        ws = binding.new_workspace(m, n, bits, group)
        xd = dev(x)
        idx, cnt = binding.spqt_sparsify(xd, t)
        y = binding.spqt_sparse_gemv(p, xd, idx, cnt, ws)
        yf, idx2, cnt2 = binding.spqt_sparsify_gemv(p, xd, t, ws)
        yd = binding.spqt_dense_gemv(p, xd, ws)
        torch.cuda.synchronize()
        what = "int%d g%d R=%d n=%d sparsity %.2f" % (bits, group, R, n, sp)
        ref_idx, ref_cnt = oracle.sparsify(x, t)
        assert int(cnt.item()) == ref_cnt and int(cnt2.item()) == ref_cnt, what
        assert np.array_equal(idx.cpu().numpy()[:ref_cnt], ref_idx) and np.array_equal(idx2.cpu().numpy()[:ref_cnt], ref_idx), what
        assert torch.equal(y.view(torch.int16), yf.view(torch.int16)), what
        rows = np.unique(rng.integers(0, m, size=64))
        codes, s, z = packed_to_host(p)
        y_ref, bound = oracle.sparse_gemv(codes, s, z, m, n, x, ref_idx, bits, group, rows=rows)
        check_y(y.cpu().numpy()[rows], y_ref, bound, what)
        y_ref, bound = oracle.dense_gemv(codes, s, z, m, n, x, bits, group, rows=rows)
        check_y(yd.cpu().numpy()[rows], y_ref, bound, what + " dense")
        assert binding.spqt_workspace_status(ws, m, group) == 0, what
        del p, ws
        torch.cuda.empty_cache()
