"""Pins for the CPU oracle: every check here compares the oracle with something
other than itself -- a hand-worked example, a closed form, a library routine,
exact integer/rational arithmetic, or an invariant the mathematics fixes."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from conftest import read_golden
from paper_2511_04477_b200 import inputs


# ------------------------------------------------------------------ fp16 conversions

def test_half_to_float_matches_numpy_exhaustively():
    bits = np.arange(65536, dtype=np.uint16)
    mine = oracle.half_to_float(bits)
    ref = bits.view(np.float16).astype(np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(mine), nan)
    assert np.array_equal(mine[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_float_to_half_matches_numpy():
    g = np.random.Generator(np.random.PCG64(7))
    # random bit patterns cover every exponent; add the rounding boundaries explicitly
    f = g.integers(0, 2**32, size=2_000_000, dtype=np.uint64).astype(np.uint32).view(np.float32)
    h = np.arange(65536, dtype=np.uint16).view(np.float16).astype(np.float32)
    h = h[np.isfinite(h)]
    up = np.nextafter(h, np.float32(np.inf))
    mid = ((h.astype(np.float64) + np.roll(h, -1).astype(np.float64)) / 2).astype(np.float32)
    edge = np.array([65504, 65519.996, 65520, 65536, 1e-8, 2.0**-25, 2.0**-24, 3 * 2.0**-25,
                     2.0**-14, 2.0**-14 - 2.0**-25, 0.0, -0.0, np.inf, -np.inf], dtype=np.float32)
    allf = np.concatenate([f, h, up, mid, -mid, edge])
    allf = allf[~np.isnan(allf)]
    with np.errstate(over="ignore"):
        ref = allf.astype(np.float16).view(np.uint16)
    assert np.array_equal(oracle.float_to_half(allf), ref)


# ------------------------------------------------------------------ hand-worked example

def test_hand_example_quantizer_and_layout(hand_example):
    e = hand_example
    q, s, z = oracle.quantize(e["W"], e["bits"], e["group"])
    assert np.array_equal(q, e["q"])
    assert np.array_equal(s.astype(np.float64), e["scales"])
    assert np.array_equal(z.astype(np.float64), e["zeros"])
    assert s[0, 2].view(np.uint16) == 0x3266
    codes = oracle.pack_codes(q, e["bits"], e["group"])
    assert codes.tolist() == e["codes"].tolist()
    assert np.array_equal(oracle.unpack_codes(e["codes"], e["m"], e["n"], e["bits"], e["group"]), e["q"])


def test_hand_example_sparse_and_dense_gemv(hand_example):
    e = hand_example
    codes, s, z = oracle.pack(e["W"], e["bits"], e["group"])
    idx, count = oracle.sparsify(e["x"], e["t"])
    assert count == 2 and idx.tolist() == e["idx"].tolist()
    y, bound = oracle.sparse_gemv(codes, s, z, e["m"], e["n"], e["x"], idx, e["bits"], e["group"])
    assert np.array_equal(y, e["y_sparse"])            # exact, not approximate
    yd, _ = oracle.dense_gemv(codes, s, z, e["m"], e["n"], e["x"], e["bits"], e["group"])
    assert np.array_equal(yd, e["y_dense"])
    # bound of row 0: |0|*1 + |2|*2 = 4 ; row 7: |0.875|*1 + |-1.5|*2 = 3.875
    assert bound[0] == 4.0 and bound[7] == 3.875


def test_int3_block_bytes_match_hand_packing():
    g = read_golden("int3_block.txt")
    G, bits = int(g["group"][0][0]), int(g["bits"][0][0])
    col = np.array([[float(v)] for v in g["column"][0]], dtype=np.float16)
    q, s, z = oracle.quantize(col, bits, G)
    assert q[:, 0].tolist() == list(range(8))
    assert float(s[0, 0]) == float(g["scale"][0][0]) and float(z[0, 0]) == float(g["zero"][0][0])
    codes = oracle.pack_codes(q, bits, G)
    assert codes.tolist() == [int(v, 16) for v in g["codes"][0]]
    assert oracle.block_bytes(3, 128) == 48 and oracle.block_bytes(3, 64) == 24
    assert oracle.block_bytes(4, 128) == 64 and oracle.block_bytes(4, 64) == 32


# ------------------------------------------------------------------ layout structure

@pytest.mark.parametrize("bits,group", [(4, 128), (4, 64), (3, 128), (3, 64), (4, 6), (3, 16)])
def test_pack_unpack_round_trip_bit_exact(bits, group):
    g = np.random.Generator(np.random.PCG64(bits * 1000 + group))
    m, n = 3 * group, 37
    q = g.integers(0, 1 << bits, size=(m, n), dtype=np.uint8)
    codes = oracle.pack_codes(q, bits, group)
    assert codes.size == 3 * n * group * bits // 8
    assert np.array_equal(oracle.unpack_codes(codes, m, n, bits, group), q)


@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64)])
def test_block_of_row_j_column_k_lives_at_r_times_n_plus_k(bits, group):
    """Zigzag order: changing one weight's code touches only bytes of block (j//G, k),
    and block index is r*n + k (row-major over (block-row, column))."""
    m, n = 2 * group, 9
    B = oracle.block_bytes(bits, group)
    base = oracle.pack_codes(np.zeros((m, n), np.uint8), bits, group)
    assert not base.any()
    for (j, k) in [(0, 0), (5, 3), (group - 1, 8), (group, 0), (group + 17, 4), (2 * group - 1, 8)]:
        q = np.zeros((m, n), np.uint8)
        q[j, k] = (1 << bits) - 1
        changed = np.nonzero(oracle.pack_codes(q, bits, group))[0]
        blk = (j // group) * n + k
        assert changed.size > 0
        assert changed.min() >= blk * B and changed.max() < (blk + 1) * B
    # int4: byte i of a block = row i in the low nibble, row i + G/2 in the high nibble
    if bits == 4:
        q = np.zeros((m, n), np.uint8)
        q[3, 2] = 0x9
        q[3 + group // 2, 2] = 0x6
        c = oracle.pack_codes(q, bits, group)
        assert c[(0 * n + 2) * B + 3] == 0x69


# ------------------------------------------------------------------ quantizer invariants

@pytest.mark.parametrize("bits,group", [(4, 128), (4, 64), (3, 128), (3, 64)])
def test_quantizer_invariants(bits, group):
    qmax = (1 << bits) - 1
    W = inputs.weights(2 * group, 96, seed=11 + bits + group)
    W[:group, 5] = np.float16(0.03125)                     # a constant group
    q, s, z = oracle.quantize(W, bits, group)
    Wf = W.astype(np.float64)
    for r in range(2):
        blk = Wf[r * group:(r + 1) * group]
        assert np.array_equal(z[r].astype(np.float64), blk.min(axis=0))          # offset = group min
        qb = q[r * group:(r + 1) * group]
        amin, amax = blk.argmin(axis=0), blk.argmax(axis=0)
        cols = np.arange(W.shape[1])
        sf = s[r].astype(np.float64)
        assert np.all(qb[amin, cols] == 0)                                       # min -> code 0
        assert np.all((qb[amax, cols] == qmax) | (sf == 0))                      # max -> qmax
        deq = sf[None, :] * qb + z[r].astype(np.float64)[None, :]
        assert np.all(np.abs(deq - blk) <= sf[None, :] / 2 * (1 + 2.0**-10) + 1e-300)
        # scale is the fp16 rounding of range/qmax computed in fp32
        rng32 = (blk.max(axis=0).astype(np.float32) - blk.min(axis=0).astype(np.float32))
        assert np.array_equal(s[r], (rng32 / np.float32(qmax)).astype(np.float16))
    assert s[0, 5] == 0 and not q[:group, 5].any() and float(z[0, 5]) == 0.03125
    assert q.max() <= qmax
    # power-of-two scaling leaves the codes alone and scales s and z
    q2, s2, z2 = oracle.quantize((W.astype(np.float32) * 4).astype(np.float16), bits, group)
    assert np.array_equal(q2, q)
    assert np.array_equal(s2.astype(np.float32), s.astype(np.float32) * 4)
    assert np.array_equal(z2.astype(np.float32), z.astype(np.float32) * 4)


def test_zero_minimum_is_stored_as_plus_zero_whatever_the_signs_and_order():
    """A group whose minimum is zero with both signs present (pruned weights): the offset is +0.0
    (bits 0x0000) for every order of the rows, and the codes are those of the non-negative values
    divided by the scale (the sign of a zero changes no quotient)."""
    group, bits = 4, 4
    pos = np.array([0.0, 0.5, 1.5, 0.0], np.float16)
    for first_zero, other_zero in ((np.float16(-0.0), np.float16(0.0)), (np.float16(0.0), np.float16(-0.0))):
        col = pos.copy()
        col[0], col[3] = first_zero, other_zero
        assert np.signbit(col[0]) != np.signbit(col[3])
        q, s, z = oracle.quantize(col.reshape(group, 1), bits, group)
        assert z.view(np.uint16)[0, 0] == 0x0000
        assert float(s[0, 0]) == 0.0999755859375            # fp16(1.5 / 15)
        assert q[:, 0].tolist() == [0, 5, 15, 0]
    # all zeros of either sign: constant group, scale 0, offset +0.0
    q, s, z = oracle.quantize(np.array([[-0.0], [-0.0], [0.0], [-0.0]], np.float16), bits, group)
    assert z.view(np.uint16)[0, 0] == 0x0000 and s.view(np.uint16)[0, 0] == 0x0000 and not q.any()


def test_quantizer_codes_match_numpy_single_precision_steps():
    """Same steps taken with numpy's IEEE float32 ufuncs (a different engine)."""
    bits, group, qmax = 4, 128, 15
    W = inputs.weights(256, 64, seed=3)
    q, s, z = oracle.quantize(W, bits, group)
    w32 = W.astype(np.float32).reshape(2, group, 64)
    lo = w32.min(axis=1, keepdims=True)
    sf = s.astype(np.float32)[:, None, :]
    with np.errstate(divide="ignore", invalid="ignore"):
        ref = np.clip(np.rint((w32 - lo) / sf), 0, qmax)
    ref = np.where(sf == 0, 0, ref).astype(np.uint8).reshape(256, 64)
    assert np.array_equal(q, ref)


def test_lossless_family_is_reproduced_exactly():
    W = inputs.lossless_weights(256, 40)
    codes, s, z = oracle.pack(W, 4, 128)
    assert np.all(s.astype(np.float64) == 1 / 16) and not z.any()
    assert np.array_equal(oracle.dequantize(codes, s, z, 256, 40, 4, 128), W.astype(np.float64))


def test_expected_scale_for_gaussian_weights():
    """W ~ N(0, 0.02^2), G = 128: E[range] = 2*E[max of 128 normals]*sigma ~ 5.2 sigma,
    so the mean scale is about 5.2*0.02/15 ~ 0.0069."""
    _, s, _ = oracle.quantize(inputs.weights(128 * 8, 512, seed=0), 4, 128)
    assert abs(float(s.astype(np.float64).mean()) - 0.0069) < 3e-4


# ------------------------------------------------------------------ dequantize / GEMV definitions

def _setup(m, n, bits, group, seed, dist="laplace", **kw):
    W = inputs.weights(m, n, seed)
    x = inputs.activations(n, seed + 100, dist, **kw)
    q, s, z = oracle.quantize(W, bits, group)
    codes = oracle.pack_codes(q, bits, group)
    return W, x, q, s, z, codes


@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64), (4, 64), (3, 128)])
def test_dequantize_is_scale_times_code_plus_offset(bits, group):
    m, n = 2 * group, 33
    _, _, q, s, z, codes = _setup(m, n, bits, group, seed=5)
    What = oracle.dequantize(codes, s, z, m, n, bits, group)
    ref = (np.repeat(s.astype(np.float64), group, axis=0) * q.astype(np.float64)
           + np.repeat(z.astype(np.float64), group, axis=0))
    assert np.array_equal(What, ref)


@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64)])
def test_threshold_at_or_below_zero_equals_dense_matrix_product(bits, group):
    m, n = 2 * group, 200
    _, x, q, s, z, codes = _setup(m, n, bits, group, seed=9)
    x[[3, 50]] = np.float16(0.0)
    x[7] = np.float16(-0.0)
    What = (np.repeat(s.astype(np.float64), group, axis=0) * q
            + np.repeat(z.astype(np.float64), group, axis=0))
    ref = What @ x.astype(np.float64)                       # library matmul on the m x n matrix
    for t in (0.0, -1.0):
        idx, cnt = oracle.sparsify(x, t)
        assert cnt == (n - 3 if t == 0.0 else n)            # +-0 is not above 0
        y, b = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
        assert np.allclose(y, ref, rtol=0, atol=1e-12 * np.abs(What).sum(axis=1).max() * 10)
    yd, bd = oracle.dense_gemv(codes, s, z, m, n, x, bits, group)
    assert np.allclose(yd, ref, rtol=0, atol=1e-11)
    assert np.allclose(bd, np.abs(What) @ np.abs(x.astype(np.float64)), rtol=1e-13)


def test_tiny_matrix_brute_force_in_exact_rationals():
    bits, group, m, n = 4, 4, 8, 5
    g = np.random.Generator(np.random.PCG64(42))
    W = (g.integers(-40, 40, size=(m, n)) / 16.0).astype(np.float16)
    x = (g.integers(-6, 7, size=n) / 4.0).astype(np.float16)
    t = 0.5
    q, s, z = oracle.quantize(W, bits, group)
    codes = oracle.pack_codes(q, bits, group)
    idx, cnt = oracle.sparsify(x, t)
    y, bound = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    active = [k for k in range(n) if abs(Fraction(float(x[k]))) > Fraction(t)]
    assert idx.tolist() == active and cnt == len(active)
    for j in range(m):
        r = j // group
        acc = sum((Fraction(float(s[r, k])) * int(q[j, k]) + Fraction(float(z[r, k]))) * Fraction(float(x[k]))
                  for k in active)
        bnd = sum(abs(Fraction(float(s[r, k])) * int(q[j, k]) + Fraction(float(z[r, k]))) * abs(Fraction(float(x[k])))
                  for k in active)
        assert abs(Fraction(y[j]) - acc) <= Fraction(1, 10**12) * (bnd + 1)
        assert abs(Fraction(bound[j]) - bnd) <= Fraction(1, 10**12) * (bnd + 1)


def test_one_hot_probe_returns_the_column():
    bits, group, m, n = 4, 128, 256, 130
    _, _, q, s, z, codes = _setup(m, n, bits, group, seed=21)
    for k in (0, 1, 64, 129):
        x = np.zeros(n, np.float16)
        x[k] = np.float16(-1.5)
        idx, cnt = oracle.sparsify(x, 0.25)
        assert idx.tolist() == [k]
        y, b = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
        col = (np.repeat(s[:, k].astype(np.float64), group) * q[:, k] + np.repeat(z[:, k].astype(np.float64), group))
        assert np.array_equal(y, -1.5 * col)
        assert np.array_equal(b, 1.5 * np.abs(col))


@pytest.mark.parametrize("bits,group", [(4, 128), (4, 64), (3, 128), (3, 64)])
def test_lossless_family_gemv_equals_integer_arithmetic(bits, group):
    m, n, levels = 256, 300, 1 << bits
    W = inputs.lossless_weights(m, n, levels=levels)
    x = inputs.small_rational_activations(n, seed=4)
    codes, s, z = oracle.pack(W, bits, group)
    assert np.all(s.astype(np.float64) == 1.0 / levels) and not z.any()
    t = 0.75                                               # drops the +-0.5 entries
    idx, cnt = oracle.sparsify(x, t)
    keep = np.abs(x.astype(np.float64)) > t
    assert np.array_equal(idx, np.nonzero(keep)[0])
    j = np.arange(m)[:, None]
    k = np.arange(n)[None, :]
    num = ((5 * j + 3 * k) % levels).astype(np.int64)      # levels * W, integers
    x2 = np.rint(x.astype(np.float64) * 2).astype(np.int64)  # 2 * x, integers
    ref = (num[:, keep] @ x2[keep]) / (2.0 * levels)       # exact
    y, _ = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    assert np.array_equal(y, ref)


def test_order_invariance_superposition_and_row_subset():
    bits, group, m, n = 4, 128, 256, 257
    _, x, q, s, z, codes = _setup(m, n, bits, group, seed=33)
    idx, cnt = oracle.sparsify(x, 0.6)
    y, b = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group)
    perm = np.random.Generator(np.random.PCG64(1)).permutation(cnt)
    yp, bp = oracle.sparse_gemv(codes, s, z, m, n, x, idx[perm], bits, group)
    assert np.allclose(yp, y, rtol=0, atol=1e-13 * b.max())
    half = cnt // 2
    y1, _ = oracle.sparse_gemv(codes, s, z, m, n, x, idx[:half], bits, group)
    y2, _ = oracle.sparse_gemv(codes, s, z, m, n, x, idx[half:], bits, group)
    assert np.allclose(y1 + y2, y, rtol=0, atol=1e-13 * b.max())
    rows = np.array([0, 5, 127, 128, 255], np.int32)
    yr, br = oracle.sparse_gemv(codes, s, z, m, n, x, idx, bits, group, rows=rows)
    assert np.array_equal(yr, y[rows]) and np.array_equal(br, b[rows])
    yd, _ = oracle.dense_gemv(codes, s, z, m, n, x, bits, group)
    ydr, _ = oracle.dense_gemv(codes, s, z, m, n, x, bits, group, rows=rows)
    assert np.array_equal(ydr, yd[rows])


# ------------------------------------------------------------------ index collection

@pytest.mark.parametrize("n", [1, 31, 32, 33, 1000, 4096])
def test_index_list_matches_a_brute_force_scan(n):
    x = inputs.activations(n, seed=n, dist="laplace")
    if n > 40:
        x[5] = np.float16(np.nan)
        x[6] = np.float16(np.inf)
        x[7] = np.float16(-np.inf)
    for t in (-1.0, 0.0, 0.3, float(np.abs(x.astype(np.float32))[0]), 2.0, float("inf")):
        idx, cnt = oracle.sparsify(x, t)
        ref = [k for k in range(n) if abs(float(x[k])) > t]          # NaN compares false
        assert idx.tolist() == ref and cnt == len(ref)
        with np.errstate(invalid="ignore"):
            dropped = np.count_nonzero(np.abs(x.astype(np.float64)) <= t) + np.count_nonzero(np.isnan(x))
        assert cnt == n - dropped
    assert oracle.sparsify(x, float("inf"))[1] == 0
    assert oracle.sparsify(x, -1.0)[1] == n - int(np.isnan(x).sum())


def test_tie_at_the_threshold_is_dropped():
    x = np.array([0.5, -0.5, 0.5004883, 0.25, -0.75], dtype=np.float16)
    idx, cnt = oracle.sparsify(x, 0.5)
    assert idx.tolist() == [2, 4]


def test_partition_is_even_and_matches_the_papers_example():
    assert oracle.partition(9, 3).tolist() == [0, 3, 6, 9]       # 9 active entries, 3 workers
    for count, S in [(0, 4), (1, 4), (10, 4), (2048, 9), (7168, 37)]:
        b = oracle.partition(count, S)
        sizes = np.diff(b)
        assert b[0] == 0 and b[-1] == count and sizes.min() >= 0
        assert sizes.max() - sizes.min() <= 1


# ------------------------------------------------------------------ input generator closed forms

def test_laplace_and_gaussian_thresholds_match_closed_forms():
    xl = inputs.activations(200_000, seed=0, dist="laplace")
    xg = inputs.activations(200_000, seed=1, dist="gauss")
    # |Laplace(0,1)| ~ Exp(1): quantile -ln(1-p); |N(0,1)|: Phi^-1((1+p)/2)
    for p, ql, qg in [(0.25, 0.2877, 0.3186), (0.40, 0.5108, 0.5244), (0.50, math.log(2), 0.6745), (0.90, 2.3026, 1.6449)]:
        assert abs(inputs.threshold_for_sparsity(xl, p) - ql) < 0.02
        assert abs(inputs.threshold_for_sparsity(xg, p) - qg) < 0.02
    x = inputs.activations(4096, seed=0)
    t = inputs.threshold_for_sparsity(x, 0.5)
    idx, cnt = oracle.sparsify(x, t)
    assert cnt <= 2048 and cnt >= 2048 - 8                 # ties at t only ever drop more
    assert abs(inputs.realised_sparsity(x, t) - (1 - cnt / 4096)) < 1e-12
    assert inputs.threshold_for_sparsity(x, 0.0) == -1.0


def test_outlier_recipe():
    x0 = inputs.activations(8192, seed=2)
    x1 = inputs.activations(8192, seed=2, outlier_frac=0.01, outlier_scale=20.0)
    changed = np.nonzero(x0 != x1)[0]
    assert 70 <= changed.size <= 82
    assert np.allclose(x1[changed].astype(np.float32), 20 * x0[changed].astype(np.float32), rtol=2e-3)


# ------------------------------------------------------------------ threshold calibration

def test_calibration_threshold_hand_example_and_rank_property():
    pool = np.array([0.5, -2.0, 1.0, 0.25, np.nan, -0.25], np.float16)     # N = 5 entries that are not NaN
    assert oracle.calibrate_threshold(pool, 0.5) == 0.5                      # rank ceil(2.5) = 3 of .25 .25 .5 1 2
    assert oracle.calibrate_threshold(pool, 0.4) == 0.25                     # rank 2
    assert oracle.calibrate_threshold(pool, 1.0) == 2.0
    assert oracle.calibrate_threshold(pool, 0.0) == -1.0
    assert oracle.calibrate_threshold(np.zeros(0, np.float16), 0.5) == -1.0
    g = np.random.Generator(np.random.PCG64(5))
    x = g.standard_normal(5000).astype(np.float16)
    a = np.abs(x.astype(np.float64))
    for s in (0.1, 0.25, 0.5, 0.9, 0.999):
        t = oracle.calibrate_threshold(x, s)
        rank = math.ceil(s * x.size - 1e-9)
        assert np.count_nonzero(a <= t) >= rank > np.count_nonzero(a < t)   # t is the rank-th smallest magnitude
        idx, cnt = oracle.sparsify(x, t)
        assert x.size - cnt >= rank                                          # at least that many entries are dropped


def test_calibration_threshold_matches_closed_forms_and_group_mean():
    g = np.random.Generator(np.random.PCG64(6))
    lap = g.laplace(0.0, 1.0, size=400_000).astype(np.float16)
    assert abs(oracle.calibrate_threshold(lap, 0.5) - math.log(2.0)) < 0.01
    assert abs(oracle.calibrate_threshold(lap, 0.25) - 0.2877) < 0.01
    gau = g.standard_normal(400_000).astype(np.float16)
    assert abs(oracle.calibrate_threshold(gau, 0.5) - 0.6745) < 0.01
    assert oracle.group_sparsity([0.3, 0.5, 0.4]) == pytest.approx(0.4, abs=1e-15)
    assert oracle.group_sparsity([0.5]) == 0.5


# ------------------------------------------------------------------ small batch over the union of active sets

def test_union_of_active_sets_matches_a_brute_force_scan():
    g = np.random.Generator(np.random.PCG64(21))
    X = g.standard_normal((5, 300)).astype(np.float16)
    X[:, 7] = np.float16(0.1)                  # column 7: below the threshold in every row, NaN in one
    X[1, 7] = np.float16(np.nan)
    X[:, 9] = np.float16(0.0)                  # column 9: active through one row only
    X[0, 9] = np.float16(-np.inf)
    t = 1.2
    idx, cnt = oracle.union_sparsify(X, t)
    brute = [k for k in range(300) if any(abs(float(X[b, k])) > t for b in range(5))]   # NaN compares false
    assert cnt == len(brute) and idx.tolist() == brute
    assert 9 in brute and 7 not in brute
    one, c1 = oracle.union_sparsify(X[:1], t)
    ref, c2 = oracle.sparsify(X[0], t)
    assert c1 == c2 and np.array_equal(one, ref)            # a batch of one is the plain index collection


def test_small_batch_rows_are_products_over_the_union_in_exact_rationals():
    m, n, bits, group, B = 8, 6, 4, 4, 3
    g = np.random.Generator(np.random.PCG64(22))
    W = (g.integers(-8, 8, size=(m, n)) / 8.0).astype(np.float16)
    X = (g.integers(-4, 5, size=(B, n)) / 2.0).astype(np.float16)
    codes, s, z = oracle.pack(W, bits, group)
    What = oracle.dequantize(codes, s, z, m, n, bits, group)
    t = 0.75
    idx, cnt = oracle.union_sparsify(X, t)
    Y, bound = oracle.sparse_gemm_small(codes, s, z, m, n, X, idx, bits, group)
    for b in range(B):
        for j in range(m):
            ref = sum(Fraction(float(What[j, k])) * Fraction(float(X[b, k])) for k in idx)
            assert Fraction(float(Y[b, j])) == ref
            assert Fraction(float(bound[b, j])) == sum(abs(Fraction(float(What[j, k])) * Fraction(float(X[b, k]))) for k in idx)
    # rows that are all the same give the single-row product in every row
    Xs = np.repeat(X[:1], 4, axis=0)
    i1, c1 = oracle.sparsify(X[0], t)
    iu, cu = oracle.union_sparsify(Xs, t)
    assert np.array_equal(i1, iu)
    y1, _ = oracle.sparse_gemv(codes, s, z, m, n, X[0], i1, bits, group)
    Ys, _ = oracle.sparse_gemm_small(codes, s, z, m, n, Xs, iu, bits, group)
    assert all(np.array_equal(Ys[b], y1) for b in range(4))


# ---------------------------------------------------------------- row-wise baseline layout (Sec. 2, Sec. 4.1.1)

def test_rowwise_hand_example():
    # The two groups of the hand-worked example (tests/golden/hand_example.txt, columns 0 and 2 of
    # block-row 0), laid along rows instead of down columns: same scales, offsets and codes.
    W = np.array([[0.0, 0.25, 0.5, 3.75], [1.0, 2.0, 3.0, 4.0]], dtype=np.float16)
    q, s, z = oracle.rowwise_quantize(W, 4, 4)
    assert q.tolist() == [[0, 1, 2, 15], [0, 5, 10, 15]]
    assert s.shape == (2, 1) and z.shape == (2, 1)
    assert float(s[0, 0]) == 0.25 and float(z[0, 0]) == 0.0
    assert s.view(np.uint16)[1, 0] == 0x3266 and float(z[1, 0]) == 1.0
    # bytes of a block: byte i = code i | code i+2 << 4 (group of 4)
    assert oracle.rowwise_pack_codes(q, 4, 4).tolist() == [0x20, 0xF1, 0xA0, 0xF5]
    x = np.array([1.0, -2.0, 0.5, 1.0], dtype=np.float16)
    y, bound = oracle.rowwise_dense_gemv(q, s, z, x, 4)
    assert y[0] == 0.0 - 0.5 + 0.25 + 3.75
    s1 = 0.199951171875
    assert y[1] == (1 + 0 * s1) * 1 + (1 + 5 * s1) * -2 + (1 + 10 * s1) * 0.5 + (1 + 15 * s1) * 1
    assert bound[0] == 0.5 + 0.25 + 3.75


def test_rowwise_thresholded_product_drops_exactly_the_inactive_entries():
    W = np.array([[0.0, 0.25, 0.5, 3.75], [1.0, 2.0, 3.0, 4.0]], dtype=np.float16)
    q, s, z = oracle.rowwise_quantize(W, 4, 4)
    x = np.array([1.0, -2.0, 0.5, np.nan], dtype=np.float16)
    y, bound = oracle.rowwise_thresholded_gemv(q, s, z, x, 0.75, 4)          # active: columns 0 and 1
    assert y[0] == 0.0 * 1 + 0.25 * -2 and bound[0] == 0.5
    s1 = 0.199951171875
    assert y[1] == (1 + 0 * s1) * 1 + (1 + 5 * s1) * -2
    y0, _ = oracle.rowwise_thresholded_gemv(q, s, z, np.array([1.0, -2.0, 0.5, 0.0], np.float16), -1.0, 4)
    yd, _ = oracle.rowwise_dense_gemv(q, s, z, np.array([1.0, -2.0, 0.5, 0.0], np.float16), 4)
    assert np.array_equal(y0, yd)


def test_rowwise_quantizer_brute_force():
    # per row and per group of consecutive columns, the quantizer's steps in numpy float32
    rng = np.random.default_rng(11)
    m, n, G = 5, 24, 8
    W = (rng.standard_normal((m, n)) * 0.05).astype(np.float16)
    q, s, z = oracle.rowwise_quantize(W, 4, G)
    for j in range(m):
        for g in range(n // G):
            w = W[j, g * G:(g + 1) * G].astype(np.float32)
            lo, hi = np.float32(w.min()), np.float32(w.max())
            sc = np.float16(np.float32(hi - lo) / np.float32(15))
            assert s[j, g] == sc and z[j, g] == np.float16(lo)
            sf = np.float32(sc)
            codes = np.clip(np.rint((w - lo) / sf), 0, 15).astype(np.uint8) if sf != 0 else np.zeros(G, np.uint8)
            assert q[j, g * G:(g + 1) * G].tolist() == codes.tolist()


def test_rowwise_layout_and_product_exact():
    from fractions import Fraction
    rng = np.random.default_rng(12)
    m, n, G = 3, 16, 8
    W = (rng.standard_normal((m, n)) * 0.1).astype(np.float16)
    x = rng.choice(np.array([1.0, -2.0, 0.5, 0.0, 3.0], dtype=np.float16), n)
    q, s, z = oracle.rowwise_quantize(W, 4, G)
    codes = oracle.rowwise_pack_codes(q, 4, G)
    B = G // 2
    assert codes.size == m * (n // G) * B
    for j in range(m):
        for g in range(n // G):
            blk = codes[(j * (n // G) + g) * B:(j * (n // G) + g + 1) * B]
            for i in range(B):
                assert blk[i] == (q[j, g * G + i] | (q[j, g * G + i + B] << 4))
    y, _ = oracle.rowwise_dense_gemv(q, s, z, x, G)
    for j in range(m):
        acc = Fraction(0)
        for k in range(n):
            acc += (Fraction(float(s[j, k // G])) * int(q[j, k]) + Fraction(float(z[j, k // G]))) * Fraction(float(x[k]))
        assert abs(float(acc) - y[j]) <= 1e-12 * max(1.0, abs(float(acc)))


# ---------------------------------------------------------------- two-level format (Sec. 2: 6-bit block scales/minimums)

def _golden_kq(name="kq_superblock.txt"):
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = vals
    return out


def test_kq_hand_worked_superblock():
    g = _golden_kq()
    W = np.array([float(v) for v in g["w"]], dtype=np.float16).reshape(8, 1)
    q, sc, mn, d, dmin = oracle.kq_quantize(W, 4, 2)
    assert q.ravel().tolist() == [int(v) for v in g["q"]]
    assert sc.ravel().tolist() == [int(v) for v in g["sc"]] and mn.ravel().tolist() == [int(v) for v in g["m"]]
    assert int(d.view(np.uint16)[0, 0]) == int(g["d_bits"][0], 16) and int(dmin.view(np.uint16)[0, 0]) == int(g["dmin_bits"][0], 16)
    assert oracle.kq_pack(q, sc, mn, d, dmin, 4, 2).tolist() == [int(v, 16) for v in g["record"]]
    assert oracle.kq_record_bytes(4, 2) == 11 and oracle.kq_record_bytes() == 144
    What = oracle.kq_dequantize_rows(q, sc, mn, d, dmin, np.arange(8), 4, 2).ravel()
    assert What.tolist() == [float(v) for v in g["dequantized"]]
    y, bound = oracle.kq_gemv(q, sc, mn, d, dmin, np.array([2.0], np.float16), sub=4, nsub=2)
    assert y.tolist() == [2 * float(v) for v in g["dequantized"]] and bound.tolist() == [2 * abs(float(v)) for v in g["dequantized"]]


@pytest.mark.parametrize("bits,name", [(2, "kq_superblock_2bit.txt"), (5, "kq_superblock_5bit.txt"),
                                       (6, "kq_superblock_6bit.txt"), (8, "kq_superblock_8bit.txt")])
def test_kq_hand_worked_superblock_other_widths(bits, name):
    g = _golden_kq(name)
    W = np.array([float(v) for v in g["w"]], dtype=np.float16).reshape(8, 1)
    q, sc, mn, d, dmin = oracle.kq_quantize(W, 4, 2, bits)
    assert q.ravel().tolist() == [int(v) for v in g["q"]]
    assert sc.ravel().tolist() == [int(v) for v in g["sc"]] and mn.ravel().tolist() == [int(v) for v in g["m"]]
    assert int(d.view(np.uint16)[0, 0]) == int(g["d_bits"][0], 16) and int(dmin.view(np.uint16)[0, 0]) == int(g["dmin_bits"][0], 16)
    assert oracle.kq_pack(q, sc, mn, d, dmin, 4, 2, bits).tolist() == [int(v, 16) for v in g["record"]]
    assert oracle.kq_record_bytes(4, 2, bits) == len(g["record"])
    assert [oracle.kq_record_bytes(bits=b) for b in (2, 5, 6, 8)] == [80, 176, 208, 272]
    What = oracle.kq_dequantize_rows(q, sc, mn, d, dmin, np.arange(8), 4, 2).ravel()
    assert What.tolist() == [float(v) for v in g["dequantized"]]


@pytest.mark.parametrize("bits", [4, 2, 5, 6, 8])
def test_kq_quantizer_against_a_scalar_restatement(bits):
    f32 = np.float32
    top = (1 << bits) - 1
    rng = np.random.default_rng(21)
    sub, nsub, n = 4, 3, 7
    W = (rng.standard_normal((2 * sub * nsub, n)) * 0.3).astype(np.float16)
    W[:sub, 0] = np.float16(0.25)                  # a constant positive block: minimum field 0
    W[:, 1] = np.float16(0.0)                      # an all-zero superblock column (both superblocks)
    W[sub:2 * sub, 2] = -np.abs(W[sub:2 * sub, 2])  # an all-negative block
    q, sc, mn, d, dmin = oracle.kq_quantize(W, sub, nsub, bits)
    G = sub * nsub
    for r in range(2):
        for k in range(n):
            blocks = [W[r * G + i * sub: r * G + (i + 1) * sub, k].astype(f32) for i in range(nsub)]
            lo = [min(f32(b.min()), f32(0)) for b in blocks]
            step = [f32(f32(b.max()) - l) / f32(top) for b, l in zip(blocks, lo)]
            neg = [f32(-l) for l in lo]
            dd = np.float16(f32(max(step)) / f32(63))
            dm = np.float16(f32(max(neg)) / f32(63))
            assert d[r, k] == dd and dmin[r, k] == dm
            for i in range(nsub):
                s_i = int(min(np.rint(step[i] / f32(dd)), 63)) if f32(dd) != 0 else 0
                m_i = int(min(np.rint(neg[i] / f32(dm)), 63)) if f32(dm) != 0 else 0
                assert sc[r, i, k] == s_i and mn[r, i, k] == m_i
                se, oe = f32(dd) * f32(s_i), f32(dm) * f32(m_i)
                for j in range(sub):
                    want = int(np.clip(np.rint(f32(blocks[i][j] + oe) / se), 0, top)) if se != 0 else 0
                    assert q[r * G + i * sub + j, k] == want
    assert not q[:, 1].any() and not sc[:, :, 1].any() and float(d[0, 1]) == 0.0
    assert mn[0, 0, 0] == 0 and mn[0, 1, 2] > 0


@pytest.mark.parametrize("bits", [2, 5, 6, 8])
def test_kq_error_bound_and_code_layout_other_widths(bits):
    rng = np.random.default_rng(24)
    m, n, top = 512, 24, (1 << bits) - 1
    W = (rng.standard_normal((m, n)) * 0.02).astype(np.float16)
    q, sc, mn, d, dmin = oracle.kq_quantize(W, bits=bits)
    assert q.max() == top and sc.max() == 63 and mn.max() == 63
    What = oracle.kq_dequantize_rows(q, sc, mn, d, dmin, np.arange(m))
    w = W.astype(np.float64).reshape(2, 8, 32, n)
    lo = np.minimum(w.min(axis=2), 0.0)
    s_eff = d.astype(np.float64)[:, None, :] * sc
    o_eff = dmin.astype(np.float64)[:, None, :] * mn
    lim = s_eff / 2 + np.abs(w.max(axis=2) - lo - top * s_eff) + np.abs(o_eff + lo) + 1e-7
    err = np.abs(What.reshape(2, 8, 32, n) - w)
    assert np.all(err <= lim[:, :, None, :])
    # finer codes, smaller error: 8-bit steps are 17 times finer than 4-bit ones, 2-bit steps 5 times coarser
    q4, sc4, mn4, d4, dmin4 = oracle.kq_quantize(W)
    err4 = np.abs(oracle.kq_dequantize_rows(q4, sc4, mn4, d4, dmin4, np.arange(m)) - W.astype(np.float64))
    ratio = np.mean(err) / np.mean(err4)
    # mean error against the 4-bit format's: about 15 / (2^bits - 1)
    assert {2: 3.0, 5: 0.35, 6: 0.17, 8: 0.03}[bits] < ratio < {2: 7.0, 5: 0.65, 6: 0.35, 8: 0.25}[bits]
    # the record: codes (2 bits: four quarter-planes per byte; 8 bits: one per byte), fields, d, dmin
    nc = 256 * bits // 8
    rec = oracle.kq_pack(q, sc, mn, d, dmin, bits=bits).reshape(2, n, nc + 16)
    for (r, k) in [(0, 0), (1, 11), (1, 23)]:
        b = rec[r, k]
        col = q[r * 256:(r + 1) * 256, k].astype(int)
        quarters = lambda v, i: v[i] | (v[64 + i] << 2) | (v[128 + i] << 4) | (v[192 + i] << 6)
        for i in range(nc):
            if bits == 8:
                assert b[i] == col[i]
            elif bits == 2:
                assert b[i] == quarters(col, i)
            elif i < 128:                               # 5 and 6 bits: the low four bits like 4-bit codes
                assert b[i] == ((col[i] & 15) | ((col[128 + i] & 15) << 4))
            elif bits == 5:                             # then one high bit per row
                assert b[i] == sum(((col[8 * (i - 128) + e] >> 4) & 1) << e for e in range(8))
            else:                                       # or two, arranged like 2-bit codes
                assert b[i] == quarters(col >> 4, i - 128)
        fb = int.from_bytes(bytes(b[nc:nc + 12].tolist()), "little")
        assert [(fb >> (6 * f)) & 63 for f in range(16)] == sc[r, :, k].tolist() + mn[r, :, k].tolist()
        assert int.from_bytes(bytes(b[nc + 12:nc + 14].tolist()), "little") == int(d.view(np.uint16)[r, k])
        assert int.from_bytes(bytes(b[nc + 14:nc + 16].tolist()), "little") == int(dmin.view(np.uint16)[r, k])


def test_kq_error_bound_scaling_and_fields():
    rng = np.random.default_rng(22)
    m, n = 512, 40
    W = (rng.standard_normal((m, n)) * 0.02).astype(np.float16)
    q, sc, mn, d, dmin = oracle.kq_quantize(W)
    assert q.max() <= 15 and sc.max() <= 63 and mn.max() <= 63 and sc.max() == 63 and mn.max() == 63
    What = oracle.kq_dequantize_rows(q, sc, mn, d, dmin, np.arange(m))
    w = W.astype(np.float64).reshape(2, 8, 32, n)
    lo = np.minimum(w.min(axis=2), 0.0)
    rng_i = w.max(axis=2) - lo
    s_eff = d.astype(np.float64)[:, None, :] * sc
    o_eff = dmin.astype(np.float64)[:, None, :] * mn
    # half a step, plus what the 6-bit rounding of the step and of the minimum can add at the ends of the range
    lim = s_eff / 2 + np.abs(rng_i - 15 * s_eff) + np.abs(o_eff + lo) + 1e-7
    err = np.abs(What.reshape(2, 8, 32, n) - w)
    assert np.all(err <= lim[:, :, None, :])
    assert np.median(err / np.maximum(s_eff[:, :, None, :], 1e-12)) < 0.3
    # scaling W by a power of two scales d and dmin and leaves every integer field alone
    q2, sc2, mn2, d2, dmin2 = oracle.kq_quantize((W.astype(np.float32) * 4).astype(np.float16))
    assert np.array_equal(q, q2) and np.array_equal(sc, sc2) and np.array_equal(mn, mn2)
    assert np.array_equal(d2.astype(np.float32), d.astype(np.float32) * 4) and np.array_equal(dmin2.astype(np.float32), dmin.astype(np.float32) * 4)
    # the record: codes, then the sixteen 6-bit fields as a little-endian bit string, then d and dmin
    rec = oracle.kq_pack(q, sc, mn, d, dmin).reshape(2, n, 144)
    for (r, k) in [(0, 0), (1, 17), (1, 39)]:
        b = rec[r, k]
        for i in range(128):
            assert b[i] == (q[r * 256 + i, k] | (q[r * 256 + 128 + i, k] << 4))
        bits = int.from_bytes(bytes(b[128:140].tolist()), "little")
        assert [(bits >> (6 * f)) & 63 for f in range(16)] == sc[r, :, k].tolist() + mn[r, :, k].tolist()
        assert int.from_bytes(bytes(b[140:142].tolist()), "little") == int(d.view(np.uint16)[r, k])
        assert int.from_bytes(bytes(b[142:144].tolist()), "little") == int(dmin.view(np.uint16)[r, k])


def test_kq_product_in_exact_rationals_and_over_a_list():
    from fractions import Fraction
    rng = np.random.default_rng(23)
    sub, nsub, n = 4, 2, 9
    W = (rng.standard_normal((16, n)) * 0.2).astype(np.float16)
    x = (rng.standard_normal(n)).astype(np.float16)
    q, sc, mn, d, dmin = oracle.kq_quantize(W, sub, nsub)
    idx = np.array([7, 0, 3], dtype=np.int32)
    y, bound = oracle.kq_gemv(q, sc, mn, d, dmin, x, idx, sub=sub, nsub=nsub)
    yd, _ = oracle.kq_gemv(q, sc, mn, d, dmin, x, sub=sub, nsub=nsub)
    for j in range(16):
        r, i = j // 8, (j % 8) // sub
        def wh(k):
            return Fraction(float(d[r, k])) * int(sc[r, i, k]) * int(q[j, k]) - Fraction(float(dmin[r, k])) * int(mn[r, i, k])
        acc = sum((wh(int(k)) * Fraction(float(x[k])) for k in idx), Fraction(0))
        accd = sum((wh(k) * Fraction(float(x[k])) for k in range(n)), Fraction(0))
        ab = sum((abs(wh(int(k))) * abs(Fraction(float(x[k]))) for k in idx), Fraction(0))
        assert abs(float(acc) - y[j]) <= 1e-12 and abs(float(accd) - yd[j]) <= 1e-12 and abs(float(ab) - bound[j]) <= 1e-12
