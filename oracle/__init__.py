"""SpQt CPU oracle (ctypes front end of ``spqt_oracle.c``) -- TEST INFRASTRUCTURE.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` /
``--impl reference`` legs of ``bench.py`` may import this package.  It shares
nothing with the CUDA library: the layout and the quantizer are restated in
``spqt_oracle.c`` from the paper (Sec. 2, Sec. 4.1.2, Sec. 4.2.3), not included
from it.  Arrays are numpy; fp16 values travel as ``numpy.float16``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import math

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spqt_oracle.c")
_LIB = os.path.join(_HERE, "libspqt_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp contraction off, so every quantizer step
    is one IEEE fp32 operation).  Returns the path of the shared object."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".%d.tmp" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.spqt_oracle_block_bytes.restype = ctypes.c_size_t
            lib.spqt_oracle_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _check(rc, what):
    if rc != 0:
        raise ValueError("oracle %s rejected its arguments (code %d)" % (what, rc))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16, a.dtype
    return a.view(np.uint16)


def block_bytes(bits: int, group: int) -> int:
    return int(_load().spqt_oracle_block_bytes(int(bits), int(group)))


def half_to_float(h_bits: np.ndarray) -> np.ndarray:
    h = np.ascontiguousarray(h_bits, dtype=np.uint16)
    out = np.empty(h.shape, np.float32)
    _load().spqt_oracle_half_to_float(_p(h), _p(out), ctypes.c_size_t(h.size))
    return out


def float_to_half(f: np.ndarray) -> np.ndarray:
    f = np.ascontiguousarray(f, dtype=np.float32)
    out = np.empty(f.shape, np.uint16)
    _load().spqt_oracle_float_to_half(_p(f), _p(out), ctypes.c_size_t(f.size))
    return out


def quantize(W: np.ndarray, bits: int = 4, group: int = 128):
    """fp16 W[m][n] -> (q uint8[m][n] natural order, scales fp16[R][n], zeros fp16[R][n])."""
    Wb = _u16(W)
    m, n = Wb.shape
    R = m // group if group else 0
    q = np.empty((m, n), np.uint8)
    s = np.empty((max(R, 0), n), np.uint16)
    z = np.empty((max(R, 0), n), np.uint16)
    _check(_load().spqt_oracle_quantize(_p(Wb), m, n, n, bits, group, _p(q), _p(s), _p(z)), "quantize")
    return q, s.view(np.float16), z.view(np.float16)


def pack_codes(q: np.ndarray, bits: int = 4, group: int = 128) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    m, n = q.shape
    codes = np.empty((m // group) * n * block_bytes(bits, group), np.uint8)
    _check(_load().spqt_oracle_pack_codes(_p(q), m, n, bits, group, _p(codes)), "pack_codes")
    return codes


def unpack_codes(codes: np.ndarray, m: int, n: int, bits: int = 4, group: int = 128) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    assert codes.size == (m // group) * n * block_bytes(bits, group)
    q = np.empty((m, n), np.uint8)
    _check(_load().spqt_oracle_unpack_codes(_p(codes), m, n, bits, group, _p(q)), "unpack_codes")
    return q


def pack(W: np.ndarray, bits: int = 4, group: int = 128):
    """fp16 W[m][n] -> (codes uint8[R*n*B] zigzag, scales fp16[R][n], zeros fp16[R][n])."""
    q, s, z = quantize(W, bits, group)
    return pack_codes(q, bits, group), s, z


def dequantize(codes, scales, zeros, m, n, bits=4, group=128) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty((m, n), np.float64)
    _check(_load().spqt_oracle_dequantize(_p(codes), _p(_u16(scales)), _p(_u16(zeros)),
                                          m, n, bits, group, _p(out)), "dequantize")
    return out


def sparsify(x: np.ndarray, t: float):
    """fp16 x[n], threshold t -> (idx int32[count] ascending, count)."""
    xb = _u16(x)
    n = xb.size
    idx = np.empty(max(n, 1), np.int32)
    cnt = np.zeros(1, np.int32)
    _check(_load().spqt_oracle_sparsify(_p(xb), n, ctypes.c_float(t), _p(idx), _p(cnt)), "sparsify")
    c = int(cnt[0])
    return idx[:c].copy(), c


def _rows_arg(rows, m):
    if rows is None:
        return None, 0, m
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    return rows, rows.size, rows.size


def sparse_gemv(codes, scales, zeros, m, n, x, idx, bits=4, group=128, rows=None):
    """-> (y float64[rows], bound float64[rows]); bound = sum |What||x| over the listed columns."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    rows_a, n_rows, out_n = _rows_arg(rows, m)
    y = np.empty(out_n, np.float64)
    b = np.empty(out_n, np.float64)
    rc = _load().spqt_oracle_sparse_gemv(
        _p(codes), _p(_u16(scales)), _p(_u16(zeros)), m, n, bits, group, _p(_u16(x)),
        _p(idx), int(idx.size), _p(rows_a) if rows_a is not None else None, n_rows, _p(y), _p(b))
    _check(rc, "sparse_gemv")
    return y, b


def dense_gemv(codes, scales, zeros, m, n, x, bits=4, group=128, rows=None):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rows_a, n_rows, out_n = _rows_arg(rows, m)
    y = np.empty(out_n, np.float64)
    b = np.empty(out_n, np.float64)
    rc = _load().spqt_oracle_dense_gemv(
        _p(codes), _p(_u16(scales)), _p(_u16(zeros)), m, n, bits, group, _p(_u16(x)),
        _p(rows_a) if rows_a is not None else None, n_rows, _p(y), _p(b))
    _check(rc, "dense_gemv")
    return y, b


def partition(count: int, S: int) -> np.ndarray:
    out = np.empty(S + 1, np.int32)
    _check(_load().spqt_oracle_partition(int(count), int(S), _p(out)), "partition")
    return out


def threads() -> int:
    return int(_load().spqt_oracle_threads())


def set_threads(t: int) -> None:
    _load().spqt_oracle_set_threads(int(t))


def calibrate_threshold(pool, sparsity: float) -> float:
    """Nearest-rank threshold of |x| over a pool of fp16 calibration activations (calibration threshold tool,
    Sec. 5): the ceil(sparsity * N)-th smallest magnitude, N = the entries that are not NaN; -1 when nothing
    is to be dropped.  Written out with a full sort."""
    a = np.abs(np.asarray(pool, dtype=np.float16).ravel().astype(np.float64))
    a = np.sort(a[~np.isnan(a)])
    if a.size == 0 or not (sparsity > 0.0):
        return -1.0
    rank = int(min(a.size, max(1, math.ceil(sparsity * a.size - 1e-9))))
    return float(a[rank - 1])


def group_sparsity(levels) -> float:
    """Sparsity shared by the matrices that read one input: the mean of their levels (customized mode, Sec. 5)."""
    levels = [float(v) for v in levels]
    return sum(levels) / len(levels)


def union_sparsify(X, t: float):
    """Small batch (several decode rows at once, Sec. 3.2 / Sec. 4.1.3 on beams): the columns that are active
    in at least one row, k with |X[b][k]| > t for some b, ascending, and their number."""
    X = np.ascontiguousarray(X, dtype=np.float16)
    active = set()
    for b in range(X.shape[0]):
        idx, cnt = sparsify(X[b], t)
        active.update(int(k) for k in idx[:cnt])
    out = np.array(sorted(active), dtype=np.int32)
    return out, int(out.size)


def sparse_gemm_small(codes, scales, zeros, m, n, X, idx, bits=4, group=128, rows=None):
    """Y[b][j] = sum over the union list of What[j][k] * X[b][k]: every row of the batch is multiplied over
    the same columns (the union of the rows' active sets), each with its own values -- also those at or
    below the threshold in that row: the block is read for the batch anyway.  Returns (Y, bound), both
    float64 [B][rows]; bound[b][j] = sum |What[j][k]| |X[b][k]| over the list."""
    X = np.ascontiguousarray(X, dtype=np.float16)
    ys, bs = [], []
    for b in range(X.shape[0]):
        y, bound = sparse_gemv(codes, scales, zeros, m, n, X[b], idx, bits, group, rows=rows)
        ys.append(y)
        bs.append(bound)
    return np.stack(ys), np.stack(bs)


def rowwise_quantize(W, bits: int = 4, group: int = 128):
    """The conventional layout the paper contrasts the zigzag layout with (Sec. 2, Sec. 4.1.1): a quantization
    group is `group` consecutive COLUMNS of one row.  Same quantizer as `quantize` (min/max, round to nearest),
    applied along the other axis: the groups of W along its rows are the groups of W^T down its columns.
    fp16 W[m][n] -> (q uint8[m][n], scales fp16[m][n/group], zeros fp16[m][n/group])."""
    Wt = np.ascontiguousarray(np.asarray(W, dtype=np.float16).T)
    q, s, z = quantize(Wt, bits, group)
    return np.ascontiguousarray(q.T), np.ascontiguousarray(s.T), np.ascontiguousarray(z.T)


def rowwise_pack_codes(q, bits: int = 4, group: int = 128) -> np.ndarray:
    """Row-wise block order: block (j, g) = the codes of columns g*group .. g*group+group-1 of row j, stored at
    block index j*(n/group) + g; inside a block the bytes follow the same rule as a zigzag block."""
    q = np.ascontiguousarray(q, dtype=np.uint8)
    m, n = q.shape
    B = block_bytes(bits, group)
    by_group_then_row = pack_codes(np.ascontiguousarray(q.T), bits, group).reshape(n // group, m, B)
    return np.ascontiguousarray(by_group_then_row.transpose(1, 0, 2)).reshape(-1)


def rowwise_dense_gemv(q, scales, zeros, x, group: int = 128):
    """y[j] = sum_k (scale[j][k/group] * q[j][k] + zero[j][k/group]) * x[k] in float64, and
    bound[j] = sum_k |What[j][k]| |x[k]|."""
    s = np.repeat(np.asarray(scales, dtype=np.float16).astype(np.float64), group, axis=1)
    z = np.repeat(np.asarray(zeros, dtype=np.float16).astype(np.float64), group, axis=1)
    What = s * np.asarray(q, dtype=np.float64) + z
    xv = np.asarray(x, dtype=np.float16).astype(np.float64)
    return What @ xv, np.abs(What) @ np.abs(xv)


def rowwise_thresholded_gemv(q, scales, zeros, x, t: float, group: int = 128):
    """The row-wise product over the active entries only: |x[k]| > t (NaN never active); the others count as zero."""
    xv = np.asarray(x, dtype=np.float16).astype(np.float64)
    with np.errstate(invalid="ignore"):
        active = np.abs(xv) > float(t)
    return rowwise_dense_gemv(q, scales, zeros, np.where(active, xv, 0.0).astype(np.float16), group)


# ---------------------------------------------------------------- two-level ("K-quant"-style) format
#
# The format the paper's implementation builds on (Sec. 2): superblocks of 256 weights split into eight
# blocks of 32, 4-bit codes, a 6-bit scale and a 6-bit minimum per block, a 16-bit scale and a 16-bit
# minimum per superblock; here in the zigzag arrangement (a superblock = 256 consecutive ROWS of one
# column, superblocks stored row-major over (block-row, column), Sec. 4.1.2).  The paper fixes neither the
# rounding rule nor the bit arrangement inside a superblock; the reading taken (both sides implement it):
#   per block i of a superblock:  lo_i = min(min_j w_j, 0),  range_i = max_j w_j - lo_i,
#                                 step_i = range_i / 15,      neg_i = 0 - lo_i                   (fp32;
#                                 zeros of either sign count as +0.0)
#   per superblock:               d = fp16(max_i step_i / 63),  dmin = fp16(max_i neg_i / 63)
#                                 sc_i = min(rint(step_i / d), 63),  m_i = min(rint(neg_i / dmin), 63)
#   weight:                       q_j = clamp(rint((w_j + dmin*m_i) / (d*sc_i)), 0, 15)   (0 if d*sc_i == 0)
#   dequantized:                  What_j = d*sc_i*q_j - dmin*m_i
# every operation a single IEEE fp32 operation (rint = round to nearest even), so that another
# implementation of the same steps produces the same bytes.
# Record of a superblock (G = sub*nsub weights): G/2 bytes of codes (byte i = q_i | q_{i+G/2} << 4), then the
# 2*nsub six-bit fields sc_0.., m_0.. as a little-endian bit string (field f at bits 6f..6f+5) padded to whole
# bytes, then d and dmin as little-endian fp16: 128 + 12 + 4 = 144 bytes for sub = 32, nsub = 8.
# Other code widths (Sec. 4.1.3: any width from 2 to 8 bits): bits = 2, 5, 6 or 8 puts 2^bits - 1 in the place
# of 15 and changes the code bytes only -- 8 bits: byte i = q_i (G bytes); 2 bits: byte i = q_i | q_{i+G/4} << 2 |
# q_{i+G/2} << 4 | q_{i+3G/4} << 6 (G/4 bytes); 5 and 6 bits: the low four bits of every code as for 4 bits, then
# the high bits q >> 4, one per row (bit j%8 of byte j/8) or two per row arranged like 2-bit codes; records of
# 80, 176, 208 and 272 bytes.  Pinned by hand-worked superblocks (tests/golden/kq_superblock_2bit.txt, _5bit,
# _6bit, _8bit), the scalar restatement, the error bound and the layout check.

def kq_record_bytes(sub: int = 32, nsub: int = 8, bits: int = 4) -> int:
    return sub * nsub * bits // 8 + (12 * nsub + 7) // 8 + 4


def kq_quantize(W, sub: int = 32, nsub: int = 8, bits: int = 4):
    """fp16 W[m][n] -> (q uint8[m][n], sc uint8[R][nsub][n], mn uint8[R][nsub][n], d fp16[R][n], dmin fp16[R][n]).
    bits = width of a code (2, 4, 5, 6 or 8): the codes run from 0 to 2^bits - 1, everything else is the same rule."""
    assert bits in (2, 4, 5, 6, 8)
    top = np.float32((1 << bits) - 1)
    W = np.ascontiguousarray(W, dtype=np.float16)
    m, n = W.shape
    G = sub * nsub
    assert m % G == 0
    R = m // G
    f32 = np.float32
    w = W.astype(f32).reshape(R, nsub, sub, n)
    with np.errstate(divide="ignore", invalid="ignore"):
        lo = np.minimum(w.min(axis=2), f32(0)) + f32(0)            # (a zero of either sign counts as +0.0)
        hi = w.max(axis=2) + f32(0)
        step = ((hi - lo).astype(f32) / top).astype(f32)
        neg = (f32(0) - lo).astype(f32)                            # (0 - 0 is +0.0)
        d = (step.max(axis=1) / f32(63)).astype(f32).astype(np.float16)
        dmin = (neg.max(axis=1) / f32(63)).astype(f32).astype(np.float16)
        df, dminf = d.astype(f32)[:, None, :], dmin.astype(f32)[:, None, :]
        sc = np.where(df != 0, np.minimum(np.rint((step / df).astype(f32)), f32(63)), f32(0)).astype(np.uint8)
        mn = np.where(dminf != 0, np.minimum(np.rint((neg / dminf).astype(f32)), f32(63)), f32(0)).astype(np.uint8)
        s_eff = (df * sc.astype(f32)).astype(f32)[:, :, None, :]
        o_eff = (dminf * mn.astype(f32)).astype(f32)[:, :, None, :]
        quo = ((w + o_eff).astype(f32) / s_eff).astype(f32)
        q = np.where(s_eff != 0, np.clip(np.rint(quo), f32(0), top), f32(0)).astype(np.uint8)
    return q.reshape(m, n), sc, mn, d, dmin


def kq_pack(q, sc, mn, d, dmin, sub: int = 32, nsub: int = 8, bits: int = 4) -> np.ndarray:
    """The records, uint8[R][n][record bytes] flattened (superblock (r, k) at record index r*n + k).  Codes of a
    superblock's G rows: 4 bits, byte i = q_i | q_{i+G/2} << 4; 8 bits, byte i = q_i; 2 bits, byte i =
    q_i | q_{i+G/4} << 2 | q_{i+G/2} << 4 | q_{i+3G/4} << 6; 5 and 6 bits, the low four bits of every code as
    for 4 bits (G/2 bytes), then the high bits h = q >> 4: one bit per row, bit j%8 of byte j/8 (5 bits), or
    two bits per row arranged like 2-bit codes (6 bits)."""
    assert bits in (2, 4, 5, 6, 8)
    G = sub * nsub
    m, n = q.shape
    R = m // G
    nf = (12 * nsub + 7) // 8
    nc = G * bits // 8
    rec = np.zeros((R, n, kq_record_bytes(sub, nsub, bits)), np.uint8)
    qb = q.reshape(R, G, n)
    def plane(v, width):                              # G values of `width` bits -> G*width/8 bytes, 8/width per byte
        nb, per = G * width // 8, 8 // width
        out = np.zeros((R, nb, n), np.uint8)
        for f in range(per):
            out |= (v[:, f * nb:(f + 1) * nb, :] << (width * f)).astype(np.uint8)
        return out
    if bits in (2, 4, 8):
        codes = plane(qb, bits)
    else:
        h = qb >> 4
        if bits == 5:                                 # bit j % 8 of byte j / 8
            high = np.zeros((R, G // 8, n), np.uint8)
            for e in range(8):
                high |= (h[:, e::8, :] << e).astype(np.uint8)
        else:
            high = plane(h, 2)
        codes = np.concatenate([plane(qb & 15, 4), high], axis=1)
    rec[:, :, :nc] = codes.transpose(0, 2, 1)
    fields = np.concatenate([sc, mn], axis=1).astype(np.uint64)        # [R][2*nsub][n]
    fbits = np.zeros((R, n), dtype=object)
    for f in range(2 * nsub):
        fbits = fbits + (fields[:, f, :].astype(object) << (6 * f))
    for b in range(nf):
        rec[:, :, nc + b] = ((fbits >> (8 * b)) & 0xFF).astype(np.uint8)
    du, mu = np.asarray(d, np.float16).view(np.uint16), np.asarray(dmin, np.float16).view(np.uint16)
    o = nc + nf
    rec[:, :, o], rec[:, :, o + 1] = (du & 0xFF).astype(np.uint8), (du >> 8).astype(np.uint8)
    rec[:, :, o + 2], rec[:, :, o + 3] = (mu & 0xFF).astype(np.uint8), (mu >> 8).astype(np.uint8)
    return rec.reshape(-1)


def kq_dequantize_rows(q, sc, mn, d, dmin, rows, sub: int = 32, nsub: int = 8) -> np.ndarray:
    """What[rows][n] in float64: d*sc_i*q - dmin*m_i with i the block of the row inside its superblock."""
    G = sub * nsub
    rows = np.asarray(rows, dtype=np.int64)
    r, i = rows // G, (rows % G) // sub
    s = d.astype(np.float64)[r, :] * sc[r, i, :].astype(np.float64)
    o = dmin.astype(np.float64)[r, :] * mn[r, i, :].astype(np.float64)
    return s * q[rows, :].astype(np.float64) - o


def kq_gemv(q, sc, mn, d, dmin, x, idx=None, rows=None, sub: int = 32, nsub: int = 8):
    """y[j] = sum over idx (all columns if None) of What[j][k] * x[k], float64; and the bound sum |What||x|."""
    m, n = q.shape
    rows = np.arange(m) if rows is None else np.asarray(rows)
    What = kq_dequantize_rows(q, sc, mn, d, dmin, rows, sub, nsub)
    xv = np.asarray(x, dtype=np.float16).astype(np.float64)
    if idx is not None:
        idx = np.asarray(idx, dtype=np.int64)
        What, xv = What[:, idx], xv[idx]
    return What @ xv, np.abs(What) @ np.abs(xv)
