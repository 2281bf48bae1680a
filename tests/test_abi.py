"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, sizes are right, and bad arguments are refused before
anything is launched."""
import ctypes
import os
import re

import pytest

from conftest import ROOT
from paper_2511_04477_b200 import binding, build


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spqt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spqt_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert "spqt_pack" in names and "spqt_sparsify" in names and "spqt_sparse_gemv" in names
    for name in names:
        assert hasattr(L, name), name
    assert set(names) == set(binding.EXPORTS)


def test_status_strings(L):
    assert binding.status_string(0) == "SPQT_OK"
    assert binding.status_string(2) == "SPQT_ERR_UNSUPPORTED"
    assert binding.status_string(6) == "SPQT_ERR_TIMEOUT"
    assert binding.status_string(99) == "SPQT_ERR_UNKNOWN"
    assert L.spqt_version() >= 2000


@pytest.mark.parametrize("m,n,bits,group,B", [(4096, 4096, 4, 128, 64), (14336, 4096, 4, 64, 32),
                                              (8192, 28672, 3, 128, 48), (128, 1, 3, 64, 24)])
def test_packed_sizes(L, m, n, bits, group, B):
    s = binding.spqt_packed_sizes(m, n, bits, group)
    R = m // group
    assert s.codes_bytes == R * n * B
    assert s.scale_zero_bytes == R * n * 4
    assert s.gemv_workspace_bytes >= R * 4 + 4 * (m + R)      # counters + one worker's partials
    assert s.gemv_workspace_bytes < 64 << 20


def test_unsupported_formats_are_refused(L):
    for args in [(4096, 4096, 5, 128), (4096, 4096, 4, 32), (4000, 4096, 4, 128), (4096, 4096, 2, 64)]:
        with pytest.raises(binding.SpqtError) as e:
            binding.spqt_packed_sizes(*args)
        assert e.value.status == 2
    with pytest.raises(binding.SpqtError) as e:
        binding.spqt_packed_sizes(0, 4096, 4, 128)
    assert e.value.status == 1


def test_bad_arguments_launch_nothing(L):
    before = binding.spqt_launch_count()
    buf = ctypes.create_string_buffer(4096)
    base = ctypes.addressof(buf)
    a16 = (base + 15) // 16 * 16            # 16-byte aligned fake "device" address; never dereferenced
    ws = binding.spqt_packed_sizes(128, 8, 4, 128).gemv_workspace_bytes
    # null pointers
    assert L.spqt_pack(None, 128, 8, 8, 4, 128, a16, a16, None) == 1
    assert L.spqt_sparsify(None, 8, 0.5, a16, a16, None) == 1
    assert L.spqt_sparse_gemv(a16, a16, 128, 8, 4, 128, a16, None, a16, a16, a16, ws, None) == 1
    assert L.spqt_dense_gemv(a16, None, 128, 8, 4, 128, a16, a16, a16, ws, None) == 1
    assert L.spqt_sparsify_gemv(a16, a16, 128, 8, 4, 128, a16, 0.5, a16, None, a16, a16, ws, None) == 1
    # ldw < n, negative n
    assert L.spqt_pack(a16, 128, 8, 4, 4, 128, a16, a16, None) == 1
    assert L.spqt_sparsify(a16, -1, 0.5, a16, a16, None) == 1
    # unsupported format; more columns than the 16-bit column numbers of the list reach
    assert L.spqt_pack(a16, 100, 8, 8, 4, 128, a16, a16, None) == 2
    assert L.spqt_sparse_gemv(a16, a16, 128, 8, 8, 128, a16, a16, a16, a16, a16, ws, None) == 2
    big = binding.spqt_packed_sizes(128, 70000, 4, 128).gemv_workspace_bytes
    assert L.spqt_sparse_gemv(a16, a16, 128, 70000, 4, 128, a16, a16, a16, a16, a16, big, None) == 2
    # misaligned
    assert L.spqt_pack(a16, 128, 8, 8, 4, 128, a16 + 4, a16, None) == 3
    assert L.spqt_sparse_gemv(a16 + 8, a16, 128, 8, 4, 128, a16, a16, a16, a16, a16, ws, None) == 3
    assert L.spqt_sparse_gemv(a16, a16, 128, 8, 4, 128, a16 + 1, a16, a16, a16, a16, ws, None) == 3
    assert L.spqt_sparsify(a16 + 1, 8, 0.5, a16, a16, None) == 3
    # workspace too small
    assert L.spqt_sparse_gemv(a16, a16, 128, 8, 4, 128, a16, a16, a16, a16, a16, ws - 1, None) == 4
    assert L.spqt_dense_gemv(a16, a16, 128, 8, 4, 128, a16, a16, a16, 16, None) == 4
    assert L.spqt_autotune(a16, a16, 128, 8, 4, 128, None, 0.5, a16, a16, a16, a16, ws, None, 0, None, None, None) == 1
    assert L.spqt_autotune(a16, a16, 128, 8, 4, 128, a16, 0.5, a16, a16, a16, a16, ws - 1, None, 0, None, None, None) == 4
    assert L.spqt_calibrate_threshold(None, 8, 0.5, a16, a16, 131072, None) == 1
    assert L.spqt_calibrate_threshold(a16, 8, 1.5, a16, a16, 131072, None) == 1
    assert L.spqt_calibrate_threshold(a16, 8, 0.5, a16, a16, 131071, None) == 4
    sws = ctypes.c_size_t(0)
    assert L.spqt_gemm_small_workspace(128, 8, 4, 128, ctypes.byref(sws)) == 0 and sws.value >= 8 * 4 * 129 * 4
    assert L.spqt_gemm_small_workspace(100, 8, 4, 128, ctypes.byref(sws)) == 2
    assert L.spqt_sparse_gemm_small(a16, a16, 128, 8, 4, 128, a16, 8, 9, 0.5, a16, a16, a16, 128, a16, sws.value, None) == 1   # batch > 8
    assert L.spqt_sparse_gemm_small(a16, a16, 128, 8, 4, 128, a16, 4, 2, 0.5, a16, a16, a16, 128, a16, sws.value, None) == 1   # ldx < n
    assert L.spqt_dense_gemm_small(a16, a16, 128, 8, 4, 128, a16, 8, 2, a16, 128, a16, sws.value - 1, None) == 4
    assert L.spqt_set_tuning(-1, 0) == 1
    assert L.spqt_set_tuning(0, 8) == 1
    assert L.spqt_workspace_status(None, 128, 128, None, None) == 1
    assert L.spqt_static_status(100, 128, None, None) == 1
    assert binding.spqt_launch_count() == before


def test_sizes_and_refusals_of_the_rowwise_and_two_level_entries(L):
    assert binding.spqt_rowwise_packed_sizes(4096, 4096, 4, 128) == (4096 * 4096 // 2, 4096 * 32 * 4)
    assert binding.spqt_rowwise_packed_sizes(3, 64, 4, 64) == (96, 12)
    sz = ctypes.c_size_t(0)
    assert L.spqt_rowwise_packed_sizes(8, 100, 4, 128, ctypes.byref(sz), None) == 2      # n not a multiple of the group
    assert L.spqt_rowwise_packed_sizes(8, 128, 3, 128, ctypes.byref(sz), None) == 2      # 4-bit only
    assert L.spqt_rowwise_packed_sizes(0, 128, 4, 128, ctypes.byref(sz), None) == 1
    rec, ws = binding.spqt_kq_packed_sizes(14336, 4096)
    assert rec == (14336 // 256) * 4096 * 144 and ws >= 56 * 4 and ws % 16 == 0
    assert L.spqt_kq_packed_sizes(128, 8, ctypes.byref(sz), None) == 2                   # m not a multiple of 256
    assert L.spqt_kq_packed_sizes(256, 0, ctypes.byref(sz), None) == 1
    # null pointers are refused before any launch (no GPU needed to say so)
    assert L.spqt_rowwise_pack(None, 8, 128, 128, 4, 128, None, None, None) == 1
    assert L.spqt_rowwise_dense_gemv(None, None, 8, 128, 4, 128, None, None, None) == 1
    assert L.spqt_kq_pack(None, 256, 8, 8, None, None) == 1
    assert L.spqt_kq_dense_gemv(None, 256, 8, None, None, None, 0, None) == 1
    assert L.spqt_kq_sparse_gemv(None, 256, 8, None, None, None, None, None, 0, None) == 1
    # other code widths of the same format: sizes per width, unsupported widths, null pointers
    assert binding.spqt_kqw_packed_sizes(14336, 4096, 4) == (rec, ws)
    assert binding.spqt_kqw_packed_sizes(14336, 4096, 2)[0] == 56 * 4096 * 80
    assert binding.spqt_kqw_packed_sizes(14336, 4096, 8) == (56 * 4096 * 272, ws)
    assert binding.spqt_kqw_packed_sizes(14336, 4096, 5)[0] == 56 * 4096 * 176
    assert binding.spqt_kqw_packed_sizes(14336, 4096, 6)[0] == 56 * 4096 * 208
    assert L.spqt_kqw_packed_sizes(256, 8, 3, ctypes.byref(sz), None) == 2
    assert L.spqt_kqw_pack(None, 256, 8, 8, 8, None, None) == 1
    assert L.spqt_kqw_dense_gemv(None, 256, 8, 2, None, None, None, 0, None) == 1
    assert L.spqt_kqw_sparse_gemv(None, 256, 8, 8, None, None, None, None, None, 0, None) == 1


def test_host_step_refuses_bad_arguments_without_touching_the_device(L):
    handle = ctypes.c_void_p(None)
    assert L.spqt_host_step_create(None, 1, ctypes.byref(handle)) == 1
    assert L.spqt_host_step_create(ctypes.c_void_p(16), 0, ctypes.byref(handle)) == 1
    assert L.spqt_host_step_create(ctypes.c_void_p(16), 1, None) == 1
    assert L.spqt_host_step_launch(None, None) == 1
    assert L.spqt_host_step_destroy(None) == 1
