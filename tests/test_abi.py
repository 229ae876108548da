"""CPU-only checks of the boundary: the library loads, exports what the header declares,
answers size queries and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2512_05409_b200 as sq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert {"sq_pack_weights", "sq_encode", "sq_gemm", "sq_decode", "sq_calib_positions"} <= set(names)
    lib = ctypes.CDLL(sq.LIBRARY_PATH)
    for n in names:
        assert hasattr(lib, n), n
    # and the binding offers the same names
    for n in names:
        assert hasattr(sq, n), n


def test_size_queries():
    f = sq.make_format(64, 8, False)
    assert sq.sq_encoded_sizes(f, 64, 4096) == [64 * 2048, 64 * 64 * 8, 64 * 64 * 8, 256, 256, 64]
    assert sq.sq_weights_sizes(f, 4096, 4096) == [4096 * 2048, 4096 * 4, 4096 * 4, 0]
    fs = sq.make_format(128, 16, True)
    assert sq.sq_encoded_sizes(fs, 4096, 8192)[2] == 0
    assert sq.sq_weights_sizes(fs, 8192, 8192)[3] == 8192 * 64 * 16
    assert sq.sq_encoded_sizes(f, 0, 128) == [0, 0, 0, 0, 0, 0]
    # payload bytes per element: 0.5 + 2k/b dynamic, 0.5 + k/b static
    s = sq.sq_encoded_sizes(f, 1, 8192)
    assert (s[0] + s[1] + s[2]) / 8192 == 0.5 + 2 * 8 / 64
    s = sq.sq_encoded_sizes(sq.make_format(64, 8, True), 1, 8192)
    assert (s[0] + s[1] + s[2]) / 8192 == 0.5 + 8 / 64


@pytest.mark.parametrize("bank,k,ver,expect", [
    (48, 4, 1, sq.SQ_ERR_INVALID_ARG), (64, 0, 1, sq.SQ_ERR_INVALID_ARG),
    (64, 33, 1, sq.SQ_ERR_INVALID_ARG), (64, 8, 2, sq.SQ_ERR_INVALID_ARG),
])
def test_bad_formats_are_rejected(bank, k, ver, expect):
    f = sq.sq_format(bank, k, 0, ver)
    out = (ctypes.c_size_t * 6)()
    assert sq.raw().sq_encoded_sizes(ctypes.byref(f), 4, 128, out) == expect


def test_bad_shapes_and_pointers_are_rejected_without_a_device():
    lib = sq.raw()
    f = sq.make_format(64, 8, False)
    out6 = (ctypes.c_size_t * 6)()
    out4 = (ctypes.c_size_t * 4)()
    assert lib.sq_encoded_sizes(ctypes.byref(f), 4, 100, out6) == sq.SQ_ERR_INVALID_ARG     # K % 128
    assert lib.sq_encoded_sizes(ctypes.byref(f), 4, sq.SQ_MAX_K + 128, out6) == sq.SQ_ERR_UNSUPPORTED
    assert lib.sq_encoded_sizes(ctypes.byref(f), -1, 128, out6) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_weights_sizes(ctypes.byref(f), 12, 128, out4) == sq.SQ_ERR_INVALID_ARG    # N % 8
    assert lib.sq_encoded_sizes(None, 4, 128, out6) == sq.SQ_ERR_NULL_POINTER
    assert lib.sq_encoded_sizes(ctypes.byref(f), 4, 128, None) == sq.SQ_ERR_NULL_POINTER
    enc = sq.sq_encoded(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000)
    # null input, misaligned input, positions given to a dynamic format
    assert lib.sq_encode(ctypes.byref(f), None, 4, 128, None, ctypes.byref(enc), None) == sq.SQ_ERR_NULL_POINTER
    assert lib.sq_encode(ctypes.byref(f), 0x1008, 4, 128, None, ctypes.byref(enc), None) == sq.SQ_ERR_ALIGNMENT
    assert lib.sq_encode(ctypes.byref(f), 0x1000, 4, 128, 0x7000, ctypes.byref(enc), None) == sq.SQ_ERR_INVALID_ARG
    bad = sq.sq_encoded(0x1000, 0x2000, None, 0x4000, 0x5000, 0x6000)      # dynamic needs idx
    assert lib.sq_encode(ctypes.byref(f), 0x1000, 4, 128, None, ctypes.byref(bad), None) == sq.SQ_ERR_NULL_POINTER
    fs = sq.make_format(64, 8, True)
    assert lib.sq_encode(ctypes.byref(fs), 0x1000, 4, 128, None, ctypes.byref(enc), None) == sq.SQ_ERR_NULL_POINTER
    w = sq.sq_weights(0x1000, 0x2000, 0x3000, None)
    assert lib.sq_gemm(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 4, 12, 128, 0x8000, None,
                       None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_gemm(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 4, 16, 128, None, None,
                       None) == sq.SQ_ERR_NULL_POINTER
    assert lib.sq_calib_positions(ctypes.byref(f), 0x1000, 8, 128, None, 0, 0x2000, None) == sq.SQ_ERR_INVALID_ARG
    assert sq.sq_status_string(sq.SQ_ERR_ALIGNMENT).startswith("pointer")


def test_zero_sized_problems_are_no_ops():
    lib = sq.raw()
    f = sq.make_format(64, 8, False)
    enc = sq.sq_encoded(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000)
    w = sq.sq_weights(0x1000, 0x2000, 0x3000, None)
    assert lib.sq_encode(ctypes.byref(f), 0x1000, 0, 128, None, ctypes.byref(enc), None) == sq.SQ_OK
    assert lib.sq_gemm(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 0, 16, 128, 0x8000, None,
                       None) == sq.SQ_OK
    assert lib.sq_decode(ctypes.byref(f), ctypes.byref(enc), None, 0, 128, 0x8000, None) == sq.SQ_OK


def test_workspace_entry_points_validate_without_a_device():
    lib = sq.raw()
    f = sq.make_format(64, 8, False)
    enc = sq.sq_encoded(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000)
    w = sq.sq_weights(0x1000, 0x2000, 0x3000, None)
    need = ctypes.c_size_t(123)
    assert lib.sq_gemm_workspace_bytes(ctypes.byref(f), 0, 4096, 4096, ctypes.byref(need)) == sq.SQ_OK
    assert need.value == 0                                                   # nothing to do, nothing needed
    assert lib.sq_gemm_workspace_bytes(ctypes.byref(f), 16, 4096, 4096, None) == sq.SQ_ERR_NULL_POINTER
    assert lib.sq_gemm_workspace_bytes(ctypes.byref(f), 16, 12, 4096, ctypes.byref(need)) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_gemm_workspace_bytes(ctypes.byref(f), 16, 4096, 100, ctypes.byref(need)) == sq.SQ_ERR_INVALID_ARG
    # sq_gemm_ws: a misaligned workspace is an argument error, a zero-sized problem is a no-op
    assert lib.sq_gemm_ws(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 4, 16, 128, 0x8000, None,
                          0x9004, 4096, None) == sq.SQ_ERR_ALIGNMENT
    assert lib.sq_gemm_ws(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 0, 16, 128, 0x8000, None,
                          0x9000, 4096, None) == sq.SQ_OK
    # sq_gemm_static_scratch: sizes beyond its fixed array are refused before anything else is looked at
    assert lib.sq_gemm_static_scratch(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 129, 16, 128,
                                      0x8000, None, None) == sq.SQ_ERR_UNSUPPORTED
    assert lib.sq_gemm_static_scratch(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 128, 16392, 128,
                                      0x8000, None, None) == sq.SQ_ERR_UNSUPPORTED
    assert lib.sq_gemm_static_scratch(ctypes.byref(f), ctypes.byref(enc), ctypes.byref(w), None, 0, 16, 128,
                                      0x8000, None, None) == sq.SQ_OK
    assert sq.SQ_STATIC_SCRATCH_BYTES == 16 << 20
