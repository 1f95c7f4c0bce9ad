"""The shared library loads without a GPU and exports every symbol the header declares."""

import ctypes
import os
import re

import numpy as np

import paper_2508_20258_b200 as sp
from paper_2508_20258_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "swizzleperf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert set(names) == set(binding.EXPORTS)
    L = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert getattr(L, n) is not None


def test_struct_layout_matches_header():
    assert ctypes.sizeof(binding.SpParams) == 72
    assert ctypes.sizeof(binding.SpTraceRec) == 64 and binding.TRACE_DTYPE.itemsize == 64
    assert binding.SpParams.custom_perm.offset == 40 and binding.SpParams.tile_m.offset == 48


def test_gemm_rejects_bad_arguments_before_touching_a_device():
    L = sp.lib()
    p = sp.make_params(tile_m=128, tile_n=128)
    a = 0x1000  # never dereferenced: every check below fails on the host first
    assert L.sp_gemm(None, a, a, 128, 128, 128, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_INVALID_ARG
    assert L.sp_gemm(a, a, a, 0, 128, 128, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_INVALID_ARG
    assert L.sp_gemm(a + 8, a, a, 128, 128, 128, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_ALIGNMENT
    assert L.sp_gemm(a, a, a, 128, 128, 100, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_ALIGNMENT
    assert L.sp_gemm(a, a, a, 128, 124, 128, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_ALIGNMENT
    q = sp.make_params(tile_m=64, tile_n=128)
    assert L.sp_gemm(a, a, a, 128, 128, 128, sp.ROW_MAJOR, ctypes.byref(q), None) == sp.ERR_UNSUPPORTED
    q = sp.make_params(tile_m=128, tile_n=128, custom_perm=[0, 0])
    assert L.sp_gemm(a, a, a, 128, 256, 128, sp.CUSTOM, ctypes.byref(q), None) == sp.ERR_NOT_BIJECTIVE
    q = sp.make_params(tile_m=128, tile_n=128, num_xcds=4)
    assert L.sp_gemm(a, a, a, 256, 640, 128, sp.XCD, ctypes.byref(q), None) == sp.ERR_NOT_BIJECTIVE
    q = sp.make_params(tile_m=128, tile_n=128, group=0)
    assert L.sp_gemm(a, a, a, 256, 640, 128, sp.GROUP_M, ctypes.byref(q), None) == sp.ERR_INVALID_ARG
    assert L.sp_gemm_trace(a, a, a, 128, 128, 128, sp.ROW_MAJOR, ctypes.byref(p), None, None) == sp.ERR_INVALID_ARG
    assert sp.last_error() != ""
    smid = np.zeros(4, dtype=np.int32)
    assert L.sp_probe_dispatch(3, 2, smid.ctypes.data, smid.ctypes.data) == sp.ERR_INVALID_ARG


def test_stencil_and_transpose_reject_bad_arguments_before_touching_a_device():
    L = sp.lib()
    a, b = 0x1000, 0x200000
    assert L.sp_stencil2d(a, b, 64, 126, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_stencil2d(a + 4, b, 64, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_stencil2d(a, a, 64, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_stencil2d(None, b, 64, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_stencil2d(a, b, -1, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_stencil2d(a, b, 64, 128, 1.0, float("nan"), sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    bad = sp.make_params(num_xcds=4, xcd_balanced=0)      # 10 tiles: the printed formula with X = 4 leaves [0, 10)
    assert L.sp_stencil2d(a, b, 640, 128, 1.0, 0.0, sp.XCD, ctypes.byref(bad), None) == sp.ERR_NOT_BIJECTIVE
    assert L.sp_transpose(a, b, 64, 60, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_transpose(a, a, 64, 64, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    first = ctypes.c_int32(0)
    assert L.sp_streamk_plan(16, 4, 8, ctypes.byref(first), None) == sp.ERR_INVALID_ARG


def test_flag_and_mode_constants_match_the_header():
    text = open(os.path.join(ROOT, "include", "swizzleperf.h")).read()
    defs = {m.group(1): int(m.group(2)) for m in re.finditer(r"#define\s+(SP_[A-Z_0-9]+)\s+(\d+)u?\b", text)}
    flags = {k[len("SP_FLAG_"):]: v for k, v in defs.items() if k.startswith("SP_FLAG_")}
    assert len(flags) >= 12 and len(set(flags.values())) == len(flags)            # one bit each, no bit twice
    assert all(v & (v - 1) == 0 for v in flags.values())
    for name, value in flags.items():
        assert getattr(binding, "FLAG_" + name) == value, name
    assert (defs["SP_SOFTMAX_SINGLE_PASS"], defs["SP_SOFTMAX_TWO_PHASE"], defs["SP_SOFTMAX_TWO_PHASE_REVERSED"]) == \
        (binding.SOFTMAX_SINGLE_PASS, binding.SOFTMAX_TWO_PHASE, binding.SOFTMAX_TWO_PHASE_REVERSED)
    assert (defs["SP_SOFTMAX_TILE_M"], defs["SP_SOFTMAX_TILE_N"]) == binding.SOFTMAX_TILE
    assert (defs["SP_STENCIL_TILE_M"], defs["SP_STENCIL_TILE_N"]) == binding.STENCIL_TILE
    assert defs["SP_TRANSPOSE_TILE"] == binding.TRANSPOSE_TILE


def test_softmax_rejects_bad_arguments_before_touching_a_device():
    L = sp.lib()
    a, b = 0x1000, 0x200000
    assert L.sp_softmax(a, b, 64, 126, 0, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_softmax(a + 4, b, 64, 128, 0, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_softmax(a, a, 64, 128, 1, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_softmax(a, b, 64, 128, 7, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_softmax(a, b, 0, 128, 0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_softmax(a, b, 64, 131076, 0, sp.ROW_MAJOR, None, None) == sp.ERR_UNSUPPORTED    # a row must fit the eight buffers of a cluster
    bad = sp.make_params(num_xcds=4, xcd_balanced=0)      # 5 x 2 tiles of 32 x 512: the printed formula leaves [0, 10)
    assert L.sp_softmax(a, b, 160, 1024, 1, sp.XCD, ctypes.byref(bad), None) == sp.ERR_NOT_BIJECTIVE
