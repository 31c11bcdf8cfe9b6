"""Host-side checks that need no GPU: the library loads, exports every declared symbol,
and rejects malformed descriptors before touching the device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2506_17506_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2506_17506_b200 import build
    build.build()
    from paper_2506_17506_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(B):
    header = open(os.path.join(ROOT, "include", "verilocc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(vl_[a-z_0-9]+)\s*\(", header))
    assert {"vl_liveness", "vl_verify"} <= declared
    lib = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)


def test_strerror_and_counters(B):
    assert B.vl_strerror(0) == "ok"
    for code in range(-8, 0):
        assert B.vl_strerror(code) not in ("ok", "unknown error")
    assert B.vl_strerror(-99) == "unknown error"
    assert B.vl_kernel_launches() == 0


def _good():
    return synth.program_from_lists([[([0], []), ([1], [0]), ([], [1, 0])], [([0], [1])]], [(0, 1), (1, 1)], 2, [1, 2], 8)


def _create(B, p):
    desc, keep = B.make_desc(p)
    rc, h = B.vl_program_create_raw(desc)
    assert not h.value or rc == 0
    return rc


@pytest.mark.parametrize("name", ["blk_off_end", "blk_off_order", "succ_range", "op_off_order", "ndefs", "vreg_range",
                                  "zero_width", "dup_def", "zero_P", "big_P", "zero_B", "no_blocks"])
def test_malformed_descriptors_are_rejected(B, name):
    p = _good()
    expect = B.VL_ERR_MALFORMED_PROGRAM
    if name == "blk_off_end":
        p.block_instr_off[-1] += 1
    elif name == "blk_off_order":
        p.block_instr_off[1] = 9
    elif name == "succ_range":
        p.succ[0] = 7
    elif name == "op_off_order":
        p.instr_op_off[1], p.instr_op_off[2] = p.instr_op_off[2], p.instr_op_off[1]
    elif name == "ndefs":
        p.instr_n_defs[0] = 3
    elif name == "vreg_range":
        p.op_vreg[0] = 2
    elif name == "zero_width":
        p.vreg_width[1] = 0
    elif name == "dup_def":
        p = synth.program_from_lists([[([0, 0], [])]], [], 1, [1], 4)
    elif name == "zero_P":
        p.P, expect = 0, B.VL_ERR_INVALID_ARG
    elif name == "big_P":
        p.P, expect = 65536, B.VL_ERR_INVALID_ARG
    elif name == "zero_B":
        p.B, expect = 0, B.VL_ERR_INVALID_ARG
    elif name == "no_blocks":
        p.n_blocks, expect = 0, B.VL_ERR_INVALID_ARG
    assert _create(B, p) == expect


def test_null_arguments(B):
    assert B.vl_program_create_raw(None)[0] == B.VL_ERR_INVALID_ARG
    lib = C.CDLL(B.LIB_PATH)
    lib.vl_program_destroy(None)
    lib.vl_liveness.restype = C.c_int
    assert lib.vl_liveness(None, None) == B.VL_ERR_INVALID_ARG
    lib.vl_verify.restype = C.c_int
    lib.vl_verify.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
    assert lib.vl_verify(None, None, 1, 8, None, None) == B.VL_ERR_INVALID_ARG
    lib.vl_liveness_batch.restype = C.c_int
    lib.vl_liveness_batch.argtypes = [C.c_uint32, C.c_void_p, C.c_void_p]
    assert lib.vl_liveness_batch(0, None, None) == B.VL_OK
    assert lib.vl_liveness_batch(2, None, None) == B.VL_ERR_INVALID_ARG
    two_nulls = (C.c_void_p * 2)(None, None)
    assert lib.vl_liveness_batch(2, two_nulls, None) == B.VL_ERR_INVALID_ARG


def test_resample_argument_checks(B):
    lib = C.CDLL(B.LIB_PATH)
    f = lib.vl_resample_stats
    f.restype = C.c_int
    f.argtypes = [C.c_int, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    ks = (C.c_uint32 * 9)(*range(1, 10))
    assert f(0, 0, None, None, 0, None, None, None, None) == B.VL_OK              # nothing to do
    assert f(0, 0, None, None, 9, ks, None, None, None) == B.VL_ERR_INVALID_ARG   # too many attempt limits
    assert f(0, 0, None, None, 2, None, None, None, None) == B.VL_ERR_INVALID_ARG # limits announced, none given
    assert f(0, 1, None, None, 0, None, None, None, None) == B.VL_ERR_INVALID_ARG # a test case without arrays
    outs, K = (C.c_void_p * 1)(None), (C.c_uint64 * 1)(5)
    assert f(0, 1, outs, K, 0, None, C.c_void_p(64), None, None) == B.VL_ERR_INVALID_ARG   # rows announced, no verdicts
    outs = (C.c_void_p * 1)(C.c_void_p(72))
    assert f(0, 1, outs, K, 0, None, C.c_void_p(64), None, None) == B.VL_ERR_INVALID_ARG   # verdicts not 16-byte aligned
    outs = (C.c_void_p * 1)(C.c_void_p(64))
    assert f(0, 1, outs, K, 0, None, C.c_void_p(68), None, None) == B.VL_ERR_INVALID_ARG   # records not 8-byte aligned
    g = lib.vl_verify_until_pass
    g.restype = C.c_int
    g.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    n = C.c_uint64(0)
    assert g(None, None, 1, 8, 1, None, C.byref(n), C.byref(n), None) == B.VL_ERR_INVALID_ARG
    h = lib.vl_program_set_constraints
    h.restype = C.c_int
    h.argtypes = [C.c_void_p, C.c_void_p]
    assert h(None, None) == B.VL_ERR_INVALID_ARG
    d = lib.vl_diagnose
    d.restype = C.c_int
    d.argtypes = [C.c_void_p] * 2 + [C.c_uint64] + [C.c_void_p] * 5
    assert d(None, None, 0, None, None, None, None, None) == B.VL_ERR_INVALID_ARG
    m = lib.vl_occupied_masks
    m.restype = C.c_int
    m.argtypes = [C.c_void_p] * 4
    assert m(None, None, None, None) == B.VL_ERR_INVALID_ARG
