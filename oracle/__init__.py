"""ctypes access to the CPU oracle (``vl_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.  The C file is built
with gcc on first use (``build()``), next to the source.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vl_oracle.c")
_LIB = os.path.join(_HERE, "libvl_oracle.so")
# The mutation test points these at a deliberately broken copy in a temp directory.
if os.environ.get("VL_ORACLE_MUTANT_SRC"):
    _SRC = os.environ["VL_ORACLE_MUTANT_SRC"]
    _LIB = os.path.splitext(_SRC)[0] + ".so"

PASS, INCONSISTENT, OUT_OF_RANGE, INTERFERENCE = 1, 2, 4, 8

SAMPLE_STATS_DTYPE = np.dtype([("first_pass", "<u8"), ("n_pass", "<u8")])

VERDICT_DTYPE = np.dtype([("flags", "<u4"), ("first_violation_instr", "<i4"),
                          ("conflict_pairs", "<u4"), ("bank_conflicts", "<u4")])


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-fPIC", "-shared", _SRC, "-o", _LIB])
    return _LIB


class _Prog(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_blocks", "n_instrs", "n_vregs", "n_operands", "n_edges", "P", "B")] + [
        ("block_instr_off", C.c_void_p), ("succ_off", C.c_void_p), ("succ", C.c_void_p),
        ("instr_op_off", C.c_void_p), ("instr_n_defs", C.c_void_p), ("op_vreg", C.c_void_p),
        ("vreg_width", C.c_void_p), ("vreg_align", C.c_void_p), ("vreg_class", C.c_void_p),
        ("class_lo", C.c_void_p), ("class_hi", C.c_void_p), ("reserved", C.c_void_p)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.vlo_block_liveness.restype = C.c_uint32
        lib.vlo_block_liveness.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
        lib.vlo_instr_liveness.restype = C.c_uint64
        lib.vlo_instr_liveness.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64]
        lib.vlo_verify_rows.restype = None
        lib.vlo_verify_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p]
        lib.vlo_violations.restype = None
        lib.vlo_violations.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.vlo_conflicts.restype = C.c_uint64
        lib.vlo_conflicts.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64]
        lib.vlo_bank_histogram.restype = None
        lib.vlo_bank_histogram.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.vlo_occupied.restype = None
        lib.vlo_occupied.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.vlo_dict_layout.restype = C.c_uint32
        lib.vlo_dict_layout.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.vlo_verify_dict_rows.restype = None
        lib.vlo_verify_dict_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p]
        lib.vlo_sample_stats_of.restype = None
        lib.vlo_sample_stats_of.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        lib.vlo_resample_summary.restype = None
        lib.vlo_resample_summary.argtypes = [C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


@dataclass
class Liveness:
    blk_live_in: np.ndarray    # uint8 [n_blocks, n_vregs]
    blk_live_out: np.ndarray   # uint8 [n_blocks, n_vregs]
    lo_off: np.ndarray         # uint64 [n_instrs+1]
    lo: np.ndarray             # uint32 [lo_off[-1]], ascending inside each instruction
    sweeps: int

    def live_after(self, i: int) -> np.ndarray:
        return self.lo[int(self.lo_off[i]): int(self.lo_off[i + 1])]

    def packed(self, which: str) -> np.ndarray:
        """Block sets as little-endian 32-bit words, [n_blocks, ceil(V/32)]."""
        a = self.blk_live_in if which == "in" else self.blk_live_out
        nB, V = a.shape
        words = (V + 31) // 32
        pad = np.zeros((nB, words * 32), dtype=np.uint8)
        pad[:, :V] = a
        return np.packbits(pad, axis=1, bitorder="little").view("<u4").reshape(nB, words)


class OracleProgram:
    """Keeps the numpy arrays alive and exposes the C struct."""

    def __init__(self, prog):
        self.src = prog
        self.arrays = dict(
            block_instr_off=np.ascontiguousarray(prog.block_instr_off, dtype=np.uint32),
            succ_off=np.ascontiguousarray(prog.succ_off, dtype=np.uint32),
            succ=np.ascontiguousarray(np.concatenate([prog.succ, [0]]), dtype=np.uint32),
            instr_op_off=np.ascontiguousarray(prog.instr_op_off, dtype=np.uint32),
            instr_n_defs=np.ascontiguousarray(np.concatenate([prog.instr_n_defs, [0]]), dtype=np.uint8),
            op_vreg=np.ascontiguousarray(np.concatenate([prog.op_vreg, [0]]), dtype=np.uint32),
            vreg_width=np.ascontiguousarray(np.concatenate([prog.vreg_width, [1]]), dtype=np.uint8),
        )
        self.c = _Prog(prog.n_blocks, prog.n_instrs, prog.n_vregs, prog.n_operands, prog.n_edges, prog.P, prog.B,
                       *[self.arrays[k].ctypes.data for k in
                         ("block_instr_off", "succ_off", "succ", "instr_op_off", "instr_n_defs", "op_vreg", "vreg_width")])
        self.n_blocks, self.n_instrs, self.n_vregs = prog.n_blocks, prog.n_instrs, prog.n_vregs
        self.P = prog.P

    def set_constraints(self, vreg_align=None, vreg_class=None, class_ranges=None, reserved=None):
        """Optional hardware rules for the Realizability check: per-vreg alignment of the base
        register, per-vreg register class with the half-open register range of every class, and
        the set of reserved registers (any iterable of register numbers).  None switches one off."""
        a = self.arrays
        for k in ("vreg_align", "vreg_class", "class_lo", "class_hi", "reserved"):
            a.pop(k, None)
            setattr(self.c, k, None)
        if vreg_align is not None:
            a["vreg_align"] = np.ascontiguousarray(np.concatenate([vreg_align, [1]]), dtype=np.uint8)
        if vreg_class is not None:
            a["vreg_class"] = np.ascontiguousarray(np.concatenate([vreg_class, [0]]), dtype=np.uint8)
            a["class_lo"] = np.ascontiguousarray([r[0] for r in class_ranges], dtype=np.uint32)
            a["class_hi"] = np.ascontiguousarray([r[1] for r in class_ranges], dtype=np.uint32)
        if reserved is not None:
            m = np.zeros(self.P + 1, dtype=np.uint8)
            m[[r for r in reserved if r < self.P]] = 1
            a["reserved"] = m
        for k in ("vreg_align", "vreg_class", "class_lo", "class_hi", "reserved"):
            if k in a:
                setattr(self.c, k, a[k].ctypes.data)

    def liveness(self, order: int = 0) -> Liveness:
        lib = _load()
        nB, V, nI = self.n_blocks, self.n_vregs, self.n_instrs
        lin = np.zeros((nB, V), dtype=np.uint8)
        lout = lin.copy()
        sweeps = lib.vlo_block_liveness(C.byref(self.c), _ptr(lin), _ptr(lout), order)
        lo_off = np.zeros(nI + 1, dtype=np.uint64)
        total = lib.vlo_instr_liveness(C.byref(self.c), _ptr(lout), _ptr(lo_off), None, 0)
        lo = np.zeros(max(int(total), 1), dtype=np.uint32)
        lib.vlo_instr_liveness(C.byref(self.c), _ptr(lout), _ptr(lo_off), _ptr(lo), total)
        return Liveness(lin, lout, lo_off, lo[: int(total)], int(sweeps))

    def verify(self, live: Liveness, rows: np.ndarray) -> np.ndarray:
        """Verdict record for every row of a uint16 [K, pitch] matrix."""
        lib = _load()
        rows = np.ascontiguousarray(rows, dtype=np.uint16)
        if rows.ndim == 1:
            rows = rows[None, :]
        K, pitch = rows.shape
        out = np.zeros(K, dtype=VERDICT_DTYPE)
        lo = live.lo if len(live.lo) else np.zeros(1, np.uint32)
        lib.vlo_verify_rows(C.byref(self.c), _ptr(live.lo_off), _ptr(lo), _ptr(rows), K, pitch, _ptr(out))
        return out

    def dict_layout(self):
        """(dict_off [n_blocks+1], dict_vreg [n_entries], entry_instr [n_entries]) of the per-basic-block
        dictionary form of a candidate: blocks in order, a block's vregs in order of first occurrence."""
        lib = _load()
        n_ops = int(self.src.n_operands)
        off = np.zeros(self.n_blocks + 1, dtype=np.uint32)
        vreg = np.zeros(n_ops + 1, dtype=np.uint32)
        instr = np.zeros(n_ops + 1, dtype=np.uint32)
        n = int(lib.vlo_dict_layout(C.byref(self.c), _ptr(off), _ptr(vreg), _ptr(instr)))
        return off, vreg[:n].copy(), instr[:n].copy()

    def verify_dict(self, live: Liveness, rows: np.ndarray) -> np.ndarray:
        """Verdict record for every row of a uint16 [K, pitch] matrix of dictionary candidates."""
        lib = _load()
        rows = np.ascontiguousarray(rows, dtype=np.uint16)
        if rows.ndim == 1:
            rows = rows[None, :]
        K, pitch = rows.shape
        out = np.zeros(K, dtype=VERDICT_DTYPE)
        lo = live.lo if len(live.lo) else np.zeros(1, np.uint32)
        lib.vlo_verify_dict_rows(C.byref(self.c), _ptr(live.lo_off), _ptr(lo), _ptr(rows), K, pitch, _ptr(out))
        return out

    def violations(self, live: Liveness, row: np.ndarray) -> np.ndarray:
        lib = _load()
        row = np.ascontiguousarray(row, dtype=np.uint16)
        kinds = np.zeros(max(self.n_instrs, 1), dtype=np.uint8)
        lo = live.lo if len(live.lo) else np.zeros(1, np.uint32)
        lib.vlo_violations(C.byref(self.c), _ptr(live.lo_off), _ptr(lo), _ptr(row), _ptr(kinds))
        return kinds[: self.n_instrs]

    def bank_histogram(self, live: Liveness, row: np.ndarray) -> np.ndarray:
        """Extra read cycles of one row per register bank (their sum is the verdict's bank_conflicts)."""
        lib = _load()
        row = np.ascontiguousarray(row, dtype=np.uint16)
        hist = np.zeros(self.src.B, dtype=np.uint64)
        lo = live.lo if len(live.lo) else np.zeros(1, np.uint32)
        lib.vlo_bank_histogram(C.byref(self.c), _ptr(live.lo_off), _ptr(lo), _ptr(row), _ptr(hist))
        return hist

    def occupied(self, live: Liveness, row: np.ndarray) -> np.ndarray:
        """uint8 [n_instrs, P]: registers the definitions of every instruction must keep off."""
        lib = _load()
        row = np.ascontiguousarray(row, dtype=np.uint16)
        occ = np.zeros((max(self.n_instrs, 1), self.P), dtype=np.uint8)
        lo = live.lo if len(live.lo) else np.zeros(1, np.uint32)
        lib.vlo_occupied(C.byref(self.c), _ptr(live.lo_off), _ptr(lo), _ptr(row), _ptr(occ))
        return occ[: self.n_instrs]

    def conflicts(self, live: Liveness, row: np.ndarray) -> np.ndarray:
        """All (instruction, defined vreg, other vreg) overlap records of one row."""
        lib = _load()
        row = np.ascontiguousarray(row, dtype=np.uint16)
        lo = live.lo if len(live.lo) else np.zeros(1, np.uint32)
        n = lib.vlo_conflicts(C.byref(self.c), _ptr(live.lo_off), _ptr(lo), _ptr(row), None, 0)
        tr = np.zeros((max(int(n), 1), 3), dtype=np.uint32)
        lib.vlo_conflicts(C.byref(self.c), _ptr(live.lo_off), _ptr(lo), _ptr(row), _ptr(tr), n)
        return tr[: int(n)]


def sample_stats(verdicts: np.ndarray) -> np.ndarray:
    """First passing row (K if none) and number of passing rows of one verdict array."""
    lib = _load()
    v = np.ascontiguousarray(verdicts, dtype=VERDICT_DTYPE)
    out = np.zeros(1, dtype=SAMPLE_STATS_DTYPE)
    keep = v if len(v) else np.zeros(1, dtype=VERDICT_DTYPE)
    lib.vlo_sample_stats_of(_ptr(keep), len(v), _ptr(out))
    return out[0]


def resample_summary(stats: np.ndarray, K, ks) -> dict:
    """Pass@k counts, attempts summed / largest over the solved test cases (Section 4 of the paper)."""
    lib = _load()
    n = len(stats)
    st = np.ascontiguousarray(stats, dtype=SAMPLE_STATS_DTYPE) if n else np.zeros(1, dtype=SAMPLE_STATS_DTYPE)
    Ks = np.ascontiguousarray(K, dtype=np.uint64) if n else np.zeros(1, dtype=np.uint64)
    kk = np.ascontiguousarray(ks, dtype=np.uint32) if len(ks) else np.zeros(1, dtype=np.uint32)
    out = np.zeros(4 + len(ks), dtype=np.uint64)
    lib.vlo_resample_summary(n, _ptr(st), _ptr(Ks), len(ks), _ptr(kk), _ptr(out))
    return dict(n_cases=int(out[0]), n_solved=int(out[1]), sum_tries=int(out[2]), max_tries=int(out[3]),
                pass_at=[int(x) for x in out[4:]])
