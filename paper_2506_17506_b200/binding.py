"""Thin ctypes binding onto ``libverilocc.so``: argument marshalling only.

Same names as the C ABI (``include/verilocc.h``).  torch is used for device memory and
streams, nothing else; every step of the check runs in the library's CUDA kernels.
Importing this module fails loudly when the library has not been built
(``python -m paper_2506_17506_b200.build``); there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libverilocc.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_17506_b200.build` "
                      "(needs nvcc); this package has no CPU fallback")
_lib = C.CDLL(LIB_PATH)

VL_OK = 0
VL_ERR_INVALID_ARG, VL_ERR_MALFORMED_PROGRAM, VL_ERR_NOT_STRICT, VL_ERR_LIVENESS_NOT_RUN = -1, -2, -3, -4
VL_ERR_UNSUPPORTED, VL_ERR_NO_CONVERGE, VL_ERR_CUDA, VL_ERR_DEVICE_WAIT = -5, -6, -7, -8
VL_PASS, VL_INCONSISTENT, VL_OUT_OF_RANGE, VL_INTERFERENCE = 1, 2, 4, 8
VL_OPT_CHUNK_INSTRS, VL_OPT_GROUP, VL_OPT_THREADS, VL_OPT_SUB_BATCH, VL_OPT_KERNEL_TIMING, VL_OPT_LANES = 1, 2, 3, 4, 5, 6
VL_OPT_TEST_WAIT = 7
VL_OPT_PREFETCH_TILES = 8
VL_OPT_STAGGER_US = 9

EXPORTS = ["vl_program_create", "vl_program_destroy", "vl_program_set_option", "vl_liveness", "vl_liveness_batch",
           "vl_liveness_result", "vl_verify", "vl_verify_batch", "vl_verify_host", "vl_verify_status",
           "vl_kernel_launches", "vl_kernel_times", "vl_last_cuda_error", "vl_strerror", "vl_block_liveness_static",
           "vl_resample_stats", "vl_verify_until_pass", "vl_program_set_constraints", "vl_diagnose", "vl_occupied_masks",
           "vl_dict_layout", "vl_verify_dict"]

VERDICT_DTYPE = np.dtype([("flags", "<u4"), ("first_violation_instr", "<i4"),
                          ("conflict_pairs", "<u4"), ("bank_conflicts", "<u4")])


class vl_program_desc(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_blocks", "n_instrs", "n_vregs", "n_operands", "n_edges", "P", "B")] + [
        ("block_instr_off", C.c_void_p), ("succ_off", C.c_void_p), ("succ", C.c_void_p),
        ("instr_op_off", C.c_void_p), ("instr_n_defs", C.c_void_p), ("op_vreg", C.c_void_p),
        ("vreg_width", C.c_void_p)]


_lib.vl_program_create.restype = C.c_int
_lib.vl_program_create.argtypes = [C.POINTER(vl_program_desc), C.c_int, C.POINTER(C.c_void_p)]
_lib.vl_program_destroy.restype = None
_lib.vl_program_destroy.argtypes = [C.c_void_p]
_lib.vl_program_set_option.restype = C.c_int
_lib.vl_program_set_option.argtypes = [C.c_void_p, C.c_int, C.c_uint32]
_lib.vl_kernel_times.restype = C.c_int
_lib.vl_kernel_times.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_uint32)]
_lib.vl_liveness.restype = C.c_int
_lib.vl_liveness.argtypes = [C.c_void_p, C.c_void_p]
_lib.vl_liveness_batch.restype = C.c_int
_lib.vl_liveness_batch.argtypes = [C.c_uint32, C.c_void_p, C.c_void_p]
_lib.vl_liveness_result.restype = C.c_int
_lib.vl_liveness_result.argtypes = [C.c_void_p] + [C.POINTER(C.c_void_p)] * 4 + [C.POINTER(C.c_uint64)]
_lib.vl_verify_dict.restype = C.c_int
_lib.vl_verify_dict.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
_lib.vl_dict_layout.restype = C.c_int
_lib.vl_dict_layout.argtypes = [C.c_void_p, C.POINTER(C.c_uint32), C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]
_lib.vl_verify.restype = C.c_int
_lib.vl_verify.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
_lib.vl_verify_batch.restype = C.c_int
_lib.vl_verify_batch.argtypes = [C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.vl_verify_host.restype = C.c_int
_lib.vl_verify_host.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
_lib.vl_verify_status.restype = C.c_int
_lib.vl_verify_status.argtypes = [C.c_void_p, C.c_void_p]
_lib.vl_kernel_launches.restype = C.c_uint64
_lib.vl_kernel_launches.argtypes = []
_lib.vl_last_cuda_error.restype = C.c_int
_lib.vl_last_cuda_error.argtypes = [C.c_void_p]
_lib.vl_strerror.restype = C.c_char_p
_lib.vl_strerror.argtypes = [C.c_int]


_lib.vl_block_liveness_static.restype = C.c_int
_lib.vl_block_liveness_static.argtypes = [C.c_int, C.c_uint32, C.c_uint32] + [C.c_void_p] * 9
VL_STATIC_SCRATCH_WORDS = 1 << 18
_lib.vl_resample_stats.restype = C.c_int
_lib.vl_resample_stats.argtypes = [C.c_int, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_void_p]
_lib.vl_verify_until_pass.restype = C.c_int
_lib.vl_verify_until_pass.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p]
VL_MAX_PASS_AT = 8
VL_MAX_CLASSES = 8


class vl_constraints(C.Structure):
    _fields_ = [("vreg_align", C.c_void_p), ("vreg_class", C.c_void_p), ("n_classes", C.c_uint32),
                ("class_lo", C.c_void_p), ("class_hi", C.c_void_p), ("reserved_mask", C.c_void_p)]


_lib.vl_diagnose.restype = C.c_int
_lib.vl_diagnose.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.vl_occupied_masks.restype = C.c_int
_lib.vl_occupied_masks.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.vl_program_set_constraints.restype = C.c_int
_lib.vl_program_set_constraints.argtypes = [C.c_void_p, C.c_void_p]
SAMPLE_STATS_DTYPE = np.dtype([("first_pass", "<u8"), ("n_pass", "<u8")])


class VlError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        self.code = code
        msg = f"{where}: {vl_strerror(code)} ({code})"
        if cuda:
            msg += f" [cuda error {cuda}]"
        super().__init__(msg)


def vl_strerror(code: int) -> str:
    return _lib.vl_strerror(code).decode()


def vl_kernel_launches() -> int:
    return int(_lib.vl_kernel_launches())


def _stream_ptr(stream) -> C.c_void_p:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(int(getattr(stream, "cuda_stream", stream)))


def make_desc(prog):
    """(descriptor, keep-alive arrays) from any object with the descriptor's fields as numpy arrays."""
    keep = dict(
        block_instr_off=np.ascontiguousarray(prog.block_instr_off, dtype=np.uint32),
        succ_off=np.ascontiguousarray(prog.succ_off, dtype=np.uint32),
        succ=np.ascontiguousarray(prog.succ, dtype=np.uint32),
        instr_op_off=np.ascontiguousarray(prog.instr_op_off, dtype=np.uint32),
        instr_n_defs=np.ascontiguousarray(prog.instr_n_defs, dtype=np.uint8),
        op_vreg=np.ascontiguousarray(prog.op_vreg, dtype=np.uint32),
        vreg_width=np.ascontiguousarray(prog.vreg_width, dtype=np.uint8),
    )
    def ptr(a):
        return a.ctypes.data if a.size else None
    d = vl_program_desc(prog.n_blocks, prog.n_instrs, prog.n_vregs, prog.n_operands, prog.n_edges, prog.P, prog.B,
                        ptr(keep["block_instr_off"]), ptr(keep["succ_off"]), ptr(keep["succ"]),
                        ptr(keep["instr_op_off"]), ptr(keep["instr_n_defs"]), ptr(keep["op_vreg"]),
                        ptr(keep["vreg_width"]))
    return d, keep


def vl_program_create_raw(desc: vl_program_desc, device: int = 0):
    """Returns (code, handle) without raising; for error-path tests."""
    h = C.c_void_p()
    rc = _lib.vl_program_create(C.byref(desc) if desc is not None else None, device, C.byref(h))
    return rc, h


class _DevView:
    """Borrowed view of library-owned device memory (int32 elements) for torch.as_tensor."""

    def __init__(self, ptr: int, count: int):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<i4", "data": (ptr, False), "version": 2}


class Program:
    """Owns a ``vl_program`` handle."""

    def __init__(self, prog, device: int = 0):
        self.n_blocks, self.n_instrs, self.n_vregs = prog.n_blocks, prog.n_instrs, prog.n_vregs
        self.n_operands = prog.n_operands
        self.pitch = max(8, (prog.n_operands + 7) // 8 * 8)
        self.device = device
        desc, keep = make_desc(prog)
        self._h = C.c_void_p()
        rc = _lib.vl_program_create(C.byref(desc), device, C.byref(self._h))
        if rc != VL_OK:
            self._h = C.c_void_p()
            raise VlError(rc, "vl_program_create")

    def _check(self, rc: int, where: str):
        if rc != VL_OK:
            raise VlError(rc, where, _lib.vl_last_cuda_error(self._h))

    def set_option(self, option: int, value: int):
        self._check(_lib.vl_program_set_option(self._h, option, value), "vl_program_set_option")

    def set_constraints(self, vreg_align=None, vreg_class=None, class_ranges=None, reserved=None, P=None):
        """Hardware rules for the Realizability check: per-vreg alignment, per-vreg class with the
        half-open register range of every class, reserved register numbers.  No argument clears them."""
        keep = []
        c = vl_constraints()
        if vreg_align is not None:
            a = np.ascontiguousarray(vreg_align, dtype=np.uint8); keep.append(a); c.vreg_align = a.ctypes.data
        if vreg_class is not None:
            a = np.ascontiguousarray(vreg_class, dtype=np.uint8); keep.append(a); c.vreg_class = a.ctypes.data
            lo = np.ascontiguousarray([r[0] for r in class_ranges], dtype=np.uint32)
            hi = np.ascontiguousarray([r[1] for r in class_ranges], dtype=np.uint32)
            keep += [lo, hi]
            c.n_classes, c.class_lo, c.class_hi = len(lo), lo.ctypes.data, hi.ctypes.data
        if reserved is not None:
            m = np.zeros((P + 31) // 32 + 1, dtype=np.uint32)
            for r in reserved:
                if r < P:
                    m[r >> 5] |= np.uint32(1 << (r & 31))
            keep.append(m); c.reserved_mask = m.ctypes.data
        self._check(_lib.vl_program_set_constraints(self._h, C.byref(c)), "vl_program_set_constraints")

    def vl_liveness(self, stream=None):
        self._check(_lib.vl_liveness(self._h, _stream_ptr(stream)), "vl_liveness")

    def vl_liveness_wait(self):
        """Blocks the host until the last vl_liveness run has finished and reports its outcome
        (vl_liveness_result with no output pointers)."""
        self._check(_lib.vl_liveness_result(self._h, None, None, None, None, None), "vl_liveness_result")

    def vl_liveness_result(self):
        """Copies of the liveness results as numpy arrays:
        (blk_live_in [nB, W] u32, blk_live_out [nB, W] u32, lo_off [nI+1] u32, lo [len] u32)."""
        import torch
        p = [C.c_void_p() for _ in range(4)]
        n = C.c_uint64()
        self._check(_lib.vl_liveness_result(self._h, *[C.byref(x) for x in p], C.byref(n)), "vl_liveness_result")
        W = max(1, (self.n_vregs + 31) // 32)
        sizes = [self.n_blocks * W, self.n_blocks * W, self.n_instrs + 1, int(n.value)]
        out = []
        torch.cuda.synchronize(self.device)
        for ptr, cnt in zip(p, sizes):
            if cnt:
                view = _DevView(ptr.value, cnt)
                out.append(torch.as_tensor(view, device=f"cuda:{self.device}").cpu().numpy().view(np.uint32).copy())
            else:
                out.append(np.zeros(0, dtype=np.uint32))
        return out[0].reshape(self.n_blocks, W), out[1].reshape(self.n_blocks, W), out[2], out[3]

    def vl_verify(self, cand, out=None, stream=None):
        """cand: CUDA uint16 tensor [K, pitch]; returns a CUDA int32 tensor [K, 4]
        (flags, first_violation_instr, conflict_pairs, bank_conflicts)."""
        import torch
        assert cand.is_cuda and cand.dtype in (torch.uint16, torch.int16) and cand.dim() == 2 and cand.is_contiguous()
        K, pitch = cand.shape
        if out is None:
            out = torch.empty((K, 4), dtype=torch.int32, device=cand.device)
        self._check(_lib.vl_verify(self._h, cand.data_ptr(), K, pitch, out.data_ptr(), _stream_ptr(stream)), "vl_verify")
        return out

    def vl_dict_layout(self):
        """(dict_off [n_blocks+1], dict_vreg [n_entries]) of rows in dictionary form, as numpy copies."""
        n = C.c_uint32(0)
        off, vreg = C.c_void_p(), C.c_void_p()
        self._check(_lib.vl_dict_layout(self._h, C.byref(n), C.byref(off), C.byref(vreg)), "vl_dict_layout")
        d_off = np.ctypeslib.as_array(C.cast(off, C.POINTER(C.c_uint32)), shape=(self.n_blocks + 1,)).copy()
        d_vreg = (np.ctypeslib.as_array(C.cast(vreg, C.POINTER(C.c_uint32)), shape=(n.value,)).copy()
                  if n.value else np.zeros(0, dtype=np.uint32))
        return d_off, d_vreg

    def vl_verify_dict(self, rows, out=None, stream=None):
        """rows: CUDA uint16 tensor [K, pitch] of dictionary rows; returns a CUDA int32 tensor [K, 4]."""
        import torch
        assert rows.is_cuda and rows.dtype in (torch.uint16, torch.int16) and rows.dim() == 2 and rows.is_contiguous()
        K, pitch = rows.shape
        if out is None:
            out = torch.empty((K, 4), dtype=torch.int32, device=rows.device)
        self._check(_lib.vl_verify_dict(self._h, rows.data_ptr(), K, pitch, out.data_ptr(), _stream_ptr(stream)),
                    "vl_verify_dict")
        return out

    def vl_verify_host(self, cand: "np.ndarray | object", out: np.ndarray | None = None, stream=None):
        """cand: host uint16 [K, pitch] (numpy array or pinned CPU tensor); returns a numpy verdict array."""
        if hasattr(cand, "data_ptr"):
            K, pitch = cand.shape
            ptr = cand.data_ptr()
        else:
            assert cand.dtype == np.uint16 and cand.ndim == 2 and cand.flags.c_contiguous
            K, pitch = cand.shape
            ptr = cand.ctypes.data
        if out is None:
            out = np.zeros(K, dtype=VERDICT_DTYPE)
        optr = out.data_ptr() if hasattr(out, "data_ptr") else out.ctypes.data
        self._check(_lib.vl_verify_host(self._h, ptr, K, pitch, optr, _stream_ptr(stream)), "vl_verify_host")
        return out

    def vl_verify_until_pass(self, cand, batch_rows: int, out=None, stream=None):
        """The re-sampling loop with early exit over a CUDA uint16 [K, pitch] tensor; returns
        (verdict tensor, rows checked, first passing row or K)."""
        import torch
        assert cand.is_cuda and cand.dtype in (torch.uint16, torch.int16) and cand.dim() == 2 and cand.is_contiguous()
        K, pitch = cand.shape
        if out is None:
            out = torch.zeros((K, 4), dtype=torch.int32, device=cand.device)
        done, first = C.c_uint64(0), C.c_uint64(0)
        self._check(_lib.vl_verify_until_pass(self._h, cand.data_ptr(), K, pitch, batch_rows, out.data_ptr(),
                                              C.byref(done), C.byref(first), _stream_ptr(stream)), "vl_verify_until_pass")
        return out, int(done.value), int(first.value)

    def vl_diagnose(self, row, cap: int = 1 << 16, n_banks: int = 4, stream=None):
        """Diagnostics of one candidate (CUDA uint16 tensor of n_operands entries or more): returns
        (conflict records [n, 3] as numpy, total count, kinds per instruction, bank histogram)."""
        import torch
        dev = row.device
        rec = torch.zeros((max(cap, 1), 3), dtype=torch.int32, device=dev)
        cnt = torch.zeros(1, dtype=torch.int64, device=dev)
        kinds = torch.zeros(max(self.n_instrs, 1), dtype=torch.uint8, device=dev)
        hist = torch.zeros(n_banks, dtype=torch.int64, device=dev)
        self._check(_lib.vl_diagnose(self._h, row.data_ptr(), cap, rec.data_ptr(), cnt.data_ptr(), kinds.data_ptr(),
                                     hist.data_ptr(), _stream_ptr(stream)), "vl_diagnose")
        torch.cuda.synchronize(dev)
        n = int(cnt.item())
        return (rec[: min(n, cap)].cpu().numpy().view(np.uint32), n, kinds[: self.n_instrs].cpu().numpy(),
                hist.cpu().numpy().view(np.uint64))

    def vl_occupied_masks(self, row, P: int, stream=None):
        """uint8 numpy array [n_instrs, P]: registers the definitions of every instruction must keep off,
        for one candidate (CUDA uint16 tensor; entries >= P mean "no register yet")."""
        import torch
        W = (P + 31) // 32
        masks = torch.zeros((max(self.n_instrs, 1), W), dtype=torch.int32, device=row.device)
        self._check(_lib.vl_occupied_masks(self._h, row.data_ptr(), masks.data_ptr(), _stream_ptr(stream)),
                    "vl_occupied_masks")
        torch.cuda.synchronize(row.device)
        words = masks[: self.n_instrs].cpu().numpy().view(np.uint32)
        bits = np.unpackbits(words.view(np.uint8).reshape(self.n_instrs, W * 4), axis=1, bitorder="little")
        return bits[:, :P]

    def vl_verify_status(self, stream=None):
        self._check(_lib.vl_verify_status(self._h, _stream_ptr(stream)), "vl_verify_status")

    def vl_kernel_times(self):
        """Summed device time (ms) of the four verify kernels since the last call, and the passes summed."""
        ms = (C.c_float * 4)()
        n = C.c_uint32(0)
        self._check(_lib.vl_kernel_times(self._h, ms, C.byref(n)), "vl_kernel_times")
        return [float(x) for x in ms], int(n.value)

    @property
    def handle(self):
        return self._h

    def close(self):
        if self._h:
            _lib.vl_program_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def vl_block_liveness_static(n_blocks, n_vregs, block_instr_off, succ_off, succ, instr_op_off, instr_n_defs, op_vreg,
                             live_in, live_out, device: int = 0, stream=None) -> int:
    """Block liveness with no allocation inside the library: every argument after the two counts is
    a CUDA tensor the caller owns (CSR arrays in, the two bitset buffers out).  Returns the C
    return code without raising, so callers can test the refusal of oversized programs."""
    def ptr(t):
        return t.data_ptr() if t is not None and t.numel() else None
    return int(_lib.vl_block_liveness_static(device, n_blocks, n_vregs, ptr(block_instr_off), ptr(succ_off), ptr(succ),
                                             ptr(instr_op_off), ptr(instr_n_defs), ptr(op_vreg), ptr(live_in),
                                             ptr(live_out), _stream_ptr(stream)))


def vl_liveness_batch(programs, stream=None):
    """vl_liveness on every program of the list in one call."""
    n = len(programs)
    hp = (C.c_void_p * n)(*[p.handle for p in programs])
    rc = _lib.vl_liveness_batch(n, hp, _stream_ptr(stream))
    if rc != VL_OK:
        raise VlError(rc, "vl_liveness_batch")


def vl_verify_batch(programs, cands, outs=None, stream=None):
    """One call over n programs; cands[j] is the CUDA uint16 [K_j, pitch_j] tensor of program j."""
    import torch
    n = len(programs)
    if outs is None:
        outs = [torch.empty((c.shape[0], 4), dtype=torch.int32, device=c.device) for c in cands]
    hp = (C.c_void_p * n)(*[p.handle for p in programs])
    cp = (C.c_void_p * n)(*[c.data_ptr() for c in cands])
    op = (C.c_void_p * n)(*[o.data_ptr() for o in outs])
    Ks = (C.c_uint64 * n)(*[c.shape[0] for c in cands])
    Ps = (C.c_uint64 * n)(*[c.shape[1] for c in cands])
    rc = _lib.vl_verify_batch(n, hp, cp, Ks, Ps, op, _stream_ptr(stream))
    if rc != VL_OK:
        raise VlError(rc, "vl_verify_batch")
    return outs


def vl_resample_stats(outs, ks=(1, 10, 100), device: int = 0, stream=None):
    """Per test case (one CUDA int32 [K_j, 4] verdict tensor each) the first passing row and the
    number of passing rows, and the summary over the test cases for the attempt limits ``ks``.
    Returns (records as a numpy array, summary as a dict); waits for the stream to read them back."""
    import torch
    n = len(outs)
    stats = torch.zeros((max(n, 1), 2), dtype=torch.int64, device=f"cuda:{device}")
    summ = torch.zeros(4 + VL_MAX_PASS_AT, dtype=torch.int64, device=f"cuda:{device}")
    op = (C.c_void_p * max(n, 1))(*[o.data_ptr() if o.numel() else None for o in outs])
    Ks = (C.c_uint64 * max(n, 1))(*[o.shape[0] for o in outs])
    kk = (C.c_uint32 * max(len(ks), 1))(*ks)
    rc = _lib.vl_resample_stats(device, n, op, Ks, len(ks), kk, stats.data_ptr(), summ.data_ptr(), _stream_ptr(stream))
    if rc != VL_OK:
        raise VlError(rc, "vl_resample_stats")
    torch.cuda.synchronize(device)
    rec = stats[:n].cpu().numpy().view(np.uint64).copy().view(SAMPLE_STATS_DTYPE).reshape(-1)
    s = summ.cpu().numpy().view(np.uint64)
    return rec, dict(n_cases=int(s[0]), n_solved=int(s[1]), sum_tries=int(s[2]), max_tries=int(s[3]),
                     pass_at=[int(x) for x in s[4:4 + len(ks)]])


def verdicts_to_numpy(t) -> np.ndarray:
    """CUDA/CPU int32 [K, 4] tensor -> structured numpy array."""
    a = t.detach().cpu().numpy().astype(np.int32, copy=False)
    return np.ascontiguousarray(a).view(VERDICT_DTYPE).reshape(-1)
