"""The allocation-free block-liveness entry point against the regular one.

Some users of this library call it from places where device memory cannot be allocated any more
(everything was handed to the application's own pools, or an allocation's device-wide stall is not
acceptable).  For them `vl_block_liveness_static` keeps its working sets in a fixed array inside the
library.  The array is shared by all calls and keeps the previous call's contents, so the check
runs different programs back to back: each result must equal what `vl_liveness` gives, bit for bit.
This file sorts last on purpose, so a run that stops at the first failure has seen every other test.
"""
import numpy as np
import pytest

from paper_2506_17506_b200 import synth

pytestmark = pytest.mark.gpu


def _device_csr(torch, p):
    def dev(a, dt):
        return torch.from_numpy(np.ascontiguousarray(a).astype(dt).view(np.int32 if dt == np.uint32 else np.uint8)).cuda()
    return (dev(p.block_instr_off, np.uint32), dev(p.succ_off, np.uint32),
            dev(p.succ if p.n_edges else np.zeros(1), np.uint32), dev(p.instr_op_off, np.uint32),
            dev(p.instr_n_defs, np.uint8), dev(p.op_vreg, np.uint32))


def _static(torch, B, p, stream=None):
    W = max(1, (p.n_vregs + 31) // 32)
    csr = _device_csr(torch, p)
    live_in = torch.full((p.n_blocks, W), -1, dtype=torch.int32, device="cuda")     # poisoned outputs
    live_out = torch.full((p.n_blocks, W), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    # free device memory as the driver sees it (torch's own counters would not notice a cudaMalloc
    # made by the library); the first call on the device, which looks up the array's address and may
    # load the module, is made by the caller before this is relied on
    free_before = torch.cuda.mem_get_info()[0]
    rc = B.vl_block_liveness_static(p.n_blocks, p.n_vregs, *csr, live_in, live_out, stream=stream)
    free_after = torch.cuda.mem_get_info()[0]
    return rc, live_in.cpu().numpy().view(np.uint32), live_out.cpu().numpy().view(np.uint32), free_before - free_after


def _regular(B, p):
    gp = B.Program(p)
    gp.vl_liveness()
    bin_, bout, _, _ = gp.vl_liveness_result()
    gp.close()
    return bin_, bout


def test_static_block_liveness_matches_regular_on_calls_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2506_17506_b200 import binding as B
    import oracle
    oracle.build()
    progs = [synth.build_program(synth.shape_attention(), 2), synth.build_program(synth.shape_gemm(), 1),
             synth.build_program(synth.shape_stress(8000, 2500), 4), synth.build_program(synth.shape_tiny(), 0)]
    side = torch.cuda.Stream()
    # same program twice in a row, then others: stale scratch contents must never leak into a result
    for n, p in enumerate([progs[0], progs[0], progs[1], progs[2], progs[3], progs[0]]):
        rc, lin, lout, grew = _static(torch, B, p, stream=side if n % 2 else None)
        assert rc == B.VL_OK
        if n > 0:                                  # (call 0 may load the module and looks up the array)
            assert grew == 0, f"the call took {grew} bytes of device memory"
        want_in, want_out = _regular(B, p)
        assert np.array_equal(lin, want_in)
        assert np.array_equal(lout, want_out)
        lv = oracle.OracleProgram(p).liveness()    # and the oracle's sets, independently of the CUDA path
        assert np.array_equal(lin, lv.packed("in"))
        assert np.array_equal(lout, lv.packed("out"))


def test_static_block_liveness_reports_bad_indices():
    """An operand that names no vreg and a successor that names no block are skipped on the device
    (nothing is read or written out of bounds) and reported."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2506_17506_b200 import binding as B
    p = synth.build_program(synth.shape_tiny(), 0)
    W = max(1, (p.n_vregs + 31) // 32)
    out = [torch.zeros((p.n_blocks, W), dtype=torch.int32, device="cuda") for _ in range(2)]
    csr = list(_device_csr(torch, p))
    bad_ops = csr[5].clone()
    bad_ops[3] = p.n_vregs + 7
    assert B.vl_block_liveness_static(p.n_blocks, p.n_vregs, *csr[:5], bad_ops, *out) == B.VL_ERR_MALFORMED_PROGRAM
    q = synth.build_program(synth.shape_gemm(), 1)
    Wq = max(1, (q.n_vregs + 31) // 32)
    outq = [torch.zeros((q.n_blocks, Wq), dtype=torch.int32, device="cuda") for _ in range(2)]
    csrq = list(_device_csr(torch, q))
    bad_succ = csrq[2].clone()
    bad_succ[0] = q.n_blocks + 3
    assert B.vl_block_liveness_static(q.n_blocks, q.n_vregs, csrq[0], csrq[1], bad_succ, *csrq[3:], *outq) == B.VL_ERR_MALFORMED_PROGRAM
    assert B.vl_block_liveness_static(q.n_blocks, q.n_vregs, *csrq, *outq) == B.VL_OK


def test_static_block_liveness_refuses_what_does_not_fit():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2506_17506_b200 import binding as B
    p = synth.build_program(synth.shape_tiny(), 0)
    W = 2048                                    # 65535 vregs -> 2048 words per row
    n_blocks = B.VL_STATIC_SCRATCH_WORDS // (2 * W) + 1
    dummy = torch.zeros(8, dtype=torch.int32, device="cuda")
    rc = B.vl_block_liveness_static(n_blocks, 65535, dummy, dummy, dummy, dummy, dummy, dummy, dummy, dummy)
    assert rc == B.VL_ERR_UNSUPPORTED
    assert B.vl_block_liveness_static(0, p.n_vregs, dummy, dummy, dummy, dummy, dummy, dummy, dummy, dummy) == B.VL_ERR_INVALID_ARG
