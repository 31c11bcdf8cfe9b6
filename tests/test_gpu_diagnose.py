"""Per-candidate diagnostics (conflict records, violation kinds per instruction, bank histogram):
CUDA path against the CPU oracle.  The records come in no particular order: compared as sorted lists."""
import numpy as np
import pytest

from paper_2506_17506_b200 import synth
from tests import helpers as H
from tests.test_gpu_parity import _garbage_rows, _to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2506_17506_b200 import binding
    return binding


def _sorted(tr):
    tr = np.asarray(tr, dtype=np.uint32).reshape(-1, 3)
    return tr[np.lexsort((tr[:, 2], tr[:, 1], tr[:, 0]))]


def _check_row(B, gp, op, lv, p, row, cap=1 << 16):
    want_tr = op.conflicts(lv, row)
    got_tr, n, kinds, hist = gp.vl_diagnose(_to_dev(row[None, :])[0], cap=cap, n_banks=p.B)
    assert n == len(want_tr)
    if n <= cap:
        assert np.array_equal(_sorted(got_tr), _sorted(want_tr))
    else:                                   # a subset of the right size, every record a true one
        assert len(got_tr) == cap
        true = {tuple(t) for t in want_tr.tolist()}
        assert all(tuple(t) in true for t in got_tr.tolist())
    assert np.array_equal(kinds, op.violations(lv, row))
    assert np.array_equal(hist, op.bank_histogram(lv, row))
    # and the diagnostics add up to what vl_verify says about the same row
    vd = B.verdicts_to_numpy(gp.vl_verify(_to_dev(row[None, :])))[0]
    assert n == vd["conflict_pairs"] and int(hist.sum()) == vd["bank_conflicts"]
    bad = np.flatnonzero(kinds)
    assert vd["first_violation_instr"] == (int(bad[0]) if len(bad) else -1)
    assert int(np.bitwise_or.reduce(kinds)) == (0 if vd["flags"] == B.VL_PASS else int(vd["flags"]))


@pytest.mark.parametrize("seed", range(16))
def test_random_small_programs(B, oracle_mod, seed):
    p = H.random_program(9000 + seed, strict=True, reachable=(seed % 4 != 0), max_instrs=60, max_vregs=20,
                         P=[8, 16, 33, 64][seed % 4], widths=(1, 1, 2, 2, 4, 8) if seed % 2 else (1, 2, 3, 5),
                         B=[4, 4, 2, 1, 3, 8][seed % 6])
    gp = B.Program(p)
    gp.vl_liveness()
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    rows = _garbage_rows(p, 18, seed)
    for k, row in enumerate(rows):
        _check_row(B, gp, op, lv, p, row, cap=5 if k % 3 == 0 else 1 << 16)
    if seed % 2:                             # with hardware rules on both sides
        rules = dict(vreg_align=np.where(p.vreg_width > 1, 2, 1), reserved=[p.P - 1])
        op.set_constraints(**rules)
        gp.set_constraints(P=p.P, **rules)
        for row in rows[:6]:
            _check_row(B, gp, op, lv, p, row)
    gp.close()


def test_attention_workload_rows(B, oracle_mod):
    """Rows of the attention-shaped workload (8,000 instructions, lists of hundreds of vregs): a valid
    row, one row of every fault kind, and the all-zero row (every live pair collides)."""
    wl = synth.workload(2)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, faults = synth.candidate_rows(p, 200, 0.5, wl.seeds[0])
    gp = B.Program(p)
    gp.vl_liveness()
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    picked = [int(np.flatnonzero(faults[:, 0] == kind)[0]) for kind in sorted(set(faults[:, 0].tolist()))]
    assert len(picked) >= 3
    for k in picked:
        _check_row(B, gp, op, lv, p, rows[k])
    zero = np.zeros(p.pitch, dtype=np.uint16)
    want = op.verify(lv, zero)[0]
    got_tr, n, kinds, hist = gp.vl_diagnose(_to_dev(zero[None, :])[0], cap=1000, n_banks=p.B)
    assert n == want["conflict_pairs"] and n > 100_000 and len(got_tr) == 1000
    assert np.array_equal(kinds, op.violations(lv, zero))
    assert np.array_equal(hist, op.bank_histogram(lv, zero))
    gp.close()


@pytest.mark.parametrize("seed", range(12))
def test_occupied_masks_random_small_programs(B, oracle_mod, seed):
    rng = np.random.default_rng(6100 + seed)
    p = H.random_program(9700 + seed, strict=True, reachable=(seed % 4 != 0), max_instrs=60, max_vregs=20,
                         P=[8, 16, 33, 64, 100][seed % 5], widths=(1, 1, 2, 2, 4, 8) if seed % 2 else (1, 2, 3, 5))
    gp = B.Program(p)
    gp.vl_liveness()
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    if seed % 3 == 0:
        reserved = sorted(set(rng.integers(0, p.P, size=3).tolist()))
        op.set_constraints(reserved=reserved)
        gp.set_constraints(P=p.P, reserved=reserved)
    rows = _garbage_rows(p, 12, seed)
    partial = H.row_from_table(p, np.where(rng.random(p.n_vregs) < 0.5, 0xFFFF, rng.integers(0, p.P, size=p.n_vregs)))
    for row in list(rows) + [partial]:
        got = gp.vl_occupied_masks(_to_dev(row[None, :])[0], p.P)
        assert np.array_equal(got, op.occupied(lv, row))
    gp.close()


def test_occupied_masks_attention_workload(B, oracle_mod):
    wl = synth.workload(2)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, _ = synth.candidate_rows(p, 4, 0.0, wl.seeds[0])
    gp = B.Program(p)
    gp.vl_liveness()
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    rng = np.random.default_rng(5)
    T = rows[1, np.array([int(np.flatnonzero(p.op_vreg == v)[0]) if (p.op_vreg == v).any() else 0 for v in range(p.n_vregs)])]
    T = np.where(rng.random(p.n_vregs) < 0.3, 0xFFFF, T)            # a third of the vregs not assigned yet
    for row in (rows[0], H.row_from_table(p, T)):
        got = gp.vl_occupied_masks(_to_dev(row[None, :])[0], p.P)
        want = op.occupied(lv, row)
        assert np.array_equal(got, want)
        assert want.sum() > 100_000                                  # hundreds of registers busy at most points
    gp.close()


def test_stress_program_rows(B, oracle_mod):
    """The largest program (32,000 instructions, 10,000 vregs, P = 512): a valid and a faulted row through
    both calls, element by element against the oracle."""
    wl = synth.workload(4)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, faults = synth.candidate_rows(p, wl.K, 0.5, wl.seeds[0], 0, 8)
    gp = B.Program(p)
    gp.vl_liveness()
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    kinds_seen = set()
    for k in range(8):
        if int(faults[k, 0]) in kinds_seen:
            continue
        kinds_seen.add(int(faults[k, 0]))
        _check_row(B, gp, op, lv, p, rows[k])
        got = gp.vl_occupied_masks(_to_dev(rows[k][None, :])[0], p.P)
        assert np.array_equal(got, op.occupied(lv, rows[k]))
    assert len(kinds_seen) >= 2
    gp.close()
