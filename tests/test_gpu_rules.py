"""Hardware rules of the Realizability check (alignment, register classes, reserved registers):
CUDA path against the CPU oracle, every verdict field, bit-exact."""
import numpy as np
import pytest

from paper_2506_17506_b200 import synth
from tests import helpers as H
from tests.test_gpu_parity import _assert_same, _garbage_rows, _gpu_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2506_17506_b200 import binding
    return binding


def _random_rules(rng, p):
    V, P = p.n_vregs, p.P
    rules = {}
    if rng.random() < 0.8:
        rules["vreg_align"] = rng.choice([1, 1, 2, 3, 4, 8], size=V)
    if rng.random() < 0.7:
        n = int(rng.integers(1, 5))
        cuts = np.sort(rng.integers(0, P + 1, size=2 * n)).reshape(n, 2)
        if rng.random() < 0.5:
            cuts[0] = (0, P)
        rules["vreg_class"] = rng.integers(0, n, size=V)
        rules["class_ranges"] = [(int(a), int(b)) for a, b in cuts]
    if rng.random() < 0.7:
        rules["reserved"] = sorted(set(rng.integers(0, P, size=int(rng.integers(0, 6))).tolist()))
    return rules


@pytest.mark.parametrize("seed", range(24))
def test_random_small_programs_with_rules(B, oracle_mod, seed):
    rng = np.random.default_rng(31000 + seed)
    p = H.random_program(6000 + seed, strict=True, reachable=(seed % 4 != 0), max_instrs=60, max_vregs=20,
                         P=[8, 16, 33, 64][seed % 4], widths=(1, 1, 2, 2, 4, 8) if seed % 2 else (1, 2, 3, 5),
                         B=[4, 4, 2, 1, 3, 8][seed % 6])
    gp = B.Program(p)
    gp.vl_liveness()
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    rows = _garbage_rows(p, 48, seed)
    plain = op.verify(lv, rows)
    seen_extra = 0
    for trial in range(3):
        rules = _random_rules(rng, p)
        op.set_constraints(**rules)
        gp.set_constraints(P=p.P, **rules)
        want = op.verify(lv, rows)
        seen_extra += int((want["flags"] != plain["flags"]).sum())
        for G in (0, 1, 2, 4, 8):
            gp.set_option(B.VL_OPT_GROUP, G)
            _assert_same(_gpu_verify(B, gp, rows), want, f"seed {seed} trial {trial} G {G} rules {sorted(rules)}")
    # rules cleared: the plain check again
    gp.set_constraints()
    _assert_same(_gpu_verify(B, gp, rows), plain, f"seed {seed} cleared")
    gp.close()


def test_gemm_workload_with_rules(B, oracle_mod):
    """The GEMM-shaped workload: its valid rows keep every tuple on a multiple of its width, so
    alignment = width changes nothing for them; reserved registers and classes fail the rows that
    use them; every field must match the oracle either way."""
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, faults = synth.candidate_rows(p, wl.K, wl.fault_rate, wl.seeds[0])
    rows = np.concatenate([rows, _garbage_rows(p, 24, 5)])
    gp = B.Program(p)
    gp.vl_liveness()
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    plain = op.verify(lv, rows)
    width = p.vreg_width.astype(np.int64)
    cases = [
        dict(vreg_align=width),
        dict(vreg_align=np.where(width == 1, 2, width)),
        dict(reserved=[0, 1, 100, 255]),
        dict(vreg_class=(width > 1).astype(np.int64), class_ranges=[(0, p.P), (0, p.P // 2)]),
        dict(vreg_align=width, vreg_class=np.arange(p.n_vregs) % 3,
             class_ranges=[(0, p.P), (8, p.P), (0, p.P - 8)], reserved=list(range(248, 256))),
    ]
    changed = []
    for j, rules in enumerate(cases):
        op.set_constraints(**rules)
        gp.set_constraints(P=p.P, **rules)
        want = op.verify(lv, rows)
        _assert_same(_gpu_verify(B, gp, rows), want, f"case {j}")
        host = gp.vl_verify_host(rows)
        _assert_same(host, want, f"case {j} host path")
        changed.append(int((want["flags"] != plain["flags"]).sum()))
    valid = np.flatnonzero(faults[:, 0] == 0)
    op.set_constraints(vreg_align=width)
    assert (op.verify(lv, rows[valid])["flags"] == 1).all()          # alignment = width keeps the valid rows valid
    assert changed[0] >= 0 and min(changed[1:]) > 0                   # the other rules do fail rows
    gp.close()


def test_rule_arguments_are_checked(B):
    p = synth.program_from_lists([[([0], []), ([1], [0]), ([], [1, 0])]], [], 2, [1, 2], 8)
    gp = B.Program(p)
    with pytest.raises(B.VlError):
        gp.set_constraints(vreg_align=[0, 1])                                   # alignment 0
    with pytest.raises(B.VlError):
        gp.set_constraints(vreg_class=[0, 2], class_ranges=[(0, 8), (0, 4)])    # class id out of range
    with pytest.raises(B.VlError):
        gp.set_constraints(vreg_class=[0, 1], class_ranges=[(0, 8), (5, 4)])    # empty-reversed range
    with pytest.raises(B.VlError):
        gp.set_constraints(vreg_class=[0, 1], class_ranges=[(0, 8), (0, 9)])    # beyond the file
    with pytest.raises(B.VlError):
        gp.set_constraints(vreg_class=[0, 0], class_ranges=[(0, 8)] * 9)        # too many classes
    gp.set_constraints(vreg_class=[0, 1], class_ranges=[(0, 8), (4, 4)])        # an empty class is allowed
    gp.close()
