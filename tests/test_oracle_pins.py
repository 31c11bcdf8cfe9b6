"""Pins for the CPU oracle: what the paper and the mathematics fix, checked against
brute force, closed forms and hand-worked programs (no GPU)."""
import os

import numpy as np
import pytest

from paper_2506_17506_b200 import synth
from tests import helpers as H

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
PASS, INCONS, RANGE, INTERF = 1, 2, 4, 8


def _oracle(oracle_mod, p):
    op = oracle_mod.OracleProgram(p)
    return op, op.liveness()


# ------------------------------------------------------------------ liveness pins
@pytest.mark.parametrize("seed", range(60))
def test_liveness_equals_path_definition(oracle_mod, seed):
    """Liveness is *defined* by paths; the fixed point must reproduce it exactly,
    on strict and non-strict programs, with loops and unreachable blocks."""
    p = H.random_program(seed, strict=(seed % 2 == 0), reachable=(seed % 3 != 0))
    op, lv = _oracle(oracle_mod, p)
    live_after, blk_in, blk_out = H.path_liveness(p)
    for i in range(p.n_instrs):
        assert list(lv.live_after(i)) == live_after[i], f"instr {i}"
    assert np.array_equal(lv.blk_live_in, blk_in)
    assert np.array_equal(lv.blk_live_out, blk_out)


def test_liveness_closed_form_single_block(oracle_mod):
    """One block: v is live after i iff the next event on v after i is a read."""
    p = synth.build_program(synth.shape_tiny(), 0)
    op, lv = _oracle(oracle_mod, p)
    ins, _, _ = H.instr_lists(p)
    for i in range(p.n_instrs):
        expect = []
        for v in range(p.n_vregs):
            for j in range(i + 1, p.n_instrs):
                d, u = ins[j]
                if v in u:
                    expect.append(v)
                    break
                if v in d:
                    break
        assert list(lv.live_after(i)) == expect


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_liveness_fixed_point_equations_and_sweep_order(oracle_mod, idx):
    wl = synth.workload(idx)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    op = oracle_mod.OracleProgram(p)
    a, b = op.liveness(order=0), op.liveness(order=1)
    assert np.array_equal(a.blk_live_in, b.blk_live_in) and np.array_equal(a.blk_live_out, b.blk_live_out)
    assert np.array_equal(a.lo_off, b.lo_off) and np.array_equal(a.lo, b.lo)
    ins, blk, succ = H.instr_lists(p)
    for bb in range(p.n_blocks):
        out = np.zeros(p.n_vregs, dtype=np.uint8)
        for s in succ[bb]:
            out |= a.blk_live_in[s]
        assert np.array_equal(out, a.blk_live_out[bb])
    assert a.blk_live_in[0].sum() == 0          # the generator's programs are strict
    # lists ascending, no duplicates
    for i in range(0, p.n_instrs, max(1, p.n_instrs // 50)):
        l = a.live_after(i)
        assert np.all(np.diff(l.astype(np.int64)) > 0)


# -------------------------------------------------------------- interference pins
@pytest.mark.parametrize("seed", range(80))
def test_def_point_rule_equals_all_pairs_definition(oracle_mod, seed):
    """Strict programs with every block reachable: the set of vreg pairs that overlap
    at a definition point equals the set of pairs that are ever live together with
    intersecting ranges; so the interference flag is the all-pairs decision."""
    p = H.random_program(1000 + seed, strict=True, reachable=True, P=12)
    op, lv = _oracle(oracle_mod, p)
    live_after, _, _ = H.path_liveness(p)
    rng = np.random.default_rng(seed)
    for trial in range(6):
        T = rng.integers(0, p.P, size=p.n_vregs)
        if trial == 0:
            T[:] = 0
        row = H.row_from_table(p, T)
        tr = op.conflicts(lv, row)
        dedup = {(min(int(v), int(u)), max(int(v), int(u))) for _, v, u in tr}
        brute = H.copointed_overlapping_pairs(p, live_after, row)
        assert dedup == brute
        vd = op.verify(lv, row)[0]
        assert bool(vd["flags"] & INTERF) == bool(brute)
        assert vd["conflict_pairs"] == len(tr)
        # each triple is a real overlap at a definition of v with u live after or co-defined
        ins, _, _ = H.instr_lists(p)
        w = p.vreg_width
        for i, v, u in tr:
            assert v in ins[i][0] and v != u
            assert (u in live_after[i]) or (u in ins[i][0])
            assert H.overlap(int(T[v]), int(w[v]), int(T[u]), int(w[u]))


@pytest.mark.parametrize("seed", range(20))
def test_conflict_count_closed_form_all_zero_candidate(oracle_mod, seed):
    """All widths 1 and every vreg on register 0: every pair overlaps, so the count is
    sum over definitions of |(live_after(i) | defs(i)) - {v}|, a function of liveness only."""
    p = H.random_program(2000 + seed, strict=True, reachable=(seed % 2 == 0), widths=(1,))
    op, lv = _oracle(oracle_mod, p)
    live_after, _, _ = H.path_liveness(p)
    ins, _, _ = H.instr_lists(p)
    expect = sum(len((set(live_after[i]) | set(d)) - {v}) for i, (d, _) in enumerate(ins) for v in d)
    vd = op.verify(lv, np.zeros(p.pitch, dtype=np.uint16))[0]
    assert vd["conflict_pairs"] == expect
    assert bool(vd["flags"] & INTERF) == (expect > 0)
    assert not vd["flags"] & (INCONS | RANGE)


def test_sequential_no_reuse_assignment(oracle_mod):
    """Appendix B's pattern (a fresh register for every vreg, no reuse) can never
    interfere; it is valid iff it fits in the register file, otherwise the first
    violation is the lowest-index definition of a vreg that sticks out."""
    shape = synth.shape_gemm()
    p = synth.build_program(shape, 1)
    w = p.vreg_width.astype(np.int64)
    T = np.concatenate([[0], np.cumsum(w)[:-1]])
    total = int(w.sum())
    row = H.row_from_table(p, T)
    for P in (total, total - 1, 256):
        q = synth.Program(**{**p.__dict__, "P": P})
        op, lv = _oracle(oracle_mod, q)
        vd = op.verify(lv, row)[0]
        assert vd["conflict_pairs"] == 0 and not vd["flags"] & (INTERF | INCONS)
        if total <= P:
            assert vd["flags"] == PASS and vd["first_violation_instr"] == -1
        else:
            assert vd["flags"] == RANGE
            sticking = np.nonzero(T + w > P)[0]
            assert vd["first_violation_instr"] == int(p.gen["first_def_instr"][sticking].min())


# ------------------------------------------------------------------ bank pins
def _bank_case(oracle_mod, regs, B=4, P=16):
    n = len(regs)
    blocks = [[([v], []) for v in range(n)] + [([n], list(range(n)))]]
    p = synth.program_from_lists(blocks, [], n + 1, [1] * (n + 1), P, B)
    # sources sit on `regs`; the result goes to a register none of them uses
    free = [r for r in range(P) if r not in regs][0]
    tab = list(regs) + [free]
    # repeated registers among the sources would interfere at their definitions; the bank
    # tally is defined regardless, which is what is checked here
    op, lv = _oracle(oracle_mod, p)
    return op.verify(lv, H.row_from_table(p, tab))[0]


def test_bank_tally_paper_example_and_hand_cases(oracle_mod):
    # Section 2: 4 banks; the FFMA of Figure 1 reads R4, R6, R9, which sit in separate banks.
    with open(os.path.join(GOLDEN, "ffma_banks.txt")) as f:
        lines = [l.split("#")[0].split() for l in f if l.strip() and not l.startswith("#")]
    for toks in lines:
        B, expect, regs = int(toks[0]), int(toks[1]), [int(t) for t in toks[2:]]
        assert _bank_case(oracle_mod, regs, B=B)["bank_conflicts"] == expect, toks
    assert _bank_case(oracle_mod, [4, 8])["bank_conflicts"] == 1
    assert _bank_case(oracle_mod, [4, 8, 12])["bank_conflicts"] == 2
    assert _bank_case(oracle_mod, [4, 4, 8])["bank_conflicts"] == 1     # same register read twice counts once
    assert _bank_case(oracle_mod, [5])["bank_conflicts"] == 0
    assert _bank_case(oracle_mod, [0, 1, 2, 3])["bank_conflicts"] == 0
    assert _bank_case(oracle_mod, [0, 4, 1, 5])["bank_conflicts"] == 2
    assert _bank_case(oracle_mod, [0, 4, 1, 5], B=1)["bank_conflicts"] == 3
    assert _bank_case(oracle_mod, [1, 4, 7, 10], B=3)["bank_conflicts"] == 3


# ------------------------------------------------------------ hand-built programs
def test_hand_straight_line_with_reuse(oracle_mod):
    #  i0: v0=       i1: v1=      i2: v2=f(v0,v1)     i3: v3=f(v2)     i4: =f(v3) (no def)
    p = synth.program_from_lists([[([0], []), ([1], []), ([2], [0, 1]), ([3], [2]), ([], [3])]], [], 4, [1, 1, 1, 1], 2)
    op, lv = _oracle(oracle_mod, p)
    assert [list(lv.live_after(i)) for i in range(5)] == [[0], [0, 1], [2], [3], []]
    ok = op.verify(lv, H.row_from_table(p, [0, 1, 0, 0]))[0]      # v2 reuses v0's register at its last use
    assert tuple(ok) == (PASS, -1, 0, 0)
    bad = op.verify(lv, H.row_from_table(p, [0, 0, 1, 0]))[0]     # v1 clobbers v0 while v0 is live
    assert bad["flags"] == INTERF and bad["first_violation_instr"] == 1 and bad["conflict_pairs"] == 1
    # bank tally of the bad row: i2 reads v0 and v1, same register -> one distinct source
    assert bad["bank_conflicts"] == 0


def test_hand_diamond_and_dead_def(oracle_mod):
    # b0: v0= ; v1=       b1: v2=f(v0)      b2: v2=f(v1) ; v3= (dead)     b3: =f(v2)
    blocks = [[([0], []), ([1], [])], [([2], [0])], [([2], [1]), ([3], [])], [([], [2])]]
    p = synth.program_from_lists(blocks, [(0, 1), (0, 2), (1, 3), (2, 3)], 4, [1, 1, 1, 1], 3)
    op, lv = _oracle(oracle_mod, p)
    assert [list(lv.live_after(i)) for i in range(6)] == [[0], [0, 1], [2], [2], [2], []]
    assert tuple(op.verify(lv, H.row_from_table(p, [0, 1, 0, 1]))[0]) == (PASS, -1, 0, 0)
    # the dead def of v3 at instr 4 clobbers v2 (live after it): interference at its own instruction
    vd = op.verify(lv, H.row_from_table(p, [0, 1, 2, 2]))[0]
    assert vd["flags"] == INTERF and vd["first_violation_instr"] == 4 and vd["conflict_pairs"] == 1
    # v2 on v1's register: b1 defines v2 while v1 is dead there, b2 reads v1 at the same instruction -> legal
    assert op.verify(lv, H.row_from_table(p, [0, 1, 1, 0]))[0]["flags"] == PASS
    # v2 on v0's register: in b2 v0 is dead as well -> legal
    assert op.verify(lv, H.row_from_table(p, [0, 1, 0, 2]))[0]["flags"] == PASS


def test_hand_loop_carried_and_self_update(oracle_mod):
    # b0: acc= ; x=      b1 (self loop): t=f(x) ; acc=f(acc,t)       b2: =f(acc)
    blocks = [[([0], []), ([1], [])], [([2], [1]), ([0], [0, 2])], [([], [0])]]
    p = synth.program_from_lists(blocks, [(0, 1), (1, 1), (1, 2)], 3, [2, 1, 1], 4)
    op, lv = _oracle(oracle_mod, p)
    assert [list(lv.live_after(i)) for i in range(5)] == [[0], [0, 1], [0, 1, 2], [0, 1], []]
    assert lv.blk_live_in.tolist() == [[0, 0, 0], [1, 1, 0], [1, 0, 0]]
    assert lv.blk_live_out.tolist() == [[1, 1, 0], [1, 1, 0], [0, 0, 0]]
    assert op.verify(lv, H.row_from_table(p, [0, 2, 3]))[0]["flags"] == PASS       # acc = {0,1}
    # t on x's register: x is loop-invariant and live around the back edge
    vd = op.verify(lv, H.row_from_table(p, [0, 2, 2]))[0]
    assert vd["flags"] == INTERF and vd["first_violation_instr"] == 2 and vd["conflict_pairs"] == 1
    # x inside the accumulator pair (register 1): seen at x's def (acc live) and at every def of acc
    vd = op.verify(lv, H.row_from_table(p, [0, 1, 3]))[0]
    assert vd["flags"] == INTERF and vd["first_violation_instr"] == 1 and vd["conflict_pairs"] == 2
    # pair sticking out of a 4-register file
    vd = op.verify(lv, H.row_from_table(p, [3, 0, 1]))[0]
    assert vd["flags"] == RANGE and vd["first_violation_instr"] == 0 and vd["conflict_pairs"] == 0


def test_hand_nested_loops(oracle_mod):
    # b0: a= ; b=   b1(outer head): c=f(a)   b2(inner, self): d=f(c,b)   b3(latch -> b1): a=f(a,c)   b4: =f(a)
    blocks = [[([0], []), ([1], [])], [([2], [0])], [([3], [2, 1])], [([0], [0, 2])], [([], [0])]]
    edges = [(0, 1), (1, 2), (2, 2), (2, 3), (3, 1), (3, 4)]
    p = synth.program_from_lists(blocks, edges, 4, [1, 1, 1, 1], 4)
    op, lv = _oracle(oracle_mod, p)
    assert [list(lv.live_after(i)) for i in range(6)] == [[0], [0, 1], [0, 1, 2], [0, 1, 2], [0, 1], []]
    assert op.verify(lv, H.row_from_table(p, [0, 1, 2, 3]))[0]["flags"] == PASS
    # d is dead (never read) but is written while a, b, c are live
    vd = op.verify(lv, H.row_from_table(p, [0, 1, 2, 1]))[0]
    assert vd["flags"] == INTERF and vd["first_violation_instr"] == 3


def test_hand_wide_tuples_contiguity(oracle_mod):
    """Section 2 / Section 4.5: a 64-bit value takes two consecutive registers
    (vgpr0_vgpr1); anything placed on either of them while it is live collides."""
    blocks = [[([0], []), ([1], []), ([], [0, 1])]]
    p = synth.program_from_lists(blocks, [], 2, [2, 1], 8)
    op, lv = _oracle(oracle_mod, p)
    assert op.verify(lv, H.row_from_table(p, [0, 2]))[0]["flags"] == PASS
    for clash in (0, 1):
        vd = op.verify(lv, H.row_from_table(p, [0, clash]))[0]
        assert vd["flags"] == INTERF and vd["first_violation_instr"] == 1
    assert op.verify(lv, H.row_from_table(p, [7, 0]))[0]["flags"] == RANGE     # {7,8} leaves an 8-register file
    assert op.verify(lv, H.row_from_table(p, [6, 0]))[0]["flags"] == PASS


def test_hand_multi_def_instruction_and_inconsistency(oracle_mod):
    # i0: (v0,v1)=     i1: v2=f(v0)     i2: =f(v1,v2)
    p = synth.program_from_lists([[([0, 1], []), ([2], [0]), ([], [1, 2])]], [], 3, [1, 1, 1], 4)
    op, lv = _oracle(oracle_mod, p)
    assert [list(lv.live_after(i)) for i in range(3)] == [[0, 1], [1, 2], []]
    # both results of i0 on one register: counted once from each side
    vd = op.verify(lv, H.row_from_table(p, [0, 0, 1]))[0]
    assert vd["flags"] == INTERF and vd["first_violation_instr"] == 0 and vd["conflict_pairs"] == 2
    # inconsistent occurrence: v0 is R0 at its definition and R3 at its read; the table keeps R0
    row = H.row_from_table(p, [0, 1, 2])
    row[3] = 3
    vd = op.verify(lv, row)[0]
    assert vd["flags"] == INCONS and vd["first_violation_instr"] == 1 and vd["conflict_pairs"] == 0
    # values beyond the file are compared as plain integers (no wrap)
    vd = op.verify(lv, H.row_from_table(p, [65535, 65535, 0]))[0]
    assert vd["flags"] == (RANGE | INTERF) and vd["conflict_pairs"] == 2


def test_hand_unreachable_block_and_dead_code(oracle_mod):
    # b0: v0= ; =f(v0)      b1 (unreachable): v1=f(v0)   -- v0 is not live into b0 (defined first)
    blocks = [[([0], []), ([], [0])], [([1], [0])]]
    p = synth.program_from_lists(blocks, [], 2, [1, 1], 2)
    op, lv = _oracle(oracle_mod, p)
    assert lv.blk_live_in.tolist() == [[0, 0], [1, 0]]
    assert [list(lv.live_after(i)) for i in range(3)] == [[0], [], []]
    assert op.verify(lv, H.row_from_table(p, [0, 0]))[0]["flags"] == PASS   # v1 may take v0's register: v0 dies at its read


# ----------------------------------------------------------- generator-based pins
@pytest.mark.parametrize("idx", [0, 1, 2])
def test_generator_valid_rows_pass_and_faults_fail_where_injected(oracle_mod, idx):
    wl = synth.workload(idx)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    K = min(wl.K, 150)
    rows, faults = synth.candidate_rows(p, wl.K, wl.fault_rate, wl.seeds[0], 0, K)
    clean, _ = synth.candidate_rows(p, wl.K, 0.0, wl.seeds[0], 0, K)
    op, lv = _oracle(oracle_mod, p)
    vd = op.verify(lv, rows)
    vc = op.verify(lv, clean)
    assert np.all(vc["flags"] == PASS) and np.all(vc["first_violation_instr"] == -1) and np.all(vc["conflict_pairs"] == 0)
    kinds = faults[:, 0]
    assert (kinds != 0).sum() > 0
    for k in range(K):
        kind, instr, v, u, o = [int(x) for x in faults[k]]
        if kind == synth.FAULT_NONE:
            assert tuple(vd[k]) == tuple(vc[k])
        elif kind == synth.FAULT_INCONSISTENT:
            # only the consistency bit; everything derived from the table is unchanged
            assert vd[k]["flags"] == INCONS and vd[k]["first_violation_instr"] == instr
            assert vd[k]["conflict_pairs"] == 0 and vd[k]["bank_conflicts"] == vc[k]["bank_conflicts"]
        elif kind == synth.FAULT_RANGE:
            assert vd[k]["flags"] == RANGE and vd[k]["first_violation_instr"] == instr
            assert vd[k]["conflict_pairs"] == 0
        else:
            assert vd[k]["flags"] & INTERF and not vd[k]["flags"] & INCONS
            assert 0 <= vd[k]["first_violation_instr"] <= instr
            assert op.violations(lv, rows[k])[instr] & INTERF
            tr = op.conflicts(lv, rows[k])
            assert any((int(a), int(b), int(c)) == (instr, v, u) for a, b, c in tr)


def test_generator_batch_members_and_stress_sample(oracle_mod):
    wl = synth.workload(3)
    for j in (0, 17, 255):
        p = synth.build_program(wl.shapes[j], wl.seeds[j])
        rows, faults = synth.candidate_rows(p, wl.K, wl.fault_rate, wl.seeds[j], 0, 40)
        op, lv = _oracle(oracle_mod, p)
        vd = op.verify(lv, rows)
        assert np.array_equal(vd["flags"] == PASS, faults[:, 0] == 0)
    wl = synth.workload(4)
    p = synth.build_program(synth.shape_stress(8000, 2500), 4)
    rows, faults = synth.candidate_rows(p, 64, 0.25, 4)
    op, lv = _oracle(oracle_mod, p)
    vd = op.verify(lv, rows)
    assert np.array_equal(vd["flags"] == PASS, faults[:, 0] == 0)


# ------------------------------------------------------- re-sampling statistics
def _verdicts(oracle_mod, pass_rows, K):
    v = np.zeros(K, dtype=oracle_mod.VERDICT_DTYPE)
    v["flags"] = INTERF
    v["first_violation_instr"] = 0
    v["flags"][list(pass_rows)] = PASS
    return v


def test_pass_rate_matches_the_paper_table(oracle_mod):
    # Table 2: one greedy attempt per test case; the printed rate is passing / all, to two decimals.
    with open(os.path.join(GOLDEN, "table2_pass_rates.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 10
    for n_pass, n_fail, printed in rows:
        n_pass, n_fail = int(n_pass), int(n_fail)
        stats = np.array([oracle_mod.sample_stats(_verdicts(oracle_mod, [0] if c < n_pass else [], 1))
                          for c in range(n_pass + n_fail)])
        s = oracle_mod.resample_summary(stats, [1] * len(stats), [1, 100])
        assert s["n_cases"] == n_pass + n_fail and s["n_solved"] == n_pass
        assert s["pass_at"] == [n_pass, n_pass]
        assert f"{100.0 * s['pass_at'][0] / s['n_cases']:.2f}" == printed
        assert (s["sum_tries"], s["max_tries"]) == (n_pass, 1 if n_pass else 0)


def test_first_passing_attempt_closed_forms(oracle_mod):
    K = 250
    # case c passes first at attempt c*c + 1 (rows are attempts in order), later rows mixed
    firsts = [c * c for c in range(15)]                     # 0, 1, 4, ..., 196
    stats = []
    for f0 in firsts:
        rows = [f0] + [r for r in range(f0 + 1, K) if (r * 7 + f0) % 5 == 0]
        st = oracle_mod.sample_stats(_verdicts(oracle_mod, rows, K))
        assert (int(st["first_pass"]), int(st["n_pass"])) == (f0, len(rows))
        stats.append(st)
    never = oracle_mod.sample_stats(_verdicts(oracle_mod, [], K))
    assert (int(never["first_pass"]), int(never["n_pass"])) == (K, 0)
    stats += [never, never]
    s = oracle_mod.resample_summary(np.array(stats), [K] * len(stats), [1, 10, 100, 197, 250])
    attempts = [f0 + 1 for f0 in firsts]
    assert s["n_cases"] == 17 and s["n_solved"] == 15
    assert s["sum_tries"] == sum(attempts) and s["max_tries"] == 197
    # attempts 1, 2, 5, 10 are within 10; squares up to 81 (+1) within 100; 197 is the last
    assert s["pass_at"] == [1, 4, 10, 15, 15]
    # Pass@k never decreases in k and ends at the solved count
    assert all(a <= b for a, b in zip(s["pass_at"], s["pass_at"][1:])) and s["pass_at"][-1] == s["n_solved"]


def test_resample_statistics_edge_cases(oracle_mod):
    empty = oracle_mod.sample_stats(np.zeros(0, dtype=oracle_mod.VERDICT_DTYPE))
    assert (int(empty["first_pass"]), int(empty["n_pass"])) == (0, 0)
    s = oracle_mod.resample_summary(np.array([empty]), [0], [1])
    assert (s["n_cases"], s["n_solved"], s["sum_tries"], s["max_tries"], s["pass_at"]) == (1, 0, 0, 0, [0])
    s = oracle_mod.resample_summary(np.zeros(0, dtype=oracle_mod.SAMPLE_STATS_DTYPE), [], [1, 10])
    assert (s["n_cases"], s["n_solved"], s["pass_at"]) == (0, 0, [0, 0])
    # a verdict that carries the pass bit together with nothing else counts; kind bits alone never do
    v = np.zeros(4, dtype=oracle_mod.VERDICT_DTYPE)
    v["flags"] = [INCONS, RANGE | INTERF, INCONS | RANGE | INTERF, PASS]
    st = oracle_mod.sample_stats(v)
    assert (int(st["first_pass"]), int(st["n_pass"])) == (3, 1)
    # statistics over real verdicts: a generated workload, rows in order
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, _faults = synth.candidate_rows(p, 100, wl.fault_rate, wl.seeds[0])
    op, live = _oracle(oracle_mod, p)
    out = op.verify(live, rows)
    passing = np.flatnonzero(out["flags"] == PASS)
    st = oracle_mod.sample_stats(out)
    assert int(st["n_pass"]) == len(passing) and int(st["first_pass"]) == (passing[0] if len(passing) else 100)


# ------------------------------------------------- hardware rules (fuller Realizability)
def _defs_then_use(widths, P):
    """v0, v1, ... defined one per instruction, all read by a last instruction (all live together)."""
    n = len(widths)
    blocks = [[([v], []) for v in range(n)] + [([], list(range(n)))]]
    return synth.program_from_lists(blocks, [], n, widths, P)


def test_hardware_rules_hand_cases(oracle_mod):
    p = _defs_then_use([2, 2, 1, 8], 32)
    op, lv = _oracle(oracle_mod, p)

    def verdict(T):
        return op.verify(lv, H.row_from_table(p, T))[0]

    base = [0, 2, 4, 8]
    assert verdict(base)["flags"] == PASS
    # alignment: pairs on even registers, the 8-tuple on a multiple of 8, singles anywhere
    op.set_constraints(vreg_align=[2, 2, 1, 8])
    assert verdict(base)["flags"] == PASS
    assert verdict([0, 2, 5, 8])["flags"] == PASS                      # width 1 may sit on an odd register
    vd = verdict([0, 3, 5, 8])                                         # pair on an odd register
    assert (vd["flags"], vd["first_violation_instr"], vd["conflict_pairs"]) == (RANGE, 1, 0)
    vd = verdict([0, 2, 4, 12])                                        # 8-tuple on 12: inside the file, misaligned
    assert (vd["flags"], vd["first_violation_instr"]) == (RANGE, 3)
    assert verdict([0, 2, 4, 24])["flags"] == PASS                     # last aligned place in the file
    # reserved registers: a tuple may sit beside one, not on one; its last register counts too
    op.set_constraints(reserved=[6, 7, 31])
    assert verdict(base)["flags"] == PASS                              # 4 and 8.. are beside 6, 7
    vd = verdict([0, 2, 6, 8])
    assert (vd["flags"], vd["first_violation_instr"]) == (RANGE, 2)
    vd = verdict([0, 5, 4, 8])                                         # pair 5..6 ends on a reserved register
    assert (vd["flags"], vd["first_violation_instr"], vd["conflict_pairs"]) == (RANGE, 1, 0)
    assert verdict([0, 2, 4, 23])["flags"] == PASS                     # 23..30 stops before 31
    assert verdict([0, 2, 4, 24])["flags"] == RANGE                    # 24..31 holds 31
    # classes: v0, v1 scalar in [0, 8); v2, v3 vector in [8, 32)
    op.set_constraints(vreg_class=[0, 0, 1, 1], class_ranges=[(0, 8), (8, 32)])
    assert verdict([0, 2, 8, 9])["flags"] == PASS
    assert verdict([0, 6, 8, 24])["flags"] == PASS                     # both classes filled to their last register
    vd = verdict([0, 7, 9, 16])                                        # scalar pair 7..8 leaves its class
    assert (vd["flags"], vd["first_violation_instr"]) == (RANGE, 1)
    vd = verdict([0, 2, 7, 16])                                        # vector single below its class
    assert (vd["flags"], vd["first_violation_instr"]) == (RANGE, 2)
    assert verdict([0, 2, 8, 25])["flags"] == RANGE                    # 25..32 beyond the class and the file
    # all rules off again: the plain range check is all that is left
    op.set_constraints()
    assert verdict([0, 3, 7, 24])["flags"] == PASS


def test_hardware_rules_hand_case_overlap_is_still_counted(oracle_mod):
    # a misplaced tuple is compared with the others where it is (no special treatment)
    p = _defs_then_use([2, 2], 16)
    op, lv = _oracle(oracle_mod, p)
    op.set_constraints(vreg_align=[2, 2], reserved=[9])
    vd = op.verify(lv, H.row_from_table(p, [4, 5]))[0]                 # v1 misaligned and on v0's second register
    assert (vd["flags"], vd["first_violation_instr"], vd["conflict_pairs"]) == (RANGE | INTERF, 1, 1)


@pytest.mark.parametrize("seed", range(12))
def test_hardware_rules_equal_register_by_register_definition(oracle_mod, seed):
    """A definition is realizable iff its base is a multiple of the alignment and every register it
    occupies exists, belongs to the vreg's class and is not reserved: enumerate registers in Python."""
    rng = np.random.default_rng(900 + seed)
    p = H.random_program(7000 + seed, strict=True, reachable=True, max_instrs=40, max_vregs=14, P=32,
                         widths=(1, 2, 2, 4))
    op, lv = _oracle(oracle_mod, p)
    V = p.n_vregs
    align = rng.choice([1, 2, 4], size=V)
    cls = rng.integers(0, 3, size=V)
    ranges = [(0, 12), (12, 32), (4, 28)]
    reserved = sorted(set(rng.integers(0, 32, size=3).tolist()))
    op.set_constraints(vreg_align=align, vreg_class=cls, class_ranges=ranges, reserved=reserved)
    first_def = {}
    for i in range(p.n_instrs):
        for o in range(p.instr_op_off[i], p.instr_op_off[i] + p.instr_n_defs[i]):
            first_def.setdefault(int(p.op_vreg[o]), i)
    plain = oracle_mod.OracleProgram(p)
    for _ in range(30):
        T = rng.integers(0, 36, size=V)
        row = H.row_from_table(p, T)
        got = op.verify(lv, row)[0]
        ref = plain.verify(lv, row)[0]                                  # same row without the rules
        bad_instrs = []
        for v, i in first_def.items():
            regs = range(int(T[v]), int(T[v]) + int(p.vreg_width[v]))
            ok = T[v] % align[v] == 0 and all(r < 32 and ranges[cls[v]][0] <= r < ranges[cls[v]][1] and r not in reserved
                                              for r in regs)
            if not ok:
                bad_instrs.append(i)
        assert bool(got["flags"] & RANGE) == bool(bad_instrs)
        assert got["conflict_pairs"] == ref["conflict_pairs"] and got["bank_conflicts"] == ref["bank_conflicts"]
        assert (got["flags"] & (INTERF | INCONS)) == (ref["flags"] & (INTERF | INCONS))
        firsts = bad_instrs + ([int(ref["first_violation_instr"])] if ref["flags"] & (INTERF | INCONS | RANGE) else [])
        assert got["first_violation_instr"] == (min(firsts) if firsts else -1)


# ------------------------------------------------------------ per-candidate diagnostics
def test_bank_histogram_hand_cases(oracle_mod):
    def hist(regs, B=4, P=16):
        n = len(regs)
        blocks = [[([v], []) for v in range(n)] + [([n], list(range(n)))]]
        p = synth.program_from_lists(blocks, [], n + 1, [1] * (n + 1), P, B)
        free = [r for r in range(P) if r not in regs][0]
        op, lv = _oracle(oracle_mod, p)
        row = H.row_from_table(p, list(regs) + [free])
        h = op.bank_histogram(lv, row)
        assert int(h.sum()) == int(op.verify(lv, row)[0]["bank_conflicts"])
        return h.tolist()

    assert hist([4, 6, 9]) == [0, 0, 0, 0]              # Section 2: R4, R6, R9 sit in separate banks
    assert hist([4, 8]) == [1, 0, 0, 0]
    assert hist([4, 8, 12, 5, 9]) == [2, 1, 0, 0]
    assert hist([3, 7, 11, 15]) == [0, 0, 0, 3]
    assert hist([4, 4, 8]) == [1, 0, 0, 0]              # the same register read twice counts once
    assert hist([1, 4, 7, 10], B=3) == [0, 3, 0]


@pytest.mark.parametrize("seed", range(10))
def test_diagnostics_agree_with_the_verdict(oracle_mod, seed):
    """Conflict records, per-instruction kinds and the bank histogram of a row add up to its verdict."""
    rng = np.random.default_rng(4100 + seed)
    p = H.random_program(8000 + seed, strict=True, reachable=True, max_instrs=50, max_vregs=16, P=24,
                         widths=(1, 2, 4), B=[4, 3, 2][seed % 3])
    op, lv = _oracle(oracle_mod, p)
    for _ in range(10):
        row = H.row_from_table(p, rng.integers(0, 28, size=p.n_vregs))
        if rng.random() < 0.5:
            row[rng.integers(0, p.n_operands)] ^= 1
        vd = op.verify(lv, row)[0]
        tr = op.conflicts(lv, row)
        kinds = op.violations(lv, row)
        assert len(tr) == vd["conflict_pairs"]
        assert int(op.bank_histogram(lv, row).sum()) == vd["bank_conflicts"]
        assert int(np.bitwise_or.reduce(kinds)) == (0 if vd["flags"] == PASS else int(vd["flags"]))
        bad = np.flatnonzero(kinds)
        assert vd["first_violation_instr"] == (int(bad[0]) if len(bad) else -1)
        assert set(np.flatnonzero(kinds & INTERF).tolist()) == set(tr[:, 0].tolist())
        for i, v, u in tr:                              # every record is a definition of v at i that overlaps u
            defs = p.op_vreg[p.instr_op_off[i]: p.instr_op_off[i] + p.instr_n_defs[i]]
            assert v in defs and u != v


# --------------------------------------------------- occupied registers at every definition point
def test_occupied_registers_hand_case(oracle_mod):
    # v0 (w2) and v1 (w1) defined, v2 defined from v0 (v0 dies), all read at the end except v0
    blocks = [[([0], []), ([1], []), ([2], [0]), ([], [1, 2])]]
    p = synth.program_from_lists(blocks, [], 3, [2, 1, 2], 8)
    op, lv = _oracle(oracle_mod, p)
    occ = op.occupied(lv, H.row_from_table(p, [4, 6, 0]))
    regs = [set(np.flatnonzero(r).tolist()) for r in occ]
    assert regs[0] == set()                 # v0 is the instruction's own definition, nothing else is live
    assert regs[1] == {4, 5}                # v0 live after the definition of v1
    assert regs[2] == {6}                   # v0 dies at its read here; v1 stays; v2 is the own definition
    assert regs[3] == set()                 # nothing is live after the last reads
    # a vreg without a register yet (entry >= P) and a tuple sticking out of the file
    occ = op.occupied(lv, H.row_from_table(p, [7, 0xFFFF, 0]))
    regs = [set(np.flatnonzero(r).tolist()) for r in occ]
    assert regs[1] == {7} and regs[2] == set()
    op.set_constraints(reserved=[3])
    occ = op.occupied(lv, H.row_from_table(p, [4, 6, 0]))
    assert set(np.flatnonzero(occ[1]).tolist()) == {3, 4, 5} and set(np.flatnonzero(occ[3]).tolist()) == {3}


@pytest.mark.parametrize("seed", range(16))
def test_occupied_registers_from_path_liveness_and_the_safety_verdict(oracle_mod, seed):
    """The mask is the union of the ranges of the vregs that the path definition of liveness finds
    live after the instruction (own definitions left out); for instructions with one definition a
    row is free of Safety violations iff no definition touches the mask of its instruction."""
    rng = np.random.default_rng(5200 + seed)
    p = H.random_program(9500 + seed, strict=True, reachable=True, max_instrs=40, max_vregs=14, P=24, widths=(1, 2, 4),
                         multi_def=(seed % 2 == 1))
    op, lv = _oracle(oracle_mod, p)
    live_after, _, _ = H.path_liveness(p)
    ins, _, _ = H.instr_lists(p)
    single = all(len(d) <= 1 for d, _ in ins)
    for _ in range(12):
        T = rng.integers(0, 26, size=p.n_vregs)
        row = H.row_from_table(p, T)
        occ = op.occupied(lv, row)
        clash = False
        for i, (defs, _) in enumerate(ins):
            want = set()
            for u in live_after[i]:
                if u not in defs:
                    want |= {r for r in range(int(T[u]), int(T[u]) + int(p.vreg_width[u])) if r < p.P}
            assert set(np.flatnonzero(occ[i]).tolist()) == want, f"instr {i}"
            for v in defs:
                clash = clash or any(r in want for r in range(int(T[v]), int(T[v]) + int(p.vreg_width[v])))
        if single:
            assert clash == bool(op.verify(lv, row)[0]["flags"] & INTERF)
    assert single == (seed % 2 == 0)


# ---------------------------------------------------------------- dictionary candidates
def _expand_dict_row(p, drow):
    """Per-occurrence row that a dictionary row stands for, by plain loops (independent of the oracle's
    own expansion): every occurrence of v in block b takes the entry of (b, v); entries are laid out
    block by block, a block's vregs in the order they first occur."""
    row = np.zeros(p.pitch, dtype=np.uint16)
    e = 0
    for b in range(p.n_blocks):
        slot = {}
        i0, i1 = int(p.block_instr_off[b]), int(p.block_instr_off[b + 1])
        for o in range(int(p.instr_op_off[i0]), int(p.instr_op_off[i1])):
            v = int(p.op_vreg[o])
            if v not in slot:
                slot[v] = e
                e += 1
            row[o] = drow[slot[v]]
    return row, e


def test_dictionary_layout_hand_case(oracle_mod):
    # block 0: v0 =; v1 = v0 ; block 1: v2 = v1, v0 ; v0 = v2 ; block 2: use v1
    p = synth.program_from_lists([[([0], []), ([1], [0])], [([2], [1, 0]), ([0], [2])], [([], [1])]],
                                 [(0, 1), (1, 1), (1, 2)], 3, [1, 1, 1], 8)
    off, vreg, instr = oracle_mod.OracleProgram(p).dict_layout()
    assert off.tolist() == [0, 2, 5, 6]
    assert vreg.tolist() == [0, 1, 2, 1, 0, 1]          # block 1: the definition (v2) before the reads (v1, v0)
    assert instr.tolist() == [0, 1, 2, 2, 2, 4]
    soff, svreg, sfirst = synth.dict_layout(p)
    assert soff.tolist() == off.tolist() and svreg.tolist() == vreg.tolist()
    assert sfirst.tolist() == [0, 1, 3, 4, 5, 8]


def test_dictionary_disagreement_between_blocks_hand_case(oracle_mod):
    p = synth.program_from_lists([[([0], []), ([1], [0])], [([2], [1, 0]), ([0], [2])], [([], [1])]],
                                 [(0, 1), (1, 1), (1, 2)], 3, [1, 1, 1], 8)
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    good = np.zeros(8, dtype=np.uint16)
    good[:6] = [0, 1, 2, 1, 0, 1]                        # v0 -> 0, v1 -> 1, v2 -> 2 in every block
    v = op.verify_dict(lv, good)[0]
    assert (v["flags"], v["first_violation_instr"], v["conflict_pairs"]) == (PASS, -1, 0)
    bad = good.copy()
    bad[5] = 5                                           # block 2 says v1 -> 5: the table keeps block 0's value
    w = op.verify_dict(lv, bad)[0]
    assert w["flags"] == INCONS and w["first_violation_instr"] == 4
    assert (w["conflict_pairs"], w["bank_conflicts"]) == (v["conflict_pairs"], v["bank_conflicts"])
    bad2 = good.copy()
    bad2[4] = 2                                          # block 1 says v0 -> 2 (= v2's register): still only inconsistent,
    w2 = op.verify_dict(lv, bad2)[0]                     # because every later check uses the table value 0
    assert w2["flags"] == INCONS and w2["first_violation_instr"] == 2
    first = good.copy()
    first[0] = 1                                         # block 0 (the table value) puts v0 on v1's register
    w3 = op.verify_dict(lv, first)[0]
    assert w3["flags"] & INCONS and w3["flags"] & INTERF
    assert w3["first_violation_instr"] == 1              # v1 is written at instruction 1 while v0 (register 1) is live


@pytest.mark.parametrize("seed", range(30))
def test_dictionary_rows_equal_their_per_occurrence_expansion(oracle_mod, seed):
    """A dictionary row means: every occurrence of v in block b has the register of entry (b, v).  Its
    verdict must be that of the expanded per-occurrence row (expansion written out here by plain loops),
    for consistent tables, for tables that disagree between blocks, and for garbage."""
    p = H.random_program(7000 + seed, strict=True, reachable=(seed % 3 != 0), max_instrs=50, max_vregs=14,
                         P=[8, 16, 32][seed % 3], widths=(1, 1, 2, 4), B=[4, 2, 3][seed % 3])
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    off, vreg, instr = op.dict_layout()
    n = len(vreg)
    soff, svreg, sfirst = synth.dict_layout(p)
    assert np.array_equal(soff, off) and np.array_equal(svreg, vreg)
    assert np.array_equal(np.searchsorted(p.instr_op_off, sfirst, side="right") - 1, instr)
    rng = np.random.default_rng(seed)
    rows = np.zeros((24, synth.dict_pitch(n)), dtype=np.uint16)
    for k in range(24):
        T = rng.integers(0, p.P + (4 if k % 4 == 3 else 0), size=p.n_vregs)
        rows[k, :n] = T[vreg]                                           # every block agrees
        if k % 3 == 1 and n:
            rows[k, rng.integers(0, n, size=2)] = rng.integers(0, p.P, size=2)   # some blocks disagree
        if k % 8 == 7:
            rows[k, :n] = rng.integers(0, 65536, size=n)
    got = op.verify_dict(lv, rows)
    for k in range(24):
        exp, used = _expand_dict_row(p, rows[k])
        assert used == n
        want = op.verify(lv, exp)[0]
        assert got[k].tobytes() == want.tobytes(), (seed, k)
        if k % 3 == 0 and k % 8 != 7:                                    # a consistent table: the row of that table
            T = {int(v): int(rows[k, e]) for e, v in enumerate(vreg)}
            tab = [T.get(v, 0) for v in range(p.n_vregs)]
            assert got[k].tobytes() == op.verify(lv, H.row_from_table(p, tab))[0].tobytes()


def test_dictionary_form_of_generator_rows(oracle_mod):
    """Generator rows in dictionary form: valid rows pass; a row with a vreg moved (interference or
    out-of-file fault: every occurrence moved, so every block's entry moved) keeps its verdict."""
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    rows, faults = synth.candidate_rows(p, 120, 0.4, 9)
    per_occ = op.verify(lv, rows)
    got = op.verify_dict(lv, synth.dict_rows(p, rows))
    keep = faults[:, 0] != synth.FAULT_INCONSISTENT
    assert keep.sum() > 60 and (~keep).sum() > 5
    assert got[keep].tobytes() == per_occ[keep].tobytes()
    assert np.all(got["flags"][faults[:, 0] == synth.FAULT_NONE] == PASS)
