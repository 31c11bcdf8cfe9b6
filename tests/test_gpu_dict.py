"""Parity of vl_verify_dict (candidates as one dictionary per basic block) with the CPU oracle,
through the C ABI, field by field and bit-exact."""
import numpy as np
import pytest

from paper_2506_17506_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2506_17506_b200 import binding
    return binding


def _to_dev(rows):
    import torch
    return torch.from_numpy(rows.view(np.int16)).cuda().view(torch.uint16)


def _gpu_verify_dict(B, gp, rows):
    import torch
    out = gp.vl_verify_dict(_to_dev(rows))
    torch.cuda.synchronize()
    gp.vl_verify_status()
    return B.verdicts_to_numpy(out)


def _assert_same(got, want, what=""):
    for f in ("flags", "first_violation_instr", "conflict_pairs", "bank_conflicts"):
        bad = np.nonzero(got[f] != want[f])[0]
        assert len(bad) == 0, f"{what} field {f}: rows {bad[:8]} got {got[f][bad[:8]]} want {want[f][bad[:8]]}"


def _dict_rows_with_garbage(p, rows, seed):
    """Dictionary form of generator rows, then rows whose blocks disagree, then garbage of every kind."""
    layout = synth.dict_layout(p)
    n = len(layout[1])
    d = synth.dict_rows(p, rows, layout)
    rng = np.random.default_rng(seed)
    extra = np.zeros((30, d.shape[1]), dtype=np.uint16)
    for k in range(30):
        extra[k] = d[k % len(d)]
        mode = k % 5
        if mode == 0 and n:                                   # a few entries changed: blocks disagree
            idx = rng.integers(0, n, size=3)
            extra[k, idx] = rng.integers(0, p.P, size=3)
        elif mode == 1:
            extra[k, :n] = 0
        elif mode == 2:
            extra[k, :n] = rng.integers(0, p.P + 9, size=n)
        elif mode == 3:
            extra[k, :n] = rng.integers(0, 65536, size=n)
        else:
            extra[k, :n] = 0xFFFF
    return np.concatenate([d, extra])


@pytest.mark.parametrize("seed", range(24))
def test_random_small_programs(B, oracle_mod, seed):
    p = H.random_program(6100 + seed, strict=True, reachable=(seed % 4 != 0), max_instrs=60, max_vregs=20,
                         P=[8, 16, 33, 64][seed % 4], widths=(1, 1, 2, 2, 4, 8) if seed % 2 else (1, 2, 3, 5),
                         B=[4, 4, 2, 1, 3, 8][seed % 6])
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    gp = B.Program(p)
    gp.vl_liveness()
    off, vreg = gp.vl_dict_layout()
    o_off, o_vreg, _ = op.dict_layout()
    assert np.array_equal(off, o_off) and np.array_equal(vreg, o_vreg)
    rng = np.random.default_rng(seed)
    base = np.stack([H.row_from_table(p, rng.integers(0, p.P, size=p.n_vregs)) for _ in range(8)])
    rows = _dict_rows_with_garbage(p, base, seed)
    want = op.verify_dict(lv, rows)
    for G in (0, 1, 4, 8):
        gp.set_option(B.VL_OPT_GROUP, G)
        _assert_same(_gpu_verify_dict(B, gp, rows), want, f"seed {seed} G {G}")
    gp.close()


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_workloads_in_dictionary_form(B, oracle_mod, idx):
    """Workloads 1-3: every generator row in dictionary form, plus rows whose blocks disagree and garbage."""
    wl = synth.workload(idx)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    gp = B.Program(p)
    gp.vl_liveness()
    rows, _ = synth.candidate_rows(p, wl.K, wl.fault_rate, wl.seeds[0])
    d = _dict_rows_with_garbage(p, rows, idx)
    want = op.verify_dict(lv, d)
    _assert_same(_gpu_verify_dict(B, gp, d), want, wl.name)
    # the two entry points side by side on one handle: same working sets, neither disturbs the other
    import torch
    out = gp.vl_verify(_to_dev(rows))
    torch.cuda.synchronize()
    _assert_same(B.verdicts_to_numpy(out), op.verify(lv, rows), wl.name + " per occurrence")
    _assert_same(_gpu_verify_dict(B, gp, d), want, wl.name + " again")
    gp.close()


def test_stress_workload_in_dictionary_form(B, oracle_mod):
    """Workload 5: 10,000 dictionary rows in one call (passes over the internal streams), every row
    against the oracle."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    wl = synth.workload(4)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    gp = B.Program(p)
    gp.vl_liveness()
    K = wl.K
    rows = np.empty((K, p.pitch), dtype=np.uint16)
    synth.candidate_rows(p, K, wl.fault_rate, wl.seeds[0], 0, K, out=rows, chunk=256)
    layout = synth.dict_layout(p)
    d = synth.dict_rows(p, rows, layout)
    rng = np.random.default_rng(5)
    n = len(layout[1])
    for k in range(0, K, 97):                                 # some rows whose blocks disagree
        d[k, rng.integers(0, n)] = rng.integers(0, p.P)
    got = _gpu_verify_dict(B, gp, d)
    threads = max(1, min(os.cpu_count() or 1, 32))
    bounds = np.linspace(0, K, threads + 1).astype(int)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        want = np.concatenate(list(ex.map(lambda j: op.verify_dict(lv, d[bounds[j]:bounds[j + 1]]), range(threads))))
    _assert_same(got, want, "stress, dictionary form")
    gp.close()
