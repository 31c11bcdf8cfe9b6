"""Parity of the CUDA path with the CPU oracle, through the C ABI, field by field and bit-exact."""
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


def _gpu_verify(B, gp, rows):
    import torch
    out = gp.vl_verify(_to_dev(rows))
    torch.cuda.synchronize()
    gp.vl_verify_status()
    return B.verdicts_to_numpy(out)


def _assert_same(got, want, what=""):
    for f in ("flags", "first_violation_instr", "conflict_pairs", "bank_conflicts"):
        bad = np.nonzero(got[f] != want[f])[0]
        assert len(bad) == 0, f"{what} field {f}: rows {bad[:8]} got {got[f][bad[:8]]} want {want[f][bad[:8]]}"


def _check_liveness(B, oracle_mod, p, gp=None):
    gp = gp or B.Program(p)
    gp.vl_liveness()
    return _check_liveness_result(B, oracle_mod, gp, p)


def _check_liveness_result(B, oracle_mod, gp, p):
    bin_, bout, lo_off, lo = gp.vl_liveness_result()
    lv = oracle_mod.OracleProgram(p).liveness()
    assert np.array_equal(bin_, lv.packed("in"))
    assert np.array_equal(bout, lv.packed("out"))
    assert np.array_equal(lo_off.astype(np.uint64), lv.lo_off)
    assert np.array_equal(lo, lv.lo)
    return gp, lv


def _garbage_rows(p, n, seed):
    rng = np.random.default_rng(seed)
    rows = np.zeros((n, p.pitch), dtype=np.uint16)
    for k in range(n):
        mode = k % 6
        if mode == 0:
            rows[k, :] = 0
        elif mode == 1:
            rows[k, :] = 0xFFFF
        elif mode == 2:                                   # consistent random table inside the file
            rows[k] = H.row_from_table(p, rng.integers(0, p.P, size=p.n_vregs))
        elif mode == 3:                                   # consistent random table, partly outside
            rows[k] = H.row_from_table(p, rng.integers(0, p.P + 40, size=p.n_vregs))
        elif mode == 4:                                   # per-operand noise (inconsistent)
            rows[k, : p.n_operands] = rng.integers(0, p.P, size=p.n_operands)
        else:                                             # full 16-bit noise
            rows[k, : p.n_operands] = rng.integers(0, 65536, size=p.n_operands)
    return rows


@pytest.mark.parametrize("seed", range(40))
def test_random_small_programs(B, oracle_mod, seed):
    """Random CFGs with multi-definition instructions, wide tuples and >4 reads per instruction;
    valid-ish and garbage rows; every verdict field must match."""
    p = H.random_program(5000 + seed, strict=True, reachable=(seed % 4 != 0), max_instrs=60, max_vregs=20,
                         P=[8, 16, 33, 64][seed % 4], widths=(1, 1, 2, 2, 4, 8) if seed % 2 else (1, 2, 3, 5),
                         B=[4, 4, 2, 1, 3, 8][seed % 6])
    gp, lv = _check_liveness(B, oracle_mod, p)
    rows = _garbage_rows(p, 48, seed)
    want = oracle_mod.OracleProgram(p).verify(lv, rows)
    for G in (0, 1, 2, 4, 8):
        gp.set_option(B.VL_OPT_GROUP, G)
        _assert_same(_gpu_verify(B, gp, rows), want, f"seed {seed} G {G}")
    gp.close()


def test_hand_programs(B, oracle_mod):
    cases = []
    cases.append((synth.program_from_lists([[([0], []), ([1], []), ([2], [0, 1]), ([3], [2]), ([], [3])]], [], 4, [1] * 4, 2),
                  [[0, 1, 0, 0], [0, 0, 1, 0]]))
    cases.append((synth.program_from_lists([[([0], []), ([1], [])], [([2], [1]), ([0], [0, 2])], [([], [0])]],
                                           [(0, 1), (1, 1), (1, 2)], 3, [2, 1, 1], 4),
                  [[0, 2, 3], [0, 2, 2], [0, 1, 3], [3, 0, 1]]))
    cases.append((synth.program_from_lists([[([0, 1], []), ([2], [0]), ([], [1, 2])]], [], 3, [1, 1, 1], 4),
                  [[0, 0, 1], [0, 1, 2], [65535, 65535, 0]]))
    cases.append((synth.program_from_lists([[([0], []), ([], [0])], [([1], [0])]], [], 2, [1, 1], 2), [[0, 0], [1, 1]]))
    for p, tables in cases:
        gp, lv = _check_liveness(B, oracle_mod, p)
        rows = np.stack([H.row_from_table(p, t) for t in tables])
        rows[-1, min(3, p.n_operands - 1)] ^= 1           # one inconsistent row as well
        _assert_same(_gpu_verify(B, gp, rows), oracle_mod.OracleProgram(p).verify(lv, rows))
        gp.close()


def test_not_strict_and_order_errors(B):
    p = synth.program_from_lists([[([], [0]), ([0], [])]], [], 1, [1], 4)      # reads v0 before writing it
    gp = B.Program(p)
    with pytest.raises(B.VlError) as e:
        gp.vl_liveness()
    assert e.value.code == B.VL_ERR_NOT_STRICT
    import torch
    cand = torch.zeros((1, 8), dtype=torch.int16, device="cuda").view(torch.uint16)
    with pytest.raises(B.VlError) as e:
        gp.vl_verify(cand)
    assert e.value.code == B.VL_ERR_LIVENESS_NOT_RUN
    gp.close()
    ok = synth.program_from_lists([[([0], []), ([], [0])]], [], 1, [1], 4)
    gp = B.Program(ok)
    gp.vl_liveness()
    bad_pitch = torch.zeros((1, 12), dtype=torch.int16, device="cuda").view(torch.uint16)
    with pytest.raises(B.VlError) as e:
        gp.vl_verify(bad_pitch)
    assert e.value.code == B.VL_ERR_INVALID_ARG
    empty = torch.zeros((0, 8), dtype=torch.int16, device="cuda").view(torch.uint16)
    assert gp.vl_verify(empty).shape[0] == 0
    gp.close()


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_workloads_full(B, oracle_mod, idx):
    """Workloads 1-3 in full: every row of the seeded candidate matrix."""
    wl = synth.workload(idx)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp, lv = _check_liveness(B, oracle_mod, p)
    rows, faults = synth.candidate_rows(p, wl.K, wl.fault_rate, wl.seeds[0])
    want = oracle_mod.OracleProgram(p).verify(lv, rows)
    got = _gpu_verify(B, gp, rows)
    _assert_same(got, want, wl.name)
    assert np.array_equal(got["flags"] == B.VL_PASS, faults[:, 0] == 0)
    # host-buffer entry point gives the same records
    host = gp.vl_verify_host(rows)
    _assert_same(host, want, wl.name + " host")
    # extra rows: garbage of every kind
    rows2 = _garbage_rows(p, 24, idx)
    _assert_same(_gpu_verify(B, gp, rows2), oracle_mod.OracleProgram(p).verify(lv, rows2), wl.name + " garbage")
    gp.close()


@pytest.mark.parametrize("chunk,G,threads", [(16, 4, 256), (64, 2, 512), (512, 1, 0), (4096, 0, 512), (128, 4, 512),
                                              (48, 8, 256), (160, 8, 512)])
def test_options_do_not_change_results(B, oracle_mod, chunk, G, threads):
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp = B.Program(p)
    gp.set_option(B.VL_OPT_CHUNK_INSTRS, chunk)
    gp.set_option(B.VL_OPT_GROUP, G)
    gp.set_option(B.VL_OPT_THREADS, threads)
    gp, lv = _check_liveness(B, oracle_mod, p, gp)
    rows, _ = synth.candidate_rows(p, wl.K, 0.5, 77)
    rows = np.concatenate([rows[:61], _garbage_rows(p, 12, 3)])     # ragged: 73 rows
    _assert_same(_gpu_verify(B, gp, rows), oracle_mod.OracleProgram(p).verify(lv, rows), f"chunk {chunk} G {G}")
    gp.close()


@pytest.mark.parametrize("P,widths", [(4000, (1, 2, 8)), (5000, (1, 3, 40)), (300, (1, 5, 40, 64)), (97, (1, 2, 33)),
                                      (1000, (1, 2, 255))])
def test_large_files_and_very_wide_tuples(B, oracle_mod, P, widths):
    """Register files of many mask words, tuples wider than one 32-bit mask word, and packed tables
    whose ranges keep crossing word boundaries."""
    for seed in range(4):
        p = H.random_program(9000 + seed, strict=True, reachable=True, max_instrs=50, max_vregs=16, P=P,
                             widths=widths, B=4)
        gp, lv = _check_liveness(B, oracle_mod, p)
        rng = np.random.default_rng(seed)
        rows = [_garbage_rows(p, 12, seed)]
        tabs = np.zeros((20, p.n_vregs), dtype=np.int64)
        for k in range(20):                                # packed tables that tend to straddle mask words
            base = int(rng.integers(0, 64)) if k % 2 else int(rng.integers(max(1, P - 200), P))
            pos = base
            for v in rng.permutation(p.n_vregs):
                tabs[k, v] = min(pos, 65535)
                pos += int(p.vreg_width[v]) if k % 4 < 3 else 1
        rows.append(np.stack([H.row_from_table(p, t) for t in tabs]))
        rows = np.concatenate(rows)
        want = oracle_mod.OracleProgram(p).verify(lv, rows)
        _assert_same(_gpu_verify(B, gp, rows), want, f"P {P} seed {seed}")
        gp.close()


def test_register_file_too_large_is_refused(B):
    p = H.random_program(1, strict=True, P=40000)
    gp = B.Program(p)
    gp.vl_liveness()
    import torch
    with pytest.raises(B.VlError) as e:
        gp.vl_verify(torch.zeros((4, p.pitch), dtype=torch.uint16, device="cuda"))
    assert e.value.code == B.VL_ERR_UNSUPPORTED
    gp.close()


@pytest.mark.parametrize("lanes,sub", [(1, 64), (2, 32), (3, 96), (4, 32), (8, 32), (4, 4096)])
def test_passes_over_lanes(B, oracle_mod, lanes, sub):
    """Many passes spread over the internal streams give the records of a single pass."""
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp, lv = _check_liveness(B, oracle_mod, p)
    rows, _ = synth.candidate_rows(p, 500, 0.3, 11)
    rows = np.concatenate([rows[:487], _garbage_rows(p, 12, 5)])     # 499 rows: ragged last pass
    want = oracle_mod.OracleProgram(p).verify(lv, rows)
    gp.set_option(B.VL_OPT_LANES, lanes)
    gp.set_option(B.VL_OPT_SUB_BATCH, sub)
    for _ in range(2):                                               # working sets reused by the next call
        _assert_same(_gpu_verify(B, gp, rows), want, f"lanes {lanes} sub {sub}")
    gp.close()


def _oracle_rows_threaded(oracle_mod, p, lv, rows):
    """Oracle verdicts of every row, the rows split over the host's threads (the oracle itself stays
    single-threaded; ctypes releases the interpreter lock during a call)."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    op = oracle_mod.OracleProgram(p)
    threads = max(1, min(os.cpu_count() or 1, 32, len(rows)))
    bounds = np.linspace(0, len(rows), threads + 1).astype(int)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        outs = list(ex.map(lambda j: op.verify(lv, rows[bounds[j]:bounds[j + 1]]), range(threads)))
    return np.concatenate(outs)


def test_batch_call(B, oracle_mod):
    """Workload 4 in full: all 256 independent programs through vl_liveness_batch and vl_verify_batch,
    every row of every program against the oracle."""
    import torch
    wl = synth.workload(3)
    members = list(range(len(wl.shapes)))
    assert len(members) == 256
    progs, gps, cands, wants = [], [], [], []
    for j in members:
        p = synth.build_program(wl.shapes[j], wl.seeds[j])
        rows, _ = synth.candidate_rows(p, wl.K, wl.fault_rate, wl.seeds[j])
        lv = oracle_mod.OracleProgram(p).liveness()
        progs.append(p); gps.append(B.Program(p)); cands.append(_to_dev(rows))
        wants.append(oracle_mod.OracleProgram(p).verify(lv, rows))
    B.vl_liveness_batch(gps)
    outs = B.vl_verify_batch(gps, cands)
    torch.cuda.synchronize()
    for j, o, w in zip(members, outs, wants):
        _assert_same(B.verdicts_to_numpy(o), w, f"batch member {j}")
    for gp, p in zip(gps, progs):
        _check_liveness_result(B, oracle_mod, gp, p)
    # liveness of all members in one call, several times (the later runs are replayed recordings):
    # same liveness results, same verdicts
    for _ in range(4):
        B.vl_liveness_batch(gps)
    for gp, p in zip(gps[::16], progs[::16]):
        _check_liveness_result(B, oracle_mod, gp, p)
    outs = B.vl_verify_batch(gps, cands)
    torch.cuda.synchronize()
    for j, o, w in zip(members, outs, wants):
        _assert_same(B.verdicts_to_numpy(o), w, f"batch member {j} after vl_liveness_batch")
    for gp in gps:
        gp.close()


def test_stress_workload_full(B, oracle_mod):
    """Workload 5 at full size, in the launch configuration the benchmark times (all 10,000 rows in
    one call, its passes spread over the internal streams): liveness compared in full, every one of
    the 10,000 verdicts compared with the oracle's, and besides that what holds by construction (a
    row passes iff no fault was injected; the host-buffer entry point gives the same records)."""
    wl = synth.workload(4)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp, lv = _check_liveness(B, oracle_mod, p)
    K = wl.K
    rows = np.empty((K, p.pitch), dtype=np.uint16)
    _, faults = synth.candidate_rows(p, K, wl.fault_rate, wl.seeds[0], 0, K, out=rows, chunk=256)
    got = _gpu_verify(B, gp, rows)
    want = _oracle_rows_threaded(oracle_mod, p, lv, rows)
    _assert_same(got, want, "stress")
    assert np.array_equal(got["flags"] == B.VL_PASS, faults[:, 0] == 0)     # valid by construction / injected
    assert np.all(got["conflict_pairs"][faults[:, 0] == 0] == 0)
    host = gp.vl_verify_host(rows[:1500])
    assert host.tobytes() == got[:1500].tobytes()
    garbage = _garbage_rows(p, 6, 9)
    _assert_same(_gpu_verify(B, gp, garbage), oracle_mod.OracleProgram(p).verify(lv, garbage), "stress garbage")
    gp.close()


def test_recount_work_list_full(B, oracle_mod):
    """Passes in which every candidate collides in nearly every chunk and through-set: the work list
    of the exact recount is as long as it gets (all-zero rows and uniform noise on the GEMM-shaped
    program, which has through-sets; 32 rows per pass)."""
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp, lv = _check_liveness(B, oracle_mod, p)
    rng = np.random.default_rng(42)
    rows = np.zeros((128, p.pitch), dtype=np.uint16)
    rows[64:, : p.n_operands] = rng.integers(0, p.P, size=(64, p.n_operands))
    for k in range(96, 128):                              # consistent random tables: every chunk collides
        rows[k] = H.row_from_table(p, rng.integers(0, p.P, size=p.n_vregs))
    want = oracle_mod.OracleProgram(p).verify(lv, rows)
    for sub, chunk in ((32, 0), (64, 24), (32, 150)):
        gp.set_option(B.VL_OPT_SUB_BATCH, sub)
        if chunk:
            gp.set_option(B.VL_OPT_CHUNK_INSTRS, chunk)
            gp.vl_liveness()
        _assert_same(_gpu_verify(B, gp, rows), want, f"sub {sub} chunk {chunk}")
    gp.close()


def test_bounded_device_wait_runs_out(B, oracle_mod):
    """The waits of the table kernel on its copy ring are bounded.  With the test hook switched on
    the kernel waits on a barrier that nothing completes, with a short poll limit: the wait gives up,
    the call still returns (nothing traps, nothing keeps spinning), vl_verify_status reports
    VL_ERR_DEVICE_WAIT, and the next call without the hook is bit-exact again."""
    import torch
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp, lv = _check_liveness(B, oracle_mod, p)
    rows, _ = synth.candidate_rows(p, 40, 0.3, 21)
    want = oracle_mod.OracleProgram(p).verify(lv, rows)
    _assert_same(_gpu_verify(B, gp, rows), want, "before")
    gp.set_option(B.VL_OPT_GROUP, 8)                      # the hook sits in the eight-candidate table kernel
    gp.set_option(B.VL_OPT_TEST_WAIT, 1)
    gp.vl_verify(_to_dev(rows))
    torch.cuda.synchronize()                              # the kernels end by themselves
    with pytest.raises(B.VlError) as e:
        gp.vl_verify_status()
    assert e.value.code == B.VL_ERR_DEVICE_WAIT
    gp.set_option(B.VL_OPT_TEST_WAIT, 0)
    for _ in range(2):
        _assert_same(_gpu_verify(B, gp, rows), want, "after the wait ran out")
    gp.close()


def test_repeated_liveness_runs(B, oracle_mod):
    """Later liveness runs of a handle return without waiting for the GPU and are replayed from a
    recording: the results stay those of the first run, a changed chunk size starts over, and the
    verdicts computed behind an unsettled run are right."""
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, _ = synth.candidate_rows(p, 64, 0.4, 3)
    gp, lv = _check_liveness(B, oracle_mod, p)
    want = oracle_mod.OracleProgram(p).verify(lv, rows)
    for run in range(6):
        gp.vl_liveness()
        if run % 2:
            _check_liveness_result(B, oracle_mod, gp, p)
        _assert_same(_gpu_verify(B, gp, rows), want, f"run {run}")
    gp.set_option(B.VL_OPT_CHUNK_INSTRS, 40)
    for run in range(5):
        gp.vl_liveness()
        _assert_same(_gpu_verify(B, gp, rows), want, f"chunk 40 run {run}")
    _check_liveness_result(B, oracle_mod, gp, p)
    gp.close()


def test_determinism(B):
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp = B.Program(p)
    gp.vl_liveness()
    rows, _ = synth.candidate_rows(p, wl.K, 0.5, 5)
    a = _gpu_verify(B, gp, rows)
    b = _gpu_verify(B, gp, rows)
    assert a.tobytes() == b.tobytes()
    gp.close()


def test_liveness_and_verify_on_different_streams(B, oracle_mod):
    """vl_liveness runs on an internal stream and holds no caller stream; vl_verify waits for it on the
    device where it reads its results.  Liveness on one stream, verify on another, no synchronisation
    in between, new rows every step, several passes per call: every verdict must be right."""
    import torch
    wl = synth.workload(2)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    gp, lv = _check_liveness(B, oracle_mod, p)
    gp.set_option(B.VL_OPT_SUB_BATCH, 128)
    orc = oracle_mod.OracleProgram(p)
    s_live, s_ver = torch.cuda.Stream(), torch.cuda.Stream()
    outs, wants = [], []
    for step in range(6):
        rows, _ = synth.candidate_rows(p, 600, 0.3, 100 + step)
        dev = _to_dev(rows)                      # (copied on the default stream; make s_ver wait for it)
        s_ver.wait_stream(torch.cuda.current_stream())
        s_live.wait_stream(s_ver)                # (the run rewrites what the previous step's verify still reads)
        gp.vl_liveness(s_live)
        outs.append((gp.vl_verify(dev, None, s_ver), dev))
        wants.append(orc.verify(lv, rows))
    torch.cuda.synchronize()
    gp.vl_verify_status()
    for step, ((out, _), want) in enumerate(zip(outs, wants)):
        _assert_same(B.verdicts_to_numpy(out), want, f"step {step}")
    _check_liveness_result(B, oracle_mod, gp, p)
    gp.close()
