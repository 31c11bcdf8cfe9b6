"""Re-sampling statistics and the early-exit loop: CUDA path against the CPU oracle, bit-exact."""
import numpy as np
import pytest

from paper_2506_17506_b200 import synth

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


def _verdict_tensor(flags):
    """A device verdict array with the given flag words (other fields arbitrary)."""
    import torch
    a = np.zeros((len(flags), 4), dtype=np.int32)
    a[:, 0] = flags
    a[:, 1] = -1
    a[:, 2] = 7
    return torch.from_numpy(a).cuda()


def _oracle_stats(oracle_mod, flag_arrays, ks):
    recs = []
    for fl in flag_arrays:
        v = np.zeros(len(fl), dtype=oracle_mod.VERDICT_DTYPE)
        v["flags"] = fl
        recs.append(oracle_mod.sample_stats(v))
    recs = np.array(recs, dtype=oracle_mod.SAMPLE_STATS_DTYPE)
    return recs, oracle_mod.resample_summary(recs, [len(f) for f in flag_arrays], ks)


def _same(got_rec, got_sum, want_rec, want_sum):
    assert np.array_equal(got_rec["first_pass"], want_rec["first_pass"])
    assert np.array_equal(got_rec["n_pass"], want_rec["n_pass"])
    assert got_sum == want_sum


def test_statistics_of_synthetic_verdicts(B, oracle_mod):
    """Many test cases (more than one launch carries), ragged lengths, empty ones, arrays long enough
    for several thread blocks, passing rows at the block seams."""
    rng = np.random.default_rng(11)
    flag_arrays = []
    for c in range(230):
        K = int(rng.integers(0, 400)) if c % 9 else 0
        fl = rng.choice(np.array([2, 4, 8, 6, 14], dtype=np.uint32), size=K)
        if c % 3 and K:
            first = int(rng.integers(0, K))
            fl[first:] = np.where(rng.random(K - first) < 0.3, 1, fl[first:])
            fl[first] = 1
        flag_arrays.append(fl.astype(np.uint32))
    for K, passing in [(8192, [8191]), (8193, [8192]), (300_000, [299_999]), (300_001, [123_457, 123_456, 8192]),
                       (70_000, []), (1, [0]), (1, []), (513, [512])]:
        fl = np.full(K, 8, dtype=np.uint32)
        fl[passing] = 1
        flag_arrays.append(fl)
    ks = [1, 10, 100, 8192, 300_000]
    outs = [_verdict_tensor(f) for f in flag_arrays]
    got_rec, got_sum = B.vl_resample_stats(outs, ks)
    _same(got_rec, got_sum, *_oracle_stats(oracle_mod, flag_arrays, ks))
    # no limits, one case; all eight limits
    got_rec, got_sum = B.vl_resample_stats(outs[:1], [])
    _same(got_rec, got_sum, *_oracle_stats(oracle_mod, flag_arrays[:1], []))
    ks8 = [1, 2, 3, 5, 8, 13, 21, 400]
    got_rec, got_sum = B.vl_resample_stats(outs[:97], ks8)
    _same(got_rec, got_sum, *_oracle_stats(oracle_mod, flag_arrays[:97], ks8))
    # nothing to summarise
    got_rec, got_sum = B.vl_resample_stats([], [1, 10])
    assert len(got_rec) == 0 and got_sum == dict(n_cases=0, n_solved=0, sum_tries=0, max_tries=0, pass_at=[0, 0])


def test_statistics_of_batch_verdicts(B, oracle_mod):
    """Verdicts as vl_verify_batch wrote them (members of the 256-program workload, 100 attempts each)
    against the statistics of the oracle's verdicts."""
    import torch
    wl = synth.workload(3)
    members = [0, 5, 17, 64, 200]
    gps, cands, want_flags = [], [], []
    for j in members:
        p = synth.build_program(wl.shapes[j], wl.seeds[j])
        gp = B.Program(p)
        gp.vl_liveness()
        rows, _ = synth.candidate_rows(p, wl.K, 0.9 if j % 2 else wl.fault_rate, wl.seeds[j])
        op = oracle_mod.OracleProgram(p)
        want_flags.append(op.verify(op.liveness(), rows)["flags"])
        gps.append(gp); cands.append(_to_dev(rows))
    outs = B.vl_verify_batch(gps, cands)
    ks = [1, 10, 100]
    got_rec, got_sum = B.vl_resample_stats(outs, ks)
    want_rec, want_sum = _oracle_stats(oracle_mod, want_flags, ks)
    _same(got_rec, got_sum, want_rec, want_sum)
    assert want_sum["n_solved"] == len(members) and want_sum["max_tries"] > 1   # the case is not trivial
    for gp in gps:
        gp.close()
    torch.cuda.synchronize()


@pytest.mark.parametrize("batch_rows", [1, 7, 32, 100, 1000])
def test_loop_stops_at_the_first_batch_with_a_passing_row(B, oracle_mod, batch_rows):
    import torch
    wl = synth.workload(1)
    p = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, _ = synth.candidate_rows(p, 100, 0.5, wl.seeds[0])
    op = oracle_mod.OracleProgram(p)
    lv = op.liveness()
    v = op.verify(lv, rows)
    bad = np.flatnonzero(v["flags"] != 1)
    good = np.flatnonzero(v["flags"] == 1)
    assert len(bad) >= 40 and len(good) >= 10
    gp = B.Program(p)
    gp.vl_liveness()
    for n_bad_first in (0, 1, 33, 40):
        order = np.concatenate([bad[:n_bad_first], good[:3], bad[n_bad_first:], good[3:]])
        r = np.ascontiguousarray(rows[order])
        want = v[order]
        out, done, first = gp.vl_verify_until_pass(_to_dev(r), batch_rows)
        torch.cuda.synchronize()
        st = oracle_mod.sample_stats(want)
        assert first == int(st["first_pass"]) == n_bad_first
        assert done == min(len(r), (first // batch_rows + 1) * batch_rows)
        got = B.verdicts_to_numpy(out)
        for f in ("flags", "first_violation_instr", "conflict_pairs", "bank_conflicts"):
            assert np.array_equal(got[f][:done], want[f][:done]), f
        assert not got["flags"][done:].any()          # rows after the stop were not written
    # nothing passes: every row is checked, the answer is K
    r = np.ascontiguousarray(rows[bad])
    out, done, first = gp.vl_verify_until_pass(_to_dev(r), batch_rows)
    assert (done, first) == (len(bad), len(bad))
    assert np.array_equal(B.verdicts_to_numpy(out)["flags"], v["flags"][bad])
    # no rows at all
    empty = torch.zeros((0, gp.pitch), dtype=torch.int16, device="cuda").view(torch.uint16)
    out, done, first = gp.vl_verify_until_pass(empty, batch_rows)
    assert (done, first) == (0, 0)
    gp.close()
