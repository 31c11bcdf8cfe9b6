"""The several-GPU path on CPU: two `gloo` ranks split the rows, each checks its shard (the oracle stands
in for the GPU here, this test is about the sharding and the reductions), and the union must equal
the single-process result with the job totals reduced correctly."""
import os
import socket

import numpy as np
import pytest
import torch.multiprocessing as mp

from paper_2506_17506_b200 import shard, synth


def test_row_range_partitions():
    for n_rows in (0, 1, 31, 32, 33, 1000, 4096, 10000):
        for world in (1, 2, 3, 8):
            prev = 0
            sizes = []
            for r in range(world):
                lo, hi = shard.row_range(r, world, n_rows)
                assert lo == prev and hi >= lo
                if hi < n_rows:
                    assert hi % 32 == 0
                sizes.append(hi - lo)
                prev = hi
            assert prev == n_rows
            assert max(sizes) - min(sizes) < 64
    with pytest.raises(ValueError):
        shard.row_range(2, 2, 10)
    assert shard.weak_rows(3, 100) == (300, 400)


def test_job_totals_single_process():
    assert shard.job_totals(7, 2.5, 3) == (7, 2.5, 3)
    assert shard.throughput(1000, 500.0) == 2000.0


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n_rows, tmpdir):
    import torch.distributed as dist
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = synth.workload(0)
        prog = synth.build_program(wl.shapes[0], wl.seeds[0])
        lo, hi = shard.row_range(rank, world, n_rows)
        rows, _ = synth.candidate_rows(prog, n_rows, 0.3, wl.seeds[0], lo, hi)
        op = oracle.OracleProgram(prog)
        v = op.verify(op.liveness(), rows)
        np.save(os.path.join(tmpdir, f"v{rank}.npy"), v)
        passing = int((v["flags"] == 1).sum())
        total, ms, npass = shard.job_totals(hi - lo, 10.0 * (rank + 1), passing)
        st = oracle.sample_stats(v)
        first, n_all = shard.job_sample_stats(int(st["first_pass"]), int(st["n_pass"]), hi - lo, lo, n_rows)
        # a job in which only the last rank has passing rows, and one in which nobody has
        late = shard.job_sample_stats(3 if rank == world - 1 else hi - lo, 1 if rank == world - 1 else 0, hi - lo, lo, n_rows)
        none = shard.job_sample_stats(hi - lo, 0, hi - lo, lo, n_rows)
        if rank == 0:
            np.save(os.path.join(tmpdir, "totals.npy"), np.array([total, ms, npass], dtype=np.float64))
            np.save(os.path.join(tmpdir, "stats.npy"), np.array([first, n_all, *late, *none], dtype=np.int64))
    finally:
        dist.destroy_process_group()


def test_two_ranks_cover_the_job(tmp_path, oracle_mod):
    n_rows, world = 100, 2
    mp.spawn(_rank_main, args=(world, _free_port(), n_rows, str(tmp_path)), nprocs=world, join=True)
    wl = synth.workload(0)
    prog = synth.build_program(wl.shapes[0], wl.seeds[0])
    rows, _ = synth.candidate_rows(prog, n_rows, 0.3, wl.seeds[0], 0, n_rows)
    op = oracle_mod.OracleProgram(prog)
    want = op.verify(op.liveness(), rows)
    got = np.concatenate([np.load(tmp_path / f"v{r}.npy") for r in range(world)])
    assert np.array_equal(got.view(np.int32), want.view(np.int32))
    total, ms, npass = np.load(tmp_path / "totals.npy")
    assert total == n_rows and ms == 20.0 and npass == int((want["flags"] == 1).sum())
    assert 0 < npass < n_rows
    first, n_all, late_first, late_n, none_first, none_n = np.load(tmp_path / "stats.npy")
    st = oracle_mod.sample_stats(want)
    assert (first, n_all) == (int(st["first_pass"]), int(st["n_pass"]))
    last_lo = shard.row_range(world - 1, world, n_rows)[0]
    assert (late_first, late_n) == (last_lo + 3, 1) and (none_first, none_n) == (n_rows, 0)


def test_job_sample_stats_single_process():
    assert shard.job_sample_stats(5, 2, 10, 100, 1000) == (105, 2)
    assert shard.job_sample_stats(10, 0, 10, 100, 1000) == (1000, 0)


def test_bench_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a launcher around it starts two ranks (here with the stub step, which
    does everything around the GPU work on CPU: process group, barrier, reductions, one JSON line)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    env["VL_BENCH_STUB"] = "1"
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "3"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(ln) for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout
    assert lines[0]["n_gpus"] == 2 and lines[0]["gpus_arg"] == 2
    assert lines[0]["rows_all"] == 2 * 300 and lines[0]["ms"] == 2.0      # sum of rows, slowest rank's time
