#!/usr/bin/env python
"""Benchmark: candidate verifications per second on the stress workload (one program of 32,000
instructions / 10,000 vregs, K = 10,000 per-operand uint16 candidate rows, about 2 GB).

A step is the whole path for one batch: vl_liveness on the program, then vl_verify over the
K rows.  `value` is measured with the rows resident in HBM; `e2e` goes through vl_verify_host
with pinned host buffers, copies inside the timed region.  vl_verify spreads its passes over
internal streams, so its kernels overlap in the timed region; the per-kernel durations behind
`roofline` come from a second timed loop with the passes in order on one stream
(VL_OPT_LANES = 1), where a kernel's duration is its own.  Prints one JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--rows R]

With --gpus N > 1 and no launcher around it (WORLD_SIZE unset) the script starts the N ranks itself,
by running itself under torch.distributed.run on 127.0.0.1; started by a launcher it reads
RANK / LOCAL_RANK / WORLD_SIZE from the environment.  One process per GPU, rows sharded over the
ranks, NCCL only for the barrier, the slowest rank's time and the row total.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_17506_b200 import shard, synth  # noqa: E402

METRIC = "candidate_verifications_per_sec"
UNIT = "verifications/s"
WORKLOAD_INDEX = 4


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-i", str(self.index),
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            parts = [x.strip() for x in s.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


def build_inputs(rank: int, rows: int, pinned: bool, fault_rate: float = -1.0):
    wl = synth.workload(WORKLOAD_INDEX)
    if fault_rate >= 0:
        wl.fault_rate = fault_rate
    prog = synth.build_program(wl.shapes[0], wl.seeds[0])
    K = rows or wl.K
    pitch = prog.pitch
    if pinned:
        import torch
        host = torch.empty((K, pitch), dtype=torch.int16, pin_memory=True)
        arr = host.numpy().view(np.uint16)
    else:
        host = None
        arr = np.empty((K, pitch), dtype=np.uint16)
    t0 = time.time()
    # rank r checks rows [r*K, (r+1)*K) of the same seeded candidate stream
    lo, hi = shard.weak_rows(rank, K)
    synth.candidate_rows(prog, hi, wl.fault_rate, wl.seeds[0], lo, hi, out=arr, chunk=256)
    log(f"[bench] rank {rank}: generated {K} rows x {pitch} operands in {time.time() - t0:.1f}s")
    return wl, prog, K, host, arr


def oracle_rate(prog, arr, n_rows: int, threads: int):
    """Oracle verdicts for the first n_rows rows, split over `threads` host threads."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    op = oracle.OracleProgram(prog)
    t0 = time.perf_counter()
    lv = op.liveness()
    t_live = time.perf_counter() - t0
    n_rows = min(n_rows, arr.shape[0])
    bounds = np.linspace(0, n_rows, threads + 1).astype(int)
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        outs = list(ex.map(lambda j: op.verify(lv, arr[bounds[j]:bounds[j + 1]]), range(threads)))
    dt = time.perf_counter() - t0
    return n_rows / dt, dt, t_live, np.concatenate(outs), lv


def config_of(prog, wl, K, world):
    """The `config` object of the JSON line: the workload both arms are quoted on."""
    return {"workload": "stress", "n_blocks": prog.n_blocks, "n_instrs": prog.n_instrs, "n_vregs": prog.n_vregs,
            "n_operands": prog.n_operands, "P": prog.P, "B": prog.B, "K_per_gpu": K, "fault_rate": wl.fault_rate,
            "parallelism": f"rows sharded over {world} GPU(s)", "l2": "inputs (2 GB per step) larger than L2, no flush"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    threads = os.cpu_count() or 1
    sample = max(threads, threads * 8)
    wl, prog, K, _, arr = build_inputs(0, sample, pinned=False)
    rates = []
    for s in range(args.warmup + args.steps):
        rate, dt, t_live, _, _ = oracle_rate(prog, arr, sample, threads)
        if s >= args.warmup:
            rates.append(rate)
    value = float(np.mean(rates))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sample / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u16", "data": "synthetic",
        # the workload is the GPU arm's; a step of this arm checks a bounded sample of its rows
        "config": config_of(prog, wl, wl.K, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"the first {sample} of the workload's {wl.K} rows per step, {threads} host threads"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def spawn_ranks(n: int) -> int:
    """Runs this script as n ranks on this node (one per GPU) and returns the launcher's exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_stub(args):
    """What the several-rank path does around the GPU work, without a GPU: process group (gloo), barrier,
    the reductions of the report, one JSON line from rank 0.  Used by the CPU test of `--gpus N`."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    rows_all, ms, _ = shard.job_totals(100 * args.steps, 1.0 + rank, 0, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"stub": True, "n_gpus": world, "gpus_arg": args.gpus, "rows_all": rows_all, "ms": ms}), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def measured_traffic(kernel_names):
    """DRAM bytes (read + write) per candidate of each verify kernel, from the profiler capture recorded in
    `profiles/dram_traffic_stress.txt`, or None when the kernels' source has changed since (the record
    carries a hash of vl_verify.cu): a figure must not outlive the kernel it was taken from."""
    import hashlib
    rec = os.path.join(ROOT, "profiles", "dram_traffic_stress.txt")
    src = os.path.join(ROOT, "paper_2506_17506_b200", "csrc", "vl_verify.cu")
    try:
        fields = dict(line.split(":", 1) for line in open(rec).read().splitlines() if ":" in line and not line.startswith("#"))
        if fields["vl_verify.cu sha256"].strip() != hashlib.sha256(open(src, "rb").read()).hexdigest():
            return None
        rows = float(fields["rows"])
        return {n: float(fields[n + " dram bytes"]) / rows for n in kernel_names if n + " dram bytes" in fields}
    except Exception:
        return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--rows", type=int, default=0, help="candidate rows per GPU (default: the workload's 10,000)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--group", type=int, default=0)
    ap.add_argument("--lanes", type=int, default=0, help="internal streams of vl_verify (default: the library's)")
    ap.add_argument("--sub-batch", type=int, default=0, help="candidates per pass (default: the library's)")
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--stagger", type=int, default=-1, help="start offset (us) between the classes of the first wave of the table kernel")
    ap.add_argument("--threads", type=int, default=0, help="threads per block of the table kernel (default: the library's)")
    ap.add_argument("--prefetch", type=int, default=-1, help="tiles the table kernel asks into L2 ahead (default: the library's)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fault-rate", type=float, default=-1.0, help="override the workload's faulted fraction")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus)
    if os.environ.get("VL_BENCH_STUB") == "1":
        return run_stub(args)

    import torch
    import torch.distributed as dist
    from paper_2506_17506_b200 import binding as vl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")   # the communicator lines show the ranks that joined
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    wl, prog, K, host, arr = build_inputs(rank, args.rows, pinned=True, fault_rate=args.fault_rate)
    gp = vl.Program(prog, device=local)
    if args.group:
        gp.set_option(vl.VL_OPT_GROUP, args.group)
    if args.chunk:
        gp.set_option(vl.VL_OPT_CHUNK_INSTRS, args.chunk)
    if args.lanes:
        gp.set_option(vl.VL_OPT_LANES, args.lanes)
    if args.sub_batch:
        gp.set_option(vl.VL_OPT_SUB_BATCH, args.sub_batch)
    if args.threads:
        gp.set_option(vl.VL_OPT_THREADS, args.threads)
    if args.stagger >= 0:
        gp.set_option(vl.VL_OPT_STAGGER_US, args.stagger)
    if args.prefetch >= 0:
        gp.set_option(vl.VL_OPT_PREFETCH_TILES, args.prefetch)
    dev_rows = host.cuda().view(torch.uint16)
    out = torch.empty((K, 4), dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        gp.vl_liveness(stream)
        gp.vl_verify(dev_rows, out, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()

    # ---- timed region: K rows per step, rows (2 GB) far larger than L2, no flush needed
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = vl.vl_kernel_launches()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    gp.set_option(vl.VL_OPT_KERNEL_TIMING, 1)   # events around each verify kernel, read after the timed region
    barrier()
    ev[0].record(stream)
    for s in range(args.steps):
        # vl_liveness goes to an internal stream and does not hold the caller's stream; vl_verify's table
        # kernels run beside it, its walk waits for it: the events around vl_verify span both
        gp.vl_liveness(stream)
        kev[s][0].record(stream)
        gp.vl_verify(dev_rows, out, stream)
        kev[s][1].record(stream)
    ev[1].record(stream)
    barrier()
    launches = vl.vl_kernel_launches() - launches0
    gp.vl_verify_status(stream)
    overlap_ms, overlap_passes = gp.vl_kernel_times()
    total_ms = ev[0].elapsed_time(ev[1])
    step_verify_ms = float(np.mean([a.elapsed_time(b) for a, b in kev]))
    # ---- vl_verify alone, as the timed region runs it (same rows, same internal streams), no liveness run in
    # flight: the figure the roofline of the verify path is computed from
    gp.set_option(vl.VL_OPT_KERNEL_TIMING, 0)
    for _ in range(3):
        gp.vl_verify(dev_rows, out, stream)
    barrier()
    for s in range(args.steps):
        kev[s][0].record(stream)
        gp.vl_verify(dev_rows, out, stream)
        kev[s][1].record(stream)
    barrier()
    # ---- vl_liveness alone: host clock around the call and the wait for its results
    t0 = time.perf_counter()
    for _ in range(args.steps):
        gp.vl_liveness(stream)
        gp.vl_liveness_wait()
    live_ms = (time.perf_counter() - t0) / args.steps * 1e3
    # ---- second timed loop, same rows: passes in order on one stream, so that the events around a
    # kernel time that kernel alone (the clock sampler keeps running)
    iso_steps = max(3, min(args.steps, 30))
    gp.set_option(vl.VL_OPT_LANES, 1)
    for _ in range(3):
        gp.vl_verify(dev_rows, out, stream)
    barrier()
    gp.set_option(vl.VL_OPT_KERNEL_TIMING, 1)
    iso_ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    iso_ev[0].record(stream)
    for _ in range(iso_steps):
        gp.vl_verify(dev_rows, out, stream)
    iso_ev[1].record(stream)
    barrier()
    kernel_ms, kernel_passes = gp.vl_kernel_times()
    iso_verify_ms = iso_ev[0].elapsed_time(iso_ev[1]) / iso_steps
    gp.set_option(vl.VL_OPT_KERNEL_TIMING, 0)
    gp.set_option(vl.VL_OPT_LANES, args.lanes or 3)
    clocks = sampler.stop() if rank == 0 else None
    verify_ms = float(np.mean([a.elapsed_time(b) for a, b in kev]))
    rows_all, total_ms, _ = shard.job_totals(K * args.steps, total_ms, 0, torch.device("cuda", local))
    value = shard.throughput(rows_all, total_ms)

    # ---- end to end through the host-buffer entry point
    e2e_steps = max(1, args.e2e_steps)
    out_host = np.zeros(K, dtype=vl.VERDICT_DTYPE)
    gp.vl_liveness(stream)
    gp.vl_verify_host(host, out_host, stream)      # warm: allocates the staging buffers
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        gp.vl_liveness(stream)
        gp.vl_verify_host(host, out_host, stream)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    rows_all, e2e_ms, _ = shard.job_totals(K * e2e_steps, e2e_s * 1e3, 0, torch.device("cuda", local))
    e2e_value = shard.throughput(rows_all, e2e_ms)

    # sanity: device-resident and host-buffer results agree
    dev_v = vl.verdicts_to_numpy(out)
    same = bool(np.array_equal(dev_v.view(np.int32), out_host.view(np.int32)))
    n_pass = int((dev_v["flags"] == 1).sum())

    if rank == 0:
        peak, peak_kind = measured_peak_gbs()
        # algorithmic bytes: every candidate row is read once (2 bytes per operand column) and one 16-byte
        # verdict is written; the table kernel is the one that streams the rows
        bytes_per_step = 2.0 * prog.pitch * K + 16.0 * K
        # the four timing slots of a pass (the table kernel; the through-set kernel and the walk; the stand-alone
        # verdict step of programs without instructions; the recount)
        names = ["k_tables8", "k_through+k_walk", "k_finish", "k_recount"]
        passes = max(1, kernel_passes)
        ksum = max(1e-9, sum(kernel_ms))
        kernels = {n: {"ms_per_launch": kernel_ms[j] / passes, "share": kernel_ms[j] / ksum} for j, n in enumerate(names)}
        osum = max(1e-9, sum(overlap_ms))
        overlapped = {n: {"ms_per_launch": overlap_ms[j] / max(1, overlap_passes), "share": overlap_ms[j] / osum}
                      for j, n in enumerate(names)}
        dom = max(range(4), key=lambda j: kernel_ms[j])
        dom_ms = kernel_ms[dom] / passes
        bytes_per_launch = bytes_per_step * iso_steps / passes
        dom_achieved = bytes_per_launch / (dom_ms * 1e-3) / 1e9
        path_achieved = bytes_per_step / (verify_ms * 1e-3) / 1e9
        per_cand = measured_traffic(names)
        traffic = sum(per_cand.values()) * K if per_cand else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u16", "data": "synthetic",
            "config": config_of(prog, wl, K, world),
            "operand_checks_per_sec": value * prog.n_operands,
            "verify_ms": verify_ms, "liveness_ms": live_ms, "verify_in_step_ms": step_verify_ms,
            # the figures of the whole vl_verify call as the timed region runs it (every verify kernel, passes
            # spread over the library's internal streams); the dominant kernel alone is a sub-field
            "roofline": {"bound": "hbm", "achieved": path_achieved, "peak": peak, "unit": "GB/s", "frac": path_achieved / peak,
                         "traffic": traffic, "kernel": "vl_verify (k_tables8 + k_through + k_walk + k_recount)",
                         "of": peak_kind, "launches": args.steps, "ms_per_launch": verify_ms,
                         "bytes_per_launch": bytes_per_step,
                         "how": "CUDA events on the caller's stream around each of the vl_verify calls of a loop of its own "
                                "(same rows, same internal streams, no liveness run in flight); algorithmic bytes = rows "
                                "read once + verdicts",
                         "in_step": {"what": "the same bytes over the whole step of the timed region (vl_liveness on its "
                                             "internal stream beside the table kernels of vl_verify)",
                                     "ms": total_ms / args.steps,
                                     "frac": bytes_per_step / (total_ms / args.steps * 1e-3) / 1e9 / peak},
                         "traffic_source": ("profiles/dram_traffic_stress.txt (ncu capture of one pass per kernel, scaled by rows)"
                                            if traffic else None),
                         "dominant_kernel": {"kernel": names[dom], "achieved": dom_achieved, "frac": dom_achieved / peak,
                                             "launches": passes, "ms_per_launch": dom_ms, "bytes_per_launch": bytes_per_launch,
                                             "how": f"CUDA events around every launch, {iso_steps} vl_verify calls with their "
                                                    "passes in order on one stream (VL_OPT_LANES=1), so that no other "
                                                    "kernel runs beside the timed one"},
                         "path_in_order": {"what": "one vl_verify call with VL_OPT_LANES=1", "ms": iso_verify_ms,
                                           "frac": bytes_per_step / (iso_verify_ms * 1e-3) / 1e9 / peak},
                         "kernels": kernels, "kernels_in_timed_region": overlapped},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(2 * prog.pitch * K),
                    "d2h_bytes_per_step": int(16 * K)},
            "gpu_launches": int(launches),
            "checks": {"host_equals_device": same, "rows_passing": n_pass},
        }
        if not args.no_cpu_baseline and world == 1:
            threads = os.cpu_count() or 1
            sample = min(K, max(threads * 256, 1024))
            rate, dt, t_live, ov, _ = oracle_rate(prog, arr, sample, threads)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
                                    "sample": f"first {sample} rows of the same workload, {dt:.1f}s on {threads} threads "
                                              f"(+{t_live:.1f}s liveness, 1 thread)"}
            line["checks"]["oracle_sample_equal"] = bool(np.array_equal(ov.view(np.int32), dev_v[:sample].view(np.int32)))
        print(json.dumps(line), flush=True)
    gp.close()
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
