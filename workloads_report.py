"""Throughput of vl_liveness + vl_verify on the five synthetic workloads, one line per workload.

    python workloads_report.py [--steps N]

For every workload: candidate verifications per second and operand checks per second with the rows
resident in device memory (CUDA events around `steps` repetitions of liveness + verify, after
warm-up), the same for vl_verify alone, the algorithmic bytes per second (2 bytes per operand
column + a 16-byte verdict per candidate) and their fraction of the measured copy bandwidth.  The
small workloads move kilobytes per call and are bound by launch latency: read their latency, not
their bandwidth fraction.  Workload 4 (256 independent programs) goes through vl_liveness_batch
and vl_verify_batch.  Also per workload: the time of one vl_resample_stats call over the verdict
arrays (launch-latency bound: three or more small kernels), the statistics it returns (test cases
solved, attempts summed and largest, Pass@1/10/100 counts), and the time of the early-exit loop
vl_verify_until_pass in batches of 100 rows (it stops after the first batch with a passing row),
and the times of vl_diagnose and vl_occupied_masks on one row, and vl_verify_dict over the rows of the
first program in dictionary form (its algorithmic bytes are 2 bytes per dictionary column + the verdict).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_17506_b200 import synth  # noqa: E402


def peak_gbs() -> float:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return 6650.0


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--workloads", default="1,2,3,4,5")
    args = ap.parse_args()
    import torch
    from paper_2506_17506_b200 import binding as vl

    peak = peak_gbs()
    stream = torch.cuda.current_stream()
    for idx in [int(x) - 1 for x in args.workloads.split(",")]:
        wl = synth.workload(idx)
        progs, gps, cands, outs = [], [], [], []
        for shape, seed in zip(wl.shapes, wl.seeds):
            p = synth.build_program(shape, seed)
            rows = np.empty((wl.K, p.pitch), dtype=np.uint16)
            synth.candidate_rows(p, wl.K, wl.fault_rate, seed, 0, wl.K, out=rows, chunk=256)
            progs.append(p)
            gps.append(vl.Program(p))
            cands.append(torch.from_numpy(rows.view(np.int16)).cuda().view(torch.uint16))
            outs.append(torch.empty((wl.K, 4), dtype=torch.int32, device="cuda"))

        def liveness():
            if len(gps) == 1:
                gps[0].vl_liveness(stream)
            else:
                vl.vl_liveness_batch(gps, stream)

        def verify():
            if len(gps) == 1:
                gps[0].vl_verify(cands[0], outs[0], stream)
            else:
                vl.vl_verify_batch(gps, cands, outs, stream)

        for _ in range(3):
            liveness()
            verify()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        ev[0].record(stream)
        for _ in range(args.steps):
            liveness()
            verify()
        ev[1].record(stream)
        ev[2].record(stream)
        for _ in range(args.steps):
            verify()
        ev[3].record(stream)
        torch.cuda.synchronize()
        for gp in gps:
            gp.vl_verify_status(stream)
        # re-sampling statistics over the verdicts just written, and the early-exit loop
        n = len(outs)
        stats = torch.zeros((n, 2), dtype=torch.int64, device="cuda")
        summ = torch.zeros(4 + vl.VL_MAX_PASS_AT, dtype=torch.int64, device="cuda")
        import ctypes as C
        op = (C.c_void_p * n)(*[o.data_ptr() for o in outs])
        Ks = (C.c_uint64 * n)(*[o.shape[0] for o in outs])
        kk = (C.c_uint32 * 3)(1, 10, 100)
        sp = C.c_void_p(stream.cuda_stream)

        def resample():
            rc = vl._lib.vl_resample_stats(0, n, op, Ks, 3, kk, stats.data_ptr(), summ.data_ptr(), sp)
            assert rc == vl.VL_OK, rc

        for _ in range(3):
            resample()
        er = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        er[0].record(stream)
        for _ in range(args.steps):
            resample()
        er[1].record(stream)
        torch.cuda.synchronize()
        _, summary = vl.vl_resample_stats(outs, (1, 10, 100), stream=stream)
        gps[0].vl_verify_until_pass(cands[0], 100, outs[0], stream)
        er[2].record(stream)
        for _ in range(args.steps):
            _, rows_done, first_pass = gps[0].vl_verify_until_pass(cands[0], 100, outs[0], stream)
        er[3].record(stream)
        torch.cuda.synchronize()
        # diagnostics of the first row of the first program
        rec = torch.zeros((4096, 3), dtype=torch.int32, device="cuda")
        cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
        kinds = torch.zeros(progs[0].n_instrs, dtype=torch.uint8, device="cuda")
        hist = torch.zeros(progs[0].B, dtype=torch.int64, device="cuda")

        def diagnose():
            rc = vl._lib.vl_diagnose(gps[0].handle, cands[0].data_ptr(), 4096, rec.data_ptr(), cnt.data_ptr(),
                                     kinds.data_ptr(), hist.data_ptr(), sp)
            assert rc == vl.VL_OK, rc

        for _ in range(3):
            diagnose()
        ed = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        ed[0].record(stream)
        for _ in range(args.steps):
            diagnose()
        ed[1].record(stream)
        torch.cuda.synchronize()
        Wm = (progs[0].P + 31) // 32
        masks = torch.zeros((progs[0].n_instrs, Wm), dtype=torch.int32, device="cuda")

        def occupied():
            rc = vl._lib.vl_occupied_masks(gps[0].handle, cands[0].data_ptr(), masks.data_ptr(), sp)
            assert rc == vl.VL_OK, rc

        for _ in range(3):
            occupied()
        eo = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        eo[0].record(stream)
        for _ in range(args.steps):
            occupied()
        eo[1].record(stream)
        torch.cuda.synchronize()
        # the same candidates in dictionary form (one column per (block, vreg of the block)): first program
        layout = synth.dict_layout(progs[0])
        d_host = synth.dict_rows(progs[0], cands[0].cpu().numpy().view(np.uint16), layout)
        d_rows = torch.from_numpy(d_host.view(np.int16)).cuda().view(torch.uint16)
        d_out = torch.empty((wl.K, 4), dtype=torch.int32, device="cuda")
        for _ in range(3):
            gps[0].vl_verify_dict(d_rows, d_out, stream)
        edd = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        edd[0].record(stream)
        for _ in range(args.steps):
            gps[0].vl_verify_dict(d_rows, d_out, stream)
        edd[1].record(stream)
        torch.cuda.synchronize()
        dict_ms = edd[0].elapsed_time(edd[1]) / args.steps
        dict_bytes = (2 * d_host.shape[1] + 16) * wl.K
        occupied_us = eo[0].elapsed_time(eo[1]) / args.steps * 1e3
        diagnose_us = ed[0].elapsed_time(ed[1]) / args.steps * 1e3
        resample_us = er[0].elapsed_time(er[1]) / args.steps * 1e3
        until_ms = er[2].elapsed_time(er[3]) / args.steps
        step_ms = ev[0].elapsed_time(ev[1]) / args.steps
        verify_ms = ev[2].elapsed_time(ev[3]) / args.steps
        n_cand = wl.K * len(progs)
        n_checks = sum(p.n_operands for p in progs) * wl.K
        n_bytes = sum(2 * p.pitch + 16 for p in progs) * wl.K
        n_pass = sum(int((o[:, 0] == vl.VL_PASS).sum()) for o in outs)
        print(json.dumps({
            "workload": idx + 1, "name": wl.name, "programs": len(progs), "candidates": n_cand,
            "operand_columns": int(sum(p.n_operands for p in progs)), "rows_passing": n_pass,
            "step_ms": step_ms, "verify_ms": verify_ms,
            "verifications_per_sec": n_cand / (step_ms * 1e-3),
            "operand_checks_per_sec": n_checks / (step_ms * 1e-3),
            "verify_only_verifications_per_sec": n_cand / (verify_ms * 1e-3),
            "verify_only_gb_per_sec": n_bytes / (verify_ms * 1e-3) / 1e9,
            "verify_only_frac_of_measured_copy_peak": n_bytes / (verify_ms * 1e-3) / 1e9 / peak,
            "resample_stats_us": resample_us, "resample_summary": summary,
            "until_pass_batch100_ms": until_ms, "until_pass_rows_checked": rows_done,
            "until_pass_first_passing_row": first_pass,
            "diagnose_one_row_us": diagnose_us,
            "occupied_masks_one_row_us": occupied_us,
            "dict_form_first_program": {"columns": int(len(layout[1])), "verify_dict_ms": dict_ms,
                                        "verifications_per_sec": wl.K / (dict_ms * 1e-3),
                                        "gb_per_sec": dict_bytes / (dict_ms * 1e-3) / 1e9,
                                        "frac_of_measured_copy_peak": dict_bytes / (dict_ms * 1e-3) / 1e9 / peak},
        }), flush=True)
        for gp in gps:
            gp.close()
    return 0


if __name__ == "__main__":
    sys.exit(main())
