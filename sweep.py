"""Throughput sweep of the CERAR pipeline on one GPU.

  python sweep.py [--quick] [--out FILE]

Points: d per worker in {2^18, 2^20, ..., 2^30} fp32, N in {4, 8, 16}, c in {N, 2N, 4N, 8N},
epsilon-construction with eps = 1e-3, i.i.d. N(0,1) gradients.  Every point runs in place
(the gradients are generated directly in the D rows of the workspace and the result
overwrites them), so the largest point (N=16, d=2^30, c=16) needs 137 GB.  Per point and
launch form: 3 warm-up and 5 timed aggregations (CUDA events around cerar_allreduce_sim,
median), the gradients are regenerated before every aggregation (outside the timed region).
Two launch forms: "round by round" (one launch per round, every hand-off through HBM: the
step bench.py reports) and "one call" (cerar_allreduce_sim as it stands: all rounds in one
launch, messages also handed on chip, so fewer bytes than the metric counts reach DRAM).

Reported: seconds per aggregation, algorithmic GB/s (N (8c+3N-8) p 4 bytes per
aggregation) and its fraction of the measured HBM copy bandwidth.  Points whose whole
state fits in the 126 MB L2 are marked: their "GB/s" is not an HBM figure.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="d in {2^20, 2^26} only")
    ap.add_argument("--out", default="")
    ap.add_argument("--eps", type=float, default=1e-3)
    ap.add_argument("--fused", action="store_true",
                    help="time cerar_allreduce_fused (ring on chip, out of place) next to the in-HBM pipeline "
                         "for the (N, c) it supports")
    ap.add_argument("--ring", action="store_true",
                    help="time the one-worker-per-rank calls (LocalRing: N workers with separate workspaces on "
                         "this one GPU, N launches per step) next to the all-workers-per-launch pipeline")
    args = ap.parse_args()

    import torch
    from paper_2609_23898_b200 import cerar, inputs

    root = os.path.dirname(os.path.abspath(__file__))
    peak = 6650.0
    pk = os.path.join(root, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        peak = float(json.load(open(pk))["hbm_gbs"])
    free, total = torch.cuda.mem_get_info()
    stream = torch.cuda.current_stream().cuda_stream
    exps = [20, 26] if args.quick else [18, 20, 22, 24, 26, 28, 30]
    rows = []
    if args.fused:
        return fused_table(args, exps, peak, free, stream)
    if args.ring:
        return ring_table(args, exps, peak, free, stream)
    print("| N | c | d | state MB | round by round: ms | GB/s | frac | launches | one call: ms | GB/s | frac | launches | note |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for N in (4, 8, 16):
        for mult in (1, 2, 4, 8):
            c = N * mult
            B = inputs.base_matrix(N, c, 0)
            note = ""
            try:
                plan = cerar.Plan.create(N, c, cerar.EPSILON, args.eps, B=B)
            except cerar.CerarError as e:
                # the encoders of this design do not fit fp32: time the kernels with
                # well-conditioned coefficients of the same shape instead
                rng = np.random.default_rng(0)
                L = c + N - 2
                U = [np.linalg.qr(rng.standard_normal((c, c)))[0] for _ in range(N)]
                R = [rng.standard_normal((L + 1, c)) / np.sqrt(L + 1) for _ in range(N)]
                plan = cerar.Plan.create_custom(N, c, U, R)
                note = "design overflows fp32: surrogate coefficients"
            for e in exps:
                d = 1 << e
                if d % c:
                    continue
                p = d // c
                ws_bytes = plan.workspace_bytes(d)
                if ws_bytes > free - (2 << 30):
                    print(f"| {N} | {c} | 2^{e} | {ws_bytes / 1e6:.0f} | - | - | - | - | - | - | - | - | "
                          f"skipped: needs {ws_bytes / 1e9:.1f} GB |")
                    continue
                ws = torch.empty(ws_bytes // 4, dtype=torch.float32, device="cuda")
                wstride = (c + N) * p
                dptr = ws.data_ptr() + 4 * N * p
                res = {}
                for form in ("round by round", "one call"):
                    # "round by round": one launch per round, every hand-off through HBM (the step bench.py
                    # reports); "one call": cerar_allreduce_sim as it stands (rounds in one launch)
                    cerar.cerar_set_tuning("rounds_one_launch_off", 1 if form == "round by round" else 0)
                    times = []
                    for rep in range(8):
                        for i in range(N):
                            ws[i * wstride + N * p:(i + 1) * wstride].normal_()
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        n0 = plan.launch_count()
                        e0.record()
                        plan.allreduce_sim(dptr, wstride, dptr, wstride, ws, d, 1.0 / N, stream)
                        e1.record()
                        torch.cuda.synchronize()
                        if rep >= 3:
                            times.append(e0.elapsed_time(e1))
                    plan.device_status(stream)
                    res[form] = (float(np.median(times)), plan.launch_count() - n0)
                cerar.cerar_set_tuning("rounds_one_launch_off", 0)
                ab = 4 * N * p * (8 * c + 3 * N - 8)
                (ms_r, l_r), (ms, launches) = res["round by round"], res["one call"]
                gbs_r, gbs = ab / ms_r / 1e6, ab / ms / 1e6
                l2 = "L2-resident" if ws_bytes < 100e6 else ""
                row = dict(N=N, c=c, d=d, state_mb=ws_bytes / 1e6, ms=ms, gbps=gbs, frac=gbs / peak, launches=launches,
                           ms_round_by_round=ms_r, gbps_round_by_round=gbs_r, frac_round_by_round=gbs_r / peak,
                           launches_round_by_round=l_r, note=", ".join(x for x in (note, l2) if x))
                rows.append(row)
                print(f"| {N} | {c} | 2^{e} | {ws_bytes / 1e6:.0f} | {ms_r:.3f} | {gbs_r:.0f} | {gbs_r / peak:.2f} | {l_r} | "
                      f"{ms:.3f} | {gbs:.0f} | {gbs / peak:.2f} | {launches} | {row['note']} |", flush=True)
                del ws
                torch.cuda.empty_cache()
            plan.destroy()
    if args.out:
        with open(args.out, "w") as f:
            json.dump(rows, f, indent=1)


def fused_table(args, exps, peak, free, stream):
    """Seconds per aggregation of the on-chip variant against the in-HBM pipeline (both out of place)."""
    import torch
    from paper_2609_23898_b200 import cerar, inputs
    print("| N | c | d | in-HBM pipeline ms | on-chip ms | speed-up | on-chip DRAM GB/s (8 N d bytes) |")
    print("|---|---|---|---|---|---|---|")
    rows = []
    for N in (4, 8, 16):
        for mult in (1, 2, 4, 8):
            c = N * mult
            B = inputs.base_matrix(N, c, 0)
            try:
                plan = cerar.Plan.create(N, c, cerar.EPSILON, args.eps, B=B)
            except cerar.CerarError:
                continue
            if not plan.fused_supported():
                plan.destroy()
                continue
            for e in exps:
                d = 1 << e
                p = d // c
                need = plan.workspace_bytes(d) + 8 * N * d
                if d % c or need > free - (2 << 30):
                    continue
                g = torch.empty(N * d, dtype=torch.float32, device="cuda").normal_()
                out = torch.empty(N * d, dtype=torch.float32, device="cuda")
                ws = torch.empty(plan.workspace_bytes(d) // 4, dtype=torch.float32, device="cuda")

                def med(f):
                    ts = []
                    for rep in range(8):
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record(); f(); e1.record(); torch.cuda.synchronize()
                        if rep >= 3:
                            ts.append(e0.elapsed_time(e1))
                    return float(np.median(ts))
                t_hbm = med(lambda: plan.allreduce_sim(g, d, out, d, ws, d, 1.0 / N, stream))
                t_chip = med(lambda: plan.allreduce_fused(g, d, out, d, d, 1.0 / N, stream))
                plan.device_status(stream)
                rows.append(dict(N=N, c=c, d=d, ms_hbm=t_hbm, ms_chip=t_chip))
                print(f"| {N} | {c} | 2^{e} | {t_hbm:.3f} | {t_chip:.3f} | {t_hbm / t_chip:.2f} | {8 * N * d / t_chip / 1e6:.0f} |",
                      flush=True)
                del g, out, ws
                torch.cuda.empty_cache()
            plan.destroy()
    if args.out:
        with open(args.out, "w") as f:
            json.dump(rows, f, indent=1)
    return 0


def ring_table(args, exps, peak, free, stream):
    """The rank-level calls on one GPU: same algorithmic bytes, N launches per step instead of one."""
    import torch
    from paper_2609_23898_b200 import cerar, inputs, ring
    print("| N | c | d | pipeline ms | rank-level ms (launches) | rank-level GB/s | frac | fused-rounds ms (launches) | "
          "fused GB/s | frac |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for (N, c) in ((4, 16), (8, 32), (8, 64)):
        rng = np.random.default_rng(0)
        L = c + N - 2
        U = [np.linalg.qr(rng.standard_normal((c, c)))[0] for _ in range(N)]
        R = [rng.standard_normal((L + 1, c)) / np.sqrt(L + 1) for _ in range(N)]
        plan = cerar.Plan.create_custom(N, c, U, R)
        for e in exps:
            d = 1 << e
            p = d // c
            if d % c or 4 * N * (2 * c + 2 * N + 1) * p + 8 * N * d > free - (2 << 30):
                continue
            g = torch.empty(N * d, dtype=torch.float32, device="cuda").normal_()
            out = torch.empty(N * d, dtype=torch.float32, device="cuda")
            ws = torch.empty(plan.workspace_bytes(d) // 4, dtype=torch.float32, device="cuda")
            r = ring.LocalRing(plan, d)
            grads = [g[i * d:(i + 1) * d] for i in range(N)]
            outs = [out[i * d:(i + 1) * d] for i in range(N)]

            def med(f):
                ts = []
                for rep in range(8):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(); f(); e1.record(); torch.cuda.synchronize()
                    if rep >= 3:
                        ts.append(e0.elapsed_time(e1))
                return float(np.median(ts))
            t_pipe = med(lambda: plan.allreduce_sim(g, d, out, d, ws, d, 1.0 / N, stream))
            t_ring = med(lambda: r.allreduce(grads, outs, 1.0 / N, stream))
            t_fus = med(lambda: r.allreduce(grads, outs, 1.0 / N, stream, fused=True))
            plan.device_status(stream)
            ab = 4 * N * p * (8 * c + 3 * N - 8)
            print(f"| {N} | {c} | 2^{e} | {t_pipe:.3f} | {t_ring:.3f} ({N * (L + 2)}) | {ab / t_ring / 1e6:.0f} | "
                  f"{ab / t_ring / 1e6 / peak:.2f} | {t_fus:.3f} ({2 * N + 1}) | {ab / t_fus / 1e6:.0f} | "
                  f"{ab / t_fus / 1e6 / peak:.2f} |", flush=True)
            del g, out, ws, r, grads, outs
            torch.cuda.empty_cache()
        plan.destroy()
    return 0


if __name__ == "__main__":
    sys.exit(main())
