#!/usr/bin/env python
"""Benchmark of the CERAR hot path (encode + L ring rounds + decode) on B200.

One "step" is one aggregation: every logical worker's gradient is encoded, the
L = c+N-2 ring rounds run, and every worker decodes its approximate mean.
Default workload: the third configuration (N=8, c=32, epsilon-construction
eps=1e-2, d=1,414,647,808 fp32 per worker, 24 layer-shaped Gaussian blocks),
the "sim time at d=1.4B" point of the metric.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is algorithmic GB/s over the whole job:
N_workers*(8c+3N-8)*p*4 bytes per aggregation (every logical buffer touched once
per use) divided by the device time per step, summed over ranks.  With more
than one GPU every rank runs its own replica of the workload (the path has no
exchange step: positions are independent), i.e. weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

def _metric_name():
    """The headline metric as the baseline file of this repository words it."""
    try:
        with open(os.path.join(ROOT, "BASELINE.json")) as f:
            return json.load(f)["metric"]
    except (OSError, KeyError, ValueError):
        return "CERAR encode+rounds+decode HBM GB/s vs B200 peak; sim time at d=1.4B"


METRIC = _metric_name()
UNIT = "GB/s"
# DRAM bytes per launch against algorithmic bytes per launch, from ncu captures of a smaller case of the
# same kernels (N=8, c=32, p=1 Mi; profiles/dram_traffic_steady_state_N8_c32_p1M.md): means over
# consecutive launches with the caches left alone between them (--cache-control none), so that what one
# launch leaves dirty in L2 is counted when the next one evicts it.  The contractions' traffic grows in
# proportion to the positions (encode 0.997, decode 1.019 of the algorithmic bytes: decode also fetches the
# stale slot between y_L and y_{L+1}).  A ring round finds the newest part of the previous round's message
# still in L2: 22.8 MB per launch at that size, a window of L2's size that does not grow with p, so it is
# subtracted rather than scaled.
NCU_TRAFFIC_OVER_ALGORITHMIC = {"round_kernel": 1.0, "encode": 0.997, "decode": 1.019}
NCU_L2_WINDOW_BYTES = {"round_kernel": 22.8e6, "encode": 0.0, "decode": 0.0}
NCU_TRAFFIC_SOURCE = ("ncu dram__bytes_read.sum + dram__bytes_write.sum, steady state over consecutive launches at "
                      "N=8, c=32, p=2^20; contractions scaled by positions, rounds: algorithmic bytes minus the "
                      "22.8 MB per launch that L2 served there")


def algorithmic_bytes(N, c, p):
    """Per aggregation, all workers: encode 2c, rounds 4c+2N-7, decode 2c+N-1 row
    passes of p fp32 per worker."""
    enc = 2 * c
    rnd = 4 * c + 2 * N - 7
    dec = 2 * c + N - 1
    return {"encode": 4 * N * p * enc, "rounds": 4 * N * p * rnd, "decode": 4 * N * p * dec,
            "total": 4 * N * p * (enc + rnd + dec)}


def round_bytes(N, c, p, k):
    terms = (1 if k >= 2 else 0) + (1 if k - 1 >= N else 0) + (1 if k <= c else 0) + 1
    return 4 * N * p * terms


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def wait_first_sample(self, timeout=3.0):
        t0 = time.time()
        while self.p is not None and time.time() - t0 < timeout:
            if os.path.getsize(self.f.name) > 0:
                return
            time.sleep(0.05)

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f:
            t = [x.strip() for x in line.split(",")]
            if len(t) < 7:
                continue
            try:
                sm.append(float(t[0])); mx.append(float(t[1])); power.append(float(t[2]))
            except ValueError:
                continue
            for n, v in zip(names, t[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            # under load = samples in the upper half of the power range
            thr = (max(power) + min(power)) / 2 if power else 0
            loaded = [s for s, w in zip(sm, power) if w >= thr] or sm
            out.update(sm_mhz=float(np.median(loaded)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=float(max(power)))
        return out


def build_design_oracle(cfg, B):
    from oracle import designs as Dz
    if cfg["kind"] == "vandermonde":
        return Dz.vandermonde(cfg["N"], cfg["c"], cfg["param"])
    if cfg["kind"] == "epsilon":
        return Dz.epsilon(cfg["N"], cfg["c"], cfg["param"], B)
    return Dz.kappa_constrained(cfg["N"], cfg["c"], cfg["param"], B)


def oracle_step(des, g_sub, scale):
    from oracle import protocol as P
    return P.allreduce([x for x in g_sub], des.U, des.R, scale)


def cpu_baseline(cfg, des, p_sample, seed=0, one_thread=False, g=None, keep=None):
    """Times the oracle, as it stands, on the first p_sample positions of the workload (all N
    workers, all c chunks).  g: those positions of the device's gradients, (N, c*p_sample) fp32, read
    back from the GPU (default: the same recipe drawn with numpy).  keep: a dict that receives the
    oracle's result (for the parity block)."""
    from paper_2609_23898_b200 import inputs
    N, c = cfg["N"], cfg["c"]
    kw = {"std": cfg["std"]} if "std" in cfg else {}
    if g is None:
        g = inputs.gradients_numpy(N, c * p_sample, cfg["workload"], seed=seed, **kw)
    g = g.astype(np.float64)
    t0 = time.perf_counter()
    res_o = oracle_step(des, g, 1.0 / N)
    dt = time.perf_counter() - t0
    if keep is not None:
        keep.update(res=res_o, g=g)
    ab = algorithmic_bytes(N, c, p_sample)["total"]
    try:
        from threadpoolctl import threadpool_info
        thr = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        thr = os.cpu_count() or 1
    res = {"value": ab / dt / 1e9, "unit": UNIT, "cores": int(thr), "kind": "oracle",
           "sample": f"first {p_sample} of p={cfg['d'] // c} positions, all {N} workers and {c} chunks; "
                     f"{dt:.2f} s of numpy fp64", "seconds": dt}
    if one_thread:
        # the same oracle held to one BLAS thread, on an eighth of the sample
        try:
            from threadpoolctl import threadpool_limits
            p1 = max(1, p_sample // 8)
            g1 = np.ascontiguousarray(g.reshape(N, c, p_sample)[:, :, :p1]).reshape(N, -1)
            with threadpool_limits(limits=1):
                t0 = time.perf_counter()
                oracle_step(des, g1, 1.0 / N)
                dt1 = time.perf_counter() - t0
            res["value_1_thread"] = algorithmic_bytes(N, c, p1)["total"] / dt1 / 1e9
            res["sample_1_thread"] = f"first {p1} positions, {dt1:.2f} s"
        except Exception:
            pass
    return res


def parity_block(des, kept, par_dev, p_sample, p_par, scale):
    """GPU against the oracle on the first p_par positions, part of the cpu_baseline leg (the
    oracle's results are those of its timed run; one more oracle pass with the coefficients rounded to
    binary32, as the device holds them, separates coefficient rounding from kernel error).  Next to
    kappa 2^-24 the block carries the a-priori fp32 rounding bound u (c+L) || |G^(i)| |M_i| |R_i| ||_F
    / || g_hat_i || (worst worker) and, for the decode alone, residual over bound
    || out - s Y_dev Rf || / (u (L+1) s || |Y_dev| |Rf| ||_F), which does not grow with kappa."""
    from oracle import protocol as P
    N, c = des.N, des.c
    L = c + N - 2
    u = 2.0 ** -24
    res, g = kept["res"], kept["g"]
    p_dev = par_dev["Y"].shape[2]                      # positions read back from the device (>= p_par)
    par_dev = {"Y": np.ascontiguousarray(par_dev["Y"][:, :, :p_par]),
               "out": np.ascontiguousarray(par_dev["out"].reshape(N, c, p_dev)[:, :, :p_par]).reshape(N, -1)}
    pick = lambda v, rows: np.ascontiguousarray(v.reshape(rows, p_sample)[:, :p_par])
    Y_ora = np.stack([res["Y"][i][:p_par].T for i in range(N)])                       # (N, L+1, p_par)
    out_ora = [pick(res["out"][i], c).reshape(-1) for i in range(N)]
    g_par = [pick(g[i], c).reshape(-1) for i in range(N)]
    Uf = [np.asarray(m, np.float32).astype(np.float64) for m in des.U]
    Rf = [np.asarray(m, np.float32).astype(np.float64) for m in des.R]
    res_f = P.allreduce(g_par, Uf, Rf, scale)
    G = [P.chunk_matrix(x, c) for x in g_par]
    kap = max(P.kappa2(P.m_matrix(des.U, i)) for i in range(N))
    rel_out = rel_out_f = bound_rel = e2e_ratio = dec_ratio = 0.0
    for i in range(N):
        od = par_dev["out"][i].astype(np.float64)
        ref = np.linalg.norm(res_f["out"][i])
        mag = np.abs(P.stacked_gradients(G, i)) @ np.abs(P.m_matrix(Uf, i)) @ np.abs(Rf[i])
        bound = u * (c + L) * scale * np.linalg.norm(mag)
        err_f = np.linalg.norm(od - res_f["out"][i])
        Yd = par_dev["Y"][i].astype(np.float64).T
        dec_bound = u * (L + 1) * scale * np.linalg.norm(np.abs(Yd) @ np.abs(Rf[i]))
        rel_out = max(rel_out, P.rel_l2(od, out_ora[i]))
        rel_out_f = max(rel_out_f, err_f / ref)
        bound_rel = max(bound_rel, bound / ref)
        e2e_ratio = max(e2e_ratio, err_f / bound)
        dec_ratio = max(dec_ratio, np.linalg.norm(od - P.unchunk(scale * (Yd @ Rf[i]))) / dec_bound)
    exact = P.exact_sum(g_par) * scale
    return {"sampled_positions": int(p_par), "which": "the first positions of every chunk, all workers",
            "rel_l2_Y": P.rel_l2(par_dev["Y"], Y_ora), "rel_l2_out": rel_out,
            "rel_l2_out_vs_fp32_rounded_coefficients": rel_out_f,
            "kappa_M": kap, "kappa_times_2^-24": kap * u, "apriori_bound_rel": bound_rel,
            "end_to_end_residual_over_bound": e2e_ratio, "decode_residual_over_bound": dec_ratio,
            "rel_l2_oracle_vs_exact_mean": max(P.rel_l2(out_ora[i], exact) for i in range(N)),
            "note": "computed outside the timed regions from the last timed aggregation; stages without "
                    "cancellation (Y) agree to fp32 roundoff, the decoded output of an ill-conditioned design "
                    "carries roundoff amplified by about kappa and is held to its a-priori bound instead"}


def run_reference(args, cfg):
    """--impl reference: the CPU oracle timed on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_23898_b200 import inputs
    N, c, d = cfg["N"], cfg["c"], cfg["d"]
    B = inputs.base_matrix(N, c, 0)
    des = build_design_oracle(cfg, B)
    # a bounded sample per step, sized so that the whole run (K steps + W short warm-ups) stays
    # within a few minutes whatever K is: about ten steps' worth of --ref-positions in total
    p_sample = min(d // c, args.ref_positions, max(4096, (10 * args.ref_positions) // max(1, args.steps)))
    for _ in range(args.warmup):
        cpu_baseline(cfg, des, max(1, p_sample // 8))
    times, base = [], None
    for _ in range(args.steps):
        base = cpu_baseline(cfg, des, p_sample)
        times.append(base["seconds"])
    dt = float(np.mean(times))
    val = algorithmic_bytes(N, c, p_sample)["total"] / dt / 1e9
    base["value"] = val
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(args.workload, cfg), "sample_positions": p_sample},
            "cpu_baseline": base,
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Slowest rank's time (the contract's max over ranks)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(bytes_per_replica: int, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank moves the same algorithmic bytes; GB/s of the whole job."""
    return world * bytes_per_replica / (ms_per_step * 1e-3) / 1e9


def workload_name(key, cfg):
    return (f"{key}: N={cfg['N']} c={cfg['c']} {cfg['kind']}({cfg['param']:g}) d={cfg['d']} fp32/worker "
            f"{cfg['workload']} gradients")


THERMAL = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}


def time_steps(plan, grads, g_stride, ws, out, o_stride, d, scale, K, W, stream, gpu_index=None, sync=None):
    """W warm-ups, then the timed region: K steps, each the C-ABI sequence cerar_encode,
    cerar_ring_round(1..L), cerar_decode, with a CUDA event after every phase (encode | the L round
    launches | decode; an event after every launch would keep consecutive launches apart) and, if
    gpu_index is given, the clocks sampled alongside.  Returns the per-phase means, this rank's
    step times and the total device time of the K steps (ms)."""
    import torch
    L = plan.L
    sync = sync or torch.cuda.synchronize
    sampler = ClockSampler(gpu_index) if gpu_index is not None else None
    for _ in range(W):                                  # the timed sequence itself, without the events
        plan.encode(grads, g_stride, ws, d, stream)
        for k in range(1, L + 1):
            plan.ring_round(ws, d, k, stream)
        plan.decode(ws, out, o_stride, d, scale, stream)
    torch.cuda.synchronize()
    plan.device_status(stream)
    if sampler:
        sampler.wait_first_sample()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    sync()
    launches0 = plan.launch_count()
    for s in range(K):
        e = ev[s]
        e[0].record()
        plan.encode(grads, g_stride, ws, d, stream)
        e[1].record()
        for k in range(1, L + 1):
            plan.ring_round(ws, d, k, stream)
        e[2].record()
        plan.decode(ws, out, o_stride, d, scale, stream)
        e[3].record()
    sync()
    launches = plan.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    plan.device_status(stream)
    return {"total_ms": ev[0][0].elapsed_time(ev[K - 1][3]),
            "enc_ms": float(np.mean([e[0].elapsed_time(e[1]) for e in ev])),
            "rounds_ms": float(np.mean([e[1].elapsed_time(e[2]) for e in ev])),
            "dec_ms": float(np.mean([e[2].elapsed_time(e[3]) for e in ev])),
            "step_ms": [e[0].elapsed_time(e[3]) for e in ev],
            "launches": int(launches), "clocks": clocks}


def time_one_call(plan, grads, g_stride, ws, out, o_stride, d, scale, K, stream, sync=None):
    """The same K aggregations through cerar_allreduce_sim with one event pair around all of them."""
    import torch
    sync = sync or torch.cuda.synchronize
    for _ in range(3):
        plan.allreduce_sim(grads, g_stride, out, o_stride, ws, d, scale, stream)
    sync()
    o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = plan.launch_count()
    o0.record()
    for _ in range(K):
        plan.allreduce_sim(grads, g_stride, out, o_stride, ws, d, scale, stream)
    o1.record()
    sync()
    plan.device_status(stream)
    return o0.elapsed_time(o1), (plan.launch_count() - n0) // K


def time_graph_replay(plan, grads, g_stride, ws, out, o_stride, d, scale, K):
    """The same step (cerar_encode, L x cerar_ring_round, cerar_decode: every hand-off through memory) captured
    once in a CUDA graph and replayed K times: what a caller gets who takes the host out of a launch-bound
    loop.  Returns ms per aggregation, or None if the capture is refused."""
    import torch
    try:
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            def step():
                plan.encode(grads, g_stride, ws, d, st.cuda_stream)
                for k in range(1, plan.L + 1):
                    plan.ring_round(ws, d, k, st.cuda_stream)
                plan.decode(ws, out, o_stride, d, scale, st.cuda_stream)
            step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=st):
                step()
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for _ in range(K):
                graph.replay()
            e1.record(st)
            torch.cuda.synchronize()
            plan.device_status(st.cuda_stream)
            return e0.elapsed_time(e1) / K
    except Exception:
        return None


SWEEP_CORNERS = [(16, 128, 1 << 24), (16, 128, 1 << 28), (4, 16, 1 << 26)]


def other_configs(headline_key, peak, gpu_index, stream, steps=20, warmup=3, only=()):
    """The remaining configurations at full size and a few corners of the sweep, each timed like the
    headline (cerar_encode, L x cerar_ring_round, cerar_decode with an event after every phase, then
    the one-call form), after the headline's buffers were freed.  The configurations run out of place,
    the sweep corners in place (as the sweep does: gradients in the D rows, result over them)."""
    import torch
    from paper_2609_23898_b200 import cerar, inputs
    kinds = {"vandermonde": cerar.VANDERMONDE, "epsilon": cerar.EPSILON, "kappa": cerar.KAPPA}
    jobs = [(k, dict(inputs.CONFIGS[k]), False) for k in ("cfg4", "cfg2", "cfg1", "cfg3") if k != headline_key]
    jobs += [(f"sweep_N{N}_c{c}_d2^{d.bit_length() - 1}",
              dict(N=N, c=c, kind="epsilon", param=1e-3, d=d, workload="normal", std=1.0), True) for N, c, d in SWEEP_CORNERS]
    out_all = {}
    dev = torch.device("cuda", torch.cuda.current_device())
    for key, cfg, inplace in jobs:
        if only and key not in only:
            continue
        N, c, d = cfg["N"], cfg["c"], cfg["d"]
        p, L = d // c, c + N - 2
        need = 4 * N * ((c + N) * p + (0 if inplace else 2 * d))
        if need > 0.9 * torch.cuda.mem_get_info()[0]:
            out_all[key] = {"skipped": f"needs {need / 1e9:.1f} GB of device memory"}
            continue
        try:
            B = inputs.base_matrix(N, c, 0)
            plan = cerar.Plan.create(N, c, kinds[cfg["kind"]], cfg["param"], B=B)
            ws = torch.empty(plan.workspace_bytes(d) // 4, dtype=torch.float32, device=dev)
            kw = {"std": cfg["std"]} if "std" in cfg else {}
            if inplace:
                wv = ws.view(N, c + N, p)
                rows = [wv[i, N:, :].reshape(-1) for i in range(N)]             # views of the D rows
                inputs.fill_gradients_torch(rows, cfg["workload"], seed=0, **kw)
                g_ptr = o_ptr = ws.data_ptr() + 4 * N * p
                g_stride = o_stride = (c + N) * p
                grads = outb = None
            else:
                grads = torch.empty(N * d, dtype=torch.float32, device=dev)
                inputs.fill_gradients_torch([grads[i * d:(i + 1) * d] for i in range(N)], cfg["workload"], seed=0, **kw)
                outb = torch.empty(N * d, dtype=torch.float32, device=dev)
                g_ptr, o_ptr, g_stride, o_stride = grads.data_ptr(), outb.data_ptr(), d, d
            ab = algorithmic_bytes(N, c, p)
            m = time_steps(plan, g_ptr, g_stride, ws, o_ptr, o_stride, d, 1.0 / N, steps, warmup, stream, gpu_index)
            ms = m["total_ms"] / steps
            one_ms, n_one = time_one_call(plan, g_ptr, g_stride, ws, o_ptr, o_stride, d, 1.0 / N, steps, stream)
            one_ms /= steps
            gbps = lambda b, t: b / t / 1e6
            out_all[key] = {
                "workload": workload_name(key, cfg), "buffers": "in place" if inplace else "out of place",
                "steps": steps, "warmup": warmup, "ms_per_step": ms, "value": gbps(ab["total"], ms), "unit": UNIT,
                "frac": gbps(ab["total"], ms) / peak, "gpu_launches": m["launches"],
                "per_kernel_GBps": {"encode": gbps(ab["encode"], m["enc_ms"]), "round_kernel": gbps(ab["rounds"], m["rounds_ms"]),
                                    "decode": gbps(ab["decode"], m["dec_ms"])},
                "per_kernel_frac": {"encode": gbps(ab["encode"], m["enc_ms"]) / peak,
                                    "round_kernel": gbps(ab["rounds"], m["rounds_ms"]) / peak,
                                    "decode": gbps(ab["decode"], m["dec_ms"]) / peak},
                "one_call": {"ms_per_step": one_ms, "value": gbps(ab["total"], one_ms), "frac_effective": gbps(ab["total"], one_ms) / peak,
                             "launches_per_step": int(n_one)},
                "l2": "inputs larger than L2" if 4 * N * (c + N) * p > 2.6e8 else "state fits in L2: launch-bound, not an HBM figure",
                "clocks": m["clocks"]}
            if ms < 0.5:                                 # launch-bound sizes: the same step replayed from a CUDA graph
                g_ms = time_graph_replay(plan, g_ptr, g_stride, ws, o_ptr, o_stride, d, 1.0 / N, steps)
                if g_ms is not None:
                    out_all[key]["graph_replay"] = {"ms_per_step": g_ms, "value": gbps(ab["total"], g_ms),
                                                    "note": "the round-by-round step captured in a CUDA graph and replayed"}
            del plan, ws, grads, outb
        except Exception as exc:                         # one failing point must not cost the headline
            out_all[key] = {"error": f"{type(exc).__name__}: {exc}"}
        torch.cuda.empty_cache()
    return out_all


def ring_block(world, rank, dev, *, plan=None, d=None, reps=3, timer=None):
    """N > 1 only: one aggregation family with ONE WORKER PER RANK (N = world, c = 4 world,
    d = 2^28 per worker, epsilon-construction), next to torch.distributed's all-reduce of the same
    gradient: (a) ring.SendRecvRing, messages moved by isend / irecv of the process group; (b)
    ring.DistributedRing, messages stored straight into the neighbour's workspace (peer-mapped symmetric
    memory), one device-side barrier per round; (c) the same with all rounds in one kernel per rank that
    orders itself against its neighbours tile by tile.  The three must give the same bits (the message
    arithmetic is the same kernel code); their parity with the oracle is the business of the tests.
    plan / d / timer are for the CPU test, which drives this function with stand-ins on gloo ranks."""
    import torch
    import torch.distributed as dist
    from paper_2609_23898_b200 import cerar, inputs, ring
    N = world
    on_gpu = dev.type == "cuda"
    if plan is None:
        c = 4 * N
        plan = cerar.Plan.create(N, c, cerar.EPSILON, 1e-2, B=inputs.base_matrix(N, c, 0))
    c, L = plan.c, plan.L
    d = d if d is not None else (1 << 28) // c * c
    p = d // c
    stream = torch.cuda.current_stream().cuda_stream if on_gpu else 0
    grad = torch.empty(d, dtype=torch.float32, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(7000 + rank)
    grad.normal_(0.0, 1.0, generator=gen)

    def default_timer(fn):
        """ms per call, max over ranks: barrier, synchronize, `reps` calls between two CUDA events."""
        fn()                                                     # warm-up
        dist.barrier()
        if on_gpu:
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            dist.barrier()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps
        else:
            t0 = time.perf_counter()
            for _ in range(reps):
                fn()
            dist.barrier()
            ms = (time.perf_counter() - t0) * 1e3 / reps
        return max_over_ranks(ms, world, dev if on_gpu else None)
    timer = timer or default_timer

    block = {"workers": N, "c": c, "L": L, "d": d, "design": "epsilon(0.01)", "reps": reps,
             "bytes_over_the_link_per_rank": 4 * p * L, "all_reduce_bytes_per_rank_ring": int(2 * (N - 1) / N * 4 * d),
             "status": "unmeasured on hardware until a multi-GPU run reports it" if not on_gpu else "measured"}
    ref = grad.clone()
    block["all_reduce_ms"] = timer(lambda: dist.all_reduce(ref.copy_(grad)))
    mean = ref.copy_(grad)
    dist.all_reduce(mean)
    mean = mean / N
    outs = {}
    forms = [("sendrecv", lambda: ring.SendRecvRing(plan, d, device=dev), {}),
             ("peer_round_by_round", lambda: ring.DistributedRing(plan, d, device=dev), {"fused": False}),
             ("peer_fused_rounds", None, {"fused": True})]
    drv = None

    def all_ranks_ok(ok: bool) -> bool:
        """A form runs only if its set-up worked on EVERY rank: a rank that skipped the timed calls while the
        others entered their barriers would leave them waiting."""
        flag = torch.tensor([1 if ok else 0], dtype=torch.int32, device=dev)
        dist.all_reduce(flag, op=dist.ReduceOp.MIN)
        return bool(flag.item())

    for name, make, kw in forms:
        err = None
        try:
            drv = make() if make is not None else drv
            if drv is None:
                err = "the driver of the form before this one could not be created"
        except Exception as exc:
            err = f"{type(exc).__name__}: {exc}"
            if make is not None:
                drv = None
        if not all_ranks_ok(err is None):
            block[name] = {"error": err or "set-up failed on another rank"}
            continue
        try:
            out = torch.empty(d, dtype=torch.float32, device=dev)
            ms = timer(lambda: drv.allreduce(grad, out, 1.0 / N, stream, **kw))
            if on_gpu:
                torch.cuda.synchronize()
                plan.device_status(stream)
            outs[name] = out
            block[name] = {"ms_per_aggregation": ms, "ratio_to_all_reduce": ms / block["all_reduce_ms"],
                           "link_GBps_per_rank": 4 * p * L / ms / 1e6}
        except Exception as exc:
            block[name] = {"error": f"{type(exc).__name__}: {exc}"}
    names = list(outs)
    block["identical_results"] = bool(names) and all(torch.equal(outs[names[0]], outs[n]) for n in names[1:])
    if names:
        o = outs[names[0]]
        block["rel_l2_vs_all_reduce_mean"] = float((o - mean).norm() / mean.norm())
    return block


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--d", type=int, default=0, help="override d per worker (multiple of c)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity", action="store_true", help="skip the parity block of the cpu_baseline leg")
    ap.add_argument("--parity-positions", type=int, default=1 << 16)
    ap.add_argument("--no-configs", action="store_true", help="skip the other configurations and the sweep corners")
    ap.add_argument("--configs", default="", help="comma-separated subset of the configs block's keys (default: all)")
    ap.add_argument("--no-ring", action="store_true", help="N > 1: skip the one-worker-per-rank ring block")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--ref-positions", type=int, default=1 << 20)
    ap.add_argument("--kernel-mode", type=int, default=0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2609_23898_b200 import inputs
    cfg = dict(inputs.CONFIGS[args.workload])
    if args.d:
        cfg["d"] = args.d
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_23898_b200 import cerar

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    N, c, d = cfg["N"], cfg["c"], cfg["d"]
    p, L = d // c, c + N - 2
    scale = 1.0 / N
    B = inputs.base_matrix(N, c, 0)
    kinds = {"vandermonde": cerar.VANDERMONDE, "epsilon": cerar.EPSILON, "kappa": cerar.KAPPA}
    plan = cerar.Plan.create(N, c, kinds[cfg["kind"]], cfg["param"], B=B)
    plan.set_kernel_mode(args.kernel_mode)

    grads = torch.empty(N * d, dtype=torch.float32, device=dev)
    kw = {"std": cfg["std"]} if "std" in cfg else {}
    inputs.fill_gradients_torch([grads[i * d:(i + 1) * d] for i in range(N)], cfg["workload"], seed=rank, **kw)
    ws = torch.empty(plan.workspace_bytes(d) // 4, dtype=torch.float32, device=dev)
    out = torch.empty(N * d, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    ab = algorithmic_bytes(N, c, p)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K = args.steps
    gi = local_rank if rank == 0 else None
    m = time_steps(plan, grads, d, ws, out, d, d, scale, K, args.warmup, stream, gi, sync_all)
    remeasured = False
    if m["clocks"] and THERMAL & set(m["clocks"].get("reasons", [])) and world == 1:
        # a thermal or hardware slowdown during the timed region: the number is not usable; once more
        first = m["clocks"]
        m = time_steps(plan, grads, d, ws, out, d, d, scale, K, args.warmup, stream, gi, sync_all)
        m["clocks"]["first_attempt_reasons"] = first["reasons"]
        remeasured = True
    launches, clocks = m["launches"], m["clocks"]
    total_ms, enc_ms, dec_ms, rounds_all_ms, step_ms = m["total_ms"], m["enc_ms"], m["dec_ms"], m["rounds_ms"], m["step_ms"]
    ms_per_step = max_over_ranks(total_ms, world, dev) / K
    value = whole_job_value(ab["total"], world, ms_per_step)
    # device results of the last timed aggregation on the first positions of every row, for the parity
    # block (compared with the oracle's run of the cpu_baseline leg, outside every timed region)
    p_par = min(p, args.parity_positions)
    rows_y = torch.tensor(list(range(L)) + [L + 1], device=dev)
    par_dev = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.no_parity:
        par_dev = {"Y": ws.view(N, c + N, p)[:, rows_y, :p_par].cpu().numpy(),
                   "out": out.view(N, c, p)[:, :, :p_par].reshape(N, -1).cpu().numpy()}

    peak, peak_kind = load_peaks()
    rounds_bytes = sum(round_bytes(N, c, p, k) for k in range(1, L + 1))
    assert rounds_bytes == ab["rounds"]
    rounds_ms = rounds_all_ms
    shares = {"round_kernel": rounds_ms, "encode": enc_ms, "decode": dec_ms}
    dominant = max(shares, key=shares.get)
    dom_bytes = {"round_kernel": ab["rounds"] / L, "encode": ab["encode"], "decode": ab["decode"]}[dominant]
    dom_ms = {"round_kernel": rounds_ms / L, "encode": enc_ms, "decode": dec_ms}[dominant]
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    traffic = NCU_TRAFFIC_OVER_ALGORITHMIC[dominant] * dom_bytes - min(NCU_L2_WINDOW_BYTES[dominant], 0.25 * dom_bytes)
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "traffic_source": NCU_TRAFFIC_SOURCE,
                # the fraction of the HBM roofline proper: DRAM bytes (not algorithmic bytes) over time over peak;
                # `achieved` / `frac` count every logical buffer once per use and can exceed 1 where L2 serves a re-read
                "dram_GBps": traffic / (dom_ms * 1e-3) / 1e9, "dram_frac": traffic / (dom_ms * 1e-3) / 1e9 / peak,
                "frac_of_nominal_8TBps": achieved / 8000.0, "whole_path_frac_of_nominal_8TBps": value / world / 8000.0,
                "algorithmic_bytes_per_launch": dom_bytes, "avg_launch_ms": dom_ms,
                "per_kernel": {
                    "encode": {"ms": enc_ms, "GBps": ab["encode"] / enc_ms / 1e6, "launches_per_step": 1},
                    "round_kernel": {"ms_total": rounds_ms, "GBps": ab["rounds"] / rounds_ms / 1e6,
                                     "launches_per_step": L},
                    "decode": {"ms": dec_ms, "GBps": ab["decode"] / dec_ms / 1e6, "launches_per_step": 1}},
                "whole_path_frac": value / world / peak}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "seconds_per_aggregation": ms_per_step * 1e-3,
            "step_ms": {"median": float(np.median(step_ms)), "min": float(np.min(step_ms)),
                        "p95": float(np.percentile(step_ms, 95)), "max": float(np.max(step_ms))},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": workload_name(args.workload, cfg), "N": N, "c": c, "L": L, "d": d,
                       "scale": "1/N", "replicas": world, "l2": "inputs larger than L2" if ab["total"] / (L + 2) > 2.6e8
                       else "working set may be L2 resident",
                       "buffers": "out of place: grads, workspace and output are separate device buffers"},
            "gpu_launches": int(launches), "roofline": roofline, "clocks": clocks, "remeasured": remeasured}

    # ---- the same K aggregations through the one-call entry point, one event pair around all of
    # them: no event between the launches, so consecutive kernels overlap their launch with the
    # previous kernel's tail (what a caller of cerar_allreduce_sim gets; matters below ~1 ms)
    one_ms, n_one = time_one_call(plan, grads, d, ws, out, d, d, scale, K, stream, sync_all)
    ms_one = max_over_ranks(one_ms, world, dev) / K
    line["one_call"] = {"ms_per_step": ms_one, "value": whole_job_value(ab["total"], world, ms_one), "unit": UNIT,
                        "frac": whole_job_value(ab["total"], world, ms_one) / world / peak,
                        "launches_per_step": int(n_one),
                        "note": "cerar_allreduce_sim, events around the K calls only" +
                                ("; all rounds in one launch: every message is stored into the neighbour's slot and "
                                 "also handed to the neighbour's warp through shared memory, so per steady round 2 reads "
                                 "+ 1 write reach memory instead of the 3 + 1 that the algorithmic bytes count"
                                 if n_one == 3 else "")}

    if n_one == 3:
        # the same three launches with an event between them (a few aggregations, outside the figure above)
        ph = []
        for _ in range(min(K, 5)):
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            e[0].record()
            plan.encode(grads, d, ws, d, stream)
            e[1].record()
            plan.ring_rounds(ws, d, 1, L, stream)
            e[2].record()
            plan.decode(ws, out, d, d, scale, stream)
            e[3].record()
            torch.cuda.synchronize()
            ph.append([e[i].elapsed_time(e[i + 1]) for i in range(3)])
        ph = np.median(np.array(ph), axis=0)
        line["one_call"]["per_launch"] = {
            "encode": {"ms": float(ph[0]), "GBps": ab["encode"] / ph[0] / 1e6},
            "rounds_one_launch": {"ms": float(ph[1]), "GBps_in_metric_bytes": ab["rounds"] / ph[1] / 1e6},
            "decode": {"ms": float(ph[2]), "GBps": ab["decode"] / ph[2] / 1e6}}
        plan.device_status(stream)

    # ---- end to end through the host-buffer entry point (pinned host memory)
    if not args.no_e2e:
        need = 2 * N * d * 4
        avail = 0
        try:
            for ln in open("/proc/meminfo"):
                if ln.startswith("MemAvailable"):
                    avail = int(ln.split()[1]) * 1024
        except OSError:
            pass
        d_e2e = d
        while need > 0.6 * avail / max(1, world) and d_e2e > c * 1024:
            d_e2e = (d_e2e // 2 // c) * c
            need = 2 * N * d_e2e * 4
        del out
        torch.cuda.empty_cache()
        h_in = torch.empty(N * d_e2e, dtype=torch.float32).pin_memory()
        h_out = torch.empty(N * d_e2e, dtype=torch.float32).pin_memory()
        pe = d_e2e // c
        # host inputs: the same device gradients (first d_e2e/c positions of every chunk)
        h_in.view(N, c, pe).copy_(grads.view(N, c, p)[:, :, :pe])
        torch.cuda.synchronize()
        ksteps = max(1, args.e2e_steps)
        plan.allreduce_sim_host(h_in, d_e2e, h_out, d_e2e, ws, d_e2e, scale, stream)      # warm-up
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(ksteps):
            plan.allreduce_sim_host(h_in, d_e2e, h_out, d_e2e, ws, d_e2e, scale, stream)
        e1.record()
        sync_all()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev) / ksteps
        abe = algorithmic_bytes(N, c, pe)["total"]
        line["e2e"] = {"value": whole_job_value(abe, world, ms_e2e), "unit": UNIT,
                       "h2d_bytes_per_step": N * d_e2e * 4, "d2h_bytes_per_step": N * d_e2e * 4,
                       "ms_per_step": ms_e2e, "steps": ksteps, "d": d_e2e,
                       "note": "cerar_allreduce_sim_host: pinned host gradients in, pinned host results out; position "
                               "slices overlap H2D, kernels (in place) and D2H; all PCIe copies inside the timed region"}
        plan.device_status(stream)
        del h_in, h_out

    g_sample = None
    p_s = min(p, args.ref_positions)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        g_sample = np.ascontiguousarray(grads.view(N, c, p)[:, :, :p_s].reshape(N, -1).cpu().numpy())
    plan_U, plan_R = [plan.get_U(i) for i in range(N)], [plan.get_R(i) for i in range(N)]
    del grads, ws, plan
    if not args.no_e2e:
        pass                      # `out` went before the pinned buffers were made
    else:
        del out
    torch.cuda.empty_cache()

    if world == 1 and not args.no_configs and not args.d:
        only = [k for k in args.configs.split(",") if k]
        line["configs"] = other_configs(args.workload, peak, local_rank, stream, only=only)

    if world > 1 and not args.no_ring:
        line["ring"] = ring_block(world, rank, dev)

    if g_sample is not None:
        if cfg["kind"] == "kappa":
            # library and oracle iterates of the constrained design agree only to ~1e-3 at this shape (the
            # first projection acts on encoders with kappa ~ 1e15), which the decoder amplifies: the protocol
            # is run with the plan's own matrices (inputs of the data path, like the gradients)
            from types import SimpleNamespace
            des = SimpleNamespace(N=N, c=c, U=plan_U, R=plan_R)
        else:
            des = build_design_oracle(cfg, B)
        kept = {}
        line["cpu_baseline"] = cpu_baseline(cfg, des, p_s, one_thread=True, g=g_sample, keep=kept)
        if par_dev is not None:
            line["parity"] = parity_block(des, kept, par_dev, p_s, min(p_par, p_s), scale)

    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
