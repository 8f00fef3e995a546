"""Accuracy against conditioning of the CERAR designs, on the host (no GPU needed).

  python -m paper_2609_23898_b200.tradeoff [--N 4] [--c 12] [--trials 16] [--seed 0]

Four tables from the library's fp64 design builder (host_only plans):
  1. epsilon-construction (Sec. II-C) over eps: Phi = O(eps^2) against kappa_2(M_i) = O(eps^-r*);
  2. the same eps with H chosen among `trials` random diagonals by the largest
     gamma(B, H) = min_l sigma_min(K^(l)(B, H)) (Sec. II-C: H can be picked by trying several), and with
     the deterministic H that coordinate ascent on gamma gives from B (cerar_design_optimize_h);
  3. the same eps with a block-structured base matrix (row r of B non-zero on its own c/N columns only),
     for which U_k and R_i are block sparse;
  4. the condition-number-constrained design (Sec. II-D) over the bound C: the Phi it reaches
     and the kappa_2(M_i) it ends with.
Phi is the squared least-squares error of Eq. (F); the relative error of the decoded sum is
about sqrt(Phi / (N c)) for i.i.d. gradients.

  python -m paper_2609_23898_b200.tradeoff --messages            (needs a GPU)

A fifth table, measured on the device: the relative error of the decoded mean (against the exact
mean of the gradients, max over workers) when the ring messages travel as binary32, bfloat16 or 8-bit
e4m3 values, for designs of increasing kappa_2(M_i): c = N (r* = 0), the constrained design with a
small bound, and an epsilon-construction with c = 2N.  One worker per workspace on this GPU
(ring.LocalRing); a "transport" is the sender's message kernel followed by the receiver's.
"""
from __future__ import annotations

import argparse

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--N", type=int, default=4)
    ap.add_argument("--c", type=int, default=12)
    ap.add_argument("--trials", type=int, default=16)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--als-iters", type=int, default=200)
    ap.add_argument("--sweeps", type=int, default=2)
    ap.add_argument("--grid", type=int, default=17)
    ap.add_argument("--messages", action="store_true", help="message precision against kappa (GPU)")
    args = ap.parse_args()
    from . import cerar, inputs
    if args.messages:
        return message_precision_table(args.seed)
    N, c = args.N, args.c
    B = inputs.base_matrix(N, c, args.seed)
    r_star = -(-c // N) - 1
    print(f"N={N} c={c} r*={r_star} rates: communication {1 + (N - 2) / c:.3f}, storage {1 + N / c:.3f}")

    def row(plan):
        i = plan.info()
        return i["phi"], i["kappa_M_max"], i["kappa_U_max"], i["abs_U_max"]

    h0 = np.linspace(-1.0, 1.0, c) if c > 1 else np.zeros(1)
    rng = np.random.default_rng(args.seed + 1)
    cands = [h0] + [rng.uniform(-1.0, 1.0, c) for _ in range(args.trials)]
    cands = [h / np.abs(h).max() for h in cands]                  # ||H||_2 = 1 for all of them
    best, gammas = cerar.select_h(N, c, B, cands)
    print(f"gamma(B, H): default H {gammas[0]:.3e}; best of {args.trials} random diagonals {gammas[best]:.3e} "
          f"(median {np.median(gammas[1:]):.3e})")
    h_det, g_det, moves = cerar.optimize_h(N, c, B, sweeps=args.sweeps, grid=args.grid)
    print(f"deterministic H (coordinate ascent on gamma, {args.sweeps} sweeps over {args.grid} values, {moves} moves): "
          f"gamma {g_det:.3e}")
    print("\n| eps | Phi (default / best trial / deterministic) | kappa_M default H | kappa_M best trial | kappa_M deterministic H "
          "| max abs U default | best trial | deterministic |")
    print("|---|---|---|---|---|---|---|---|")
    for eps in (1e-1, 3e-2, 1e-2, 3e-3, 1e-3):
        out = []
        for h in (cands[0], cands[best], h_det):
            try:
                p = cerar.Plan.create(N, c, cerar.EPSILON, eps, B=B, h=h, host_only=True)
                out.append(row(p))
                p.destroy()
            except cerar.CerarError as e:
                out.append((float("nan"),) * 4)
        print(f"| {eps:g} | {out[0][0]:.3e} / {out[1][0]:.3e} / {out[2][0]:.3e} | {out[0][1]:.3e} | {out[1][1]:.3e} | "
              f"{out[2][1]:.3e} | {out[0][3]:.2e} | {out[1][3]:.2e} | {out[2][3]:.2e} |", flush=True)
    if c % N == 0 and c > N:
        # block-structured base matrix (row r on its own c/N columns): U_k, R_i come out block sparse
        Bs, hs = inputs.structured_base(N, c, args.seed)
        print(f"\nblock-structured B (c/N = {c // N} non-zeros per column of U_k instead of {c}): gamma {cerar.design_gamma(N, c, Bs, hs):.3e}")
        print("\n| eps | Phi | kappa_M | max abs U |")
        print("|---|---|---|---|")
        for eps in (1e-1, 3e-2, 1e-2, 3e-3, 1e-3):
            try:
                p = cerar.Plan.create(N, c, cerar.EPSILON, eps, B=Bs, h=hs, host_only=True)
                r = row(p)
                p.destroy()
                print(f"| {eps:g} | {r[0]:.3e} | {r[1]:.3e} | {r[3]:.2e} |", flush=True)
            except cerar.CerarError as e:
                print(f"| {eps:g} | - | - | {e} |", flush=True)
    print("\n| C (bound on kappa_M) | Phi reached | kappa_M reached | ALS iterations |")
    print("|---|---|---|---|")
    for C in (1e2, 1e3, 1e4, 1e5, 1e6):
        try:
            p = cerar.Plan.create(N, c, cerar.KAPPA, C, B=B, als_iters=args.als_iters, host_only=True)
            i = p.info()
            print(f"| {C:g} | {i["phi"]:.3e} | {i["kappa_M_max"]:.3e} | {i["als_iters_done"]} |", flush=True)
            p.destroy()
        except cerar.CerarError as e:
            print(f"| {C:g} | - | - | {e} |", flush=True)


def message_precision_table(seed=0, p=1 << 16):
    import torch
    from . import cerar, inputs, ring
    stream = torch.cuda.current_stream().cuda_stream
    designs = [("epsilon 1e-3, c = N", 4, 4, cerar.EPSILON, 1e-3), ("epsilon 1e-3, c = N", 8, 8, cerar.EPSILON, 1e-3),
               ("epsilon 1e-3, c = N", 16, 16, cerar.EPSILON, 1e-3), ("kappa <= 30", 4, 12, cerar.KAPPA, 30.0),
               ("kappa <= 100", 4, 12, cerar.KAPPA, 100.0), ("kappa <= 100", 8, 32, cerar.KAPPA, 100.0),
               ("epsilon 1e-2, c = 2N", 4, 8, cerar.EPSILON, 1e-2)]
    print("| design | N | c | kappa_M | Phi | binary32 | bfloat16 | e4m3 + tile scale | bytes per message value |")
    print("|---|---|---|---|---|---|---|---|---|")
    for name, N, c, kind, param in designs:
        d = c * p
        plan = cerar.Plan.create(N, c, kind, param, B=inputs.base_matrix(N, c, seed))
        info = plan.info()
        g = torch.empty(N, d, device="cuda")
        inputs.fill_gradients_torch([g[i] for i in range(N)], "normal", seed=seed)
        mean = g.double().mean(dim=0)
        errs = []
        for fmt in ("f32", "bf16", "fp8"):
            r = ring.LocalRing(plan, d)
            r.encode([g[i] for i in range(N)], stream)
            if fmt == "f32":
                for k in range(1, plan.L + 1):
                    r.round(k, stream)
            else:
                nb = p * 2 if fmt == "bf16" else (plan.fp8_message_bytes(d) + 15) // 16 * 16
                raw = torch.empty(N, nb, dtype=torch.uint8, device="cuda")
                send = plan.rank_round_msg_bf16 if fmt == "bf16" else plan.rank_round_msg_fp8
                recv = plan.rank_recv_bf16 if fmt == "bf16" else plan.rank_recv_fp8
                for k in range(1, plan.L + 1):
                    for i in range(N):
                        send(i, r.ws[i], raw[i], d, k, stream)
                    for i in range(N):
                        recv((i + 1) % N, r.ws[(i + 1) % N], raw[i], d, k, stream)
            outs = [torch.empty(d, device="cuda") for _ in range(N)]
            r.decode(outs, 1.0 / N, stream)
            torch.cuda.synchronize()
            plan.device_status(stream)
            errs.append(max(float((o.double() - mean).norm() / mean.norm()) for o in outs))
            del r, outs
        print(f"| {name} | {N} | {c} | {info['kappa_M_max']:.2e} | {info['phi']:.2e} | {errs[0]:.2e} | {errs[1]:.2e} | "
              f"{errs[2]:.2e} | 4 / 2 / {plan.fp8_message_bytes(d) / p:.3f} |", flush=True)
        plan.destroy()
        del g
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
