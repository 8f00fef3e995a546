"""Shared helpers of the GPU parity tests: run the library step by step on
torch device buffers and the oracle on the same inputs."""
import numpy as np

from oracle import protocol as P


def torch_stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


def ws_view(ws, N, c, p):
    """(N, c+N, p) numpy view of a workspace tensor copied to the host."""
    return ws.detach().cpu().numpy().reshape(N, c + N, p)


GUARD_FLOATS = 1024                       # 4 KB on either side of every device buffer
GUARD_PATTERN = 0x7FC0DEAD                # a quiet NaN with a payload (fits a signed 32-bit integer)


class Guarded:
    """A device buffer of n floats with 4 KB of a sentinel bit pattern before and after it, inside one
    allocation.  check() fails if a kernel stored anything outside the buffer proper (a store past the end
    of a workspace or an output would otherwise go unnoticed: the NaN pre-fill only catches elements INSIDE a
    buffer that were not written).  The payload starts on the same 4 KB boundary an allocation of its own
    would, so alignment-dependent kernel paths are the ones a caller gets."""

    def __init__(self, n, device, fill=float("nan")):
        import torch
        self.whole = torch.empty(n + 2 * GUARD_FLOATS, dtype=torch.float32, device=device)
        self.whole.view(torch.int32).fill_(GUARD_PATTERN)
        self.t = self.whole[GUARD_FLOATS:GUARD_FLOATS + n]
        if fill is not None:
            self.t.fill_(fill)
        self.n = n

    def check(self, name="buffer"):
        import torch
        ints = self.whole.view(torch.int32)
        lo, hi = ints[:GUARD_FLOATS], ints[GUARD_FLOATS + self.n:]
        assert bool((lo == GUARD_PATTERN).all()), f"a kernel wrote in front of the {name}"
        assert bool((hi == GUARD_PATTERN).all()), f"a kernel wrote past the end of the {name}"


def run_library(plan, grads_np, scale=1.0, *, inplace=False, stepwise=True, sync_check=True):
    """grads_np: (N, d) fp32.  Returns dict(out (N,d) fp32, Delta, Y as numpy).  Workspace, gradients and
    output sit between guard regions that are checked after the run."""
    import torch
    N, c, L = plan.N, plan.c, plan.L
    d = grads_np.shape[1]
    p = d // c
    dev = torch.device("cuda:0")
    gws = Guarded(N * (c + N) * p, dev)          # NaN inside: anything the kernels forget to write shows up
    ws = gws.t
    s = torch_stream()
    wstride = (c + N) * p
    gg = go = None
    if inplace:
        wv = ws.view(N, c + N, p)
        wv[:, N:, :] = torch.from_numpy(grads_np).to(dev).view(N, c, p)
        g_ptr, g_stride = ws.data_ptr() + 4 * N * p, wstride
    else:
        gg = Guarded(N * d, dev, fill=None)
        gg.t.copy_(torch.from_numpy(grads_np).reshape(-1))
        g_ptr, g_stride = gg.t.data_ptr(), d
    res = {}
    if stepwise:
        plan.encode(g_ptr, g_stride, ws, d, s)
        res["Delta"] = ws_view(ws, N, c, p)[:, N:, :].copy()          # (N, c, p): row j = delta_{i,j+1}
        for k in range(1, L + 1):
            plan.ring_round(ws, d, k, s)
        wsn = ws_view(ws, N, c, p)
        res["Y"] = np.concatenate([wsn[:, :L, :], wsn[:, L + 1:L + 2, :]], axis=1).copy()   # (N, L+1, p)
        if inplace:
            plan.decode(ws, ws.data_ptr() + 4 * N * p, wstride, d, scale, s)
            out = ws_view(ws, N, c, p)[:, N:, :].reshape(N, d).copy()
        else:
            go = Guarded(N * d, dev)
            plan.decode(ws, go.t, d, d, scale, s)
            out = go.t.view(N, d).cpu().numpy()
    else:
        if inplace:
            plan.allreduce_sim(g_ptr, g_stride, g_ptr, g_stride, ws, d, scale, s)
            out = ws_view(ws, N, c, p)[:, N:, :].reshape(N, d).copy()
        else:
            go = Guarded(N * d, dev)
            plan.allreduce_sim(g_ptr, g_stride, go.t, d, ws, d, scale, s)
            out = go.t.view(N, d).cpu().numpy()
    torch.cuda.synchronize()
    if sync_check:
        plan.device_status(s)
    gws.check("workspace")
    if gg is not None:
        gg.check("gradients")
        assert np.array_equal(gg.t.view(N, d).cpu().numpy(), grads_np), "the gradients were modified"
    if go is not None:
        go.check("output")
    res["out"] = out
    res["counters"] = plan.counters()
    return res


def run_oracle(U, R, grads_np, scale=1.0):
    res = P.allreduce([g.astype(np.float64) for g in grads_np], U, R, scale)
    N = len(U)
    # same shapes as run_library: Delta (N, c, p), Y (N, L+1, p)
    res["Delta_rows"] = np.stack([res["Delta"][i].T for i in range(N)])
    res["Y_rows"] = np.stack([res["Y"][i].T for i in range(N)])
    return res


def rel_l2(a, b):
    return P.rel_l2(a, b)


def sampled_parity(cfg, des, plan, grads, ws, out, scale, n_tiles=6, tile=512):
    """Full-size check on sampled position tiles: positions are independent, so
    the oracle runs the whole protocol on the sampled columns only."""
    import torch
    N, c, d = cfg["N"], cfg["c"], cfg["d"]
    p, L = d // c, c + N - 2
    rng = np.random.default_rng(123)
    starts = sorted(set([0, max(0, p - tile)] + [int(x) for x in rng.integers(0, max(1, p - tile), n_tiles)]))
    idx = np.concatenate([np.arange(s, min(s + tile, p)) for s in starts])
    idx_t = torch.from_numpy(idx).to(grads.device)
    g_sub = grads.view(N, c, p)[:, :, idx_t].reshape(N, -1).cpu().numpy().astype(np.float64)
    ora = P.allreduce([x for x in g_sub], des.U, des.R, scale)
    wsv = ws.view(N, c + N, p)
    rows_t = torch.tensor(list(range(L)) + [L + 1], device=grads.device)
    Y_dev = wsv[:, rows_t[:, None], idx_t[None, :]].cpu().numpy()         # (N, L+1, S)
    Y_ora = np.stack([ora["Y"][i].T for i in range(N)])
    out_dev = out.view(N, c, p)[:, :, idx_t].reshape(N, -1).cpu().numpy()
    kap = max(P.kappa2(P.m_matrix(des.U, i)) for i in range(N))
    yard = rounding_yardsticks(des.U, des.R, g_sub, scale, Y_dev=Y_dev, out_dev=out_dev)
    return {"positions": int(idx.size), "rel_l2_Y": P.rel_l2(Y_dev, Y_ora), "yardsticks": yard,
            "rel_l2_out_max": max(P.rel_l2(out_dev[i], ora["out"][i]) for i in range(N)),
            "kappa_M": kap, "kappa_times_2^-24": kap * 2.0 ** -24,
            "rel_l2_oracle_vs_exact_mean": max(P.rel_l2(ora["out"][i], P.exact_sum(list(g_sub)) * scale)
                                               for i in range(N))}


U32 = 2.0 ** -24


def fp32_copy(mats):
    """The coefficients as the device holds them: rounded to binary32, returned in fp64."""
    return [np.asarray(m, dtype=np.float32).astype(np.float64) for m in mats]


def rounding_yardsticks(U, R, grads, scale, *, Delta_dev=None, Y_dev=None, out_dev=None):
    """A-priori fp32 rounding bounds for the device results, stage by stage and end to end, in fp64 from
    the oracle's matrices.  An ill-conditioned design amplifies fp32 roundoff by about kappa_2(M_i), so
    its decoded output cannot be held to 1e-4 of the exact-arithmetic result; what CAN be held to is
    the standard bound for dot products in floating point, |fl(x.y) - x.y| <= n u |x|.|y|, applied to
    what each stage really computes with the coefficients the device really holds (their binary32 copies):

      encode      || Delta_dev - G_i Uf_i ||_F          <=  u c     || |G_i| |Uf_i| ||_F
      rounds      || Y_dev - rounds(Delta_dev) ||_F     <=  u 2(N+1) || sum of |delta| over the terms of each message ||_F
      decode      || out_dev - s Y_dev Rf_i ||_F        <=  u (L+1) s || |Y_dev| |Rf_i| ||_F
      end to end  || out_dev - s G^(i) M_i(Uf) Rf_i ||_F <=  u (c+L) s || |G^(i)| |M_i(Uf)| |Rf_i| ||_F

    (u = 2^-24; the tensor-core contraction computes 3 x TF32 products with a per-product error of about
    2^-22, still inside these worst-case bounds by a wide margin.)  A wrong index, a dropped term or a
    coefficient damaged on its way to the tensor cores shows as a residual of the size of |x|.|y| itself,
    i.e. about 1/(n u) ~ 1e5 times the bound, however ill-conditioned the design.

    grads: (N, d) array; Delta_dev (N, c, p), Y_dev (N, L+1, p), out_dev (N, d): device results (any may
    be None).  Returns the worst ratio residual / bound over the workers per stage, and the relative
    deviations of the output from the fp64 oracle with the rounded and with the exact coefficients'
    end-to-end bound."""
    N = len(U)
    c = np.asarray(U[0]).shape[0]
    L = c + N - 2
    Uf, Rf = fp32_copy(U), fp32_copy(R)
    g64 = [np.asarray(x, dtype=np.float64) for x in grads]
    G = [P.chunk_matrix(x, c) for x in g64]
    res = {}
    if Delta_dev is not None:
        worst = 0.0
        for i in range(N):
            got = np.asarray(Delta_dev[i], np.float64).T
            bound = U32 * c * np.linalg.norm(np.abs(G[i]) @ np.abs(Uf[i]))
            worst = max(worst, np.linalg.norm(got - G[i] @ Uf[i]) / bound)
        res["encode_ratio"] = float(worst)
        if Y_dev is not None:
            D64 = [np.asarray(Delta_dev[i], np.float64).T for i in range(N)]
            Y_ref, _, _ = P.run_rounds(D64)
            eye = [np.eye(c)] * N
            worst = 0.0
            for i in range(N):
                mag = P.stacked_gradients([np.abs(x) for x in D64], i) @ P.m_matrix(eye, i)
                bound = U32 * 2 * (N + 1) * np.linalg.norm(mag)
                worst = max(worst, np.linalg.norm(np.asarray(Y_dev[i], np.float64).T - Y_ref[i]) / bound)
            res["rounds_ratio"] = float(worst)
    if Y_dev is not None and out_dev is not None:
        worst = 0.0
        for i in range(N):
            Yd = np.asarray(Y_dev[i], np.float64).T
            bound = U32 * (L + 1) * scale * np.linalg.norm(np.abs(Yd) @ np.abs(Rf[i]))
            worst = max(worst, np.linalg.norm(np.asarray(out_dev[i], np.float64) - P.unchunk(scale * (Yd @ Rf[i]))) / bound)
        res["decode_ratio"] = float(worst)
    if out_dev is not None:
        ora_f = P.allreduce(g64, Uf, Rf, scale)
        worst = worst_rel = bound_rel = 0.0
        for i in range(N):
            mag = np.abs(P.stacked_gradients(G, i)) @ np.abs(P.m_matrix(Uf, i)) @ np.abs(Rf[i])
            bound = U32 * (c + L) * scale * np.linalg.norm(mag)
            err = np.linalg.norm(np.asarray(out_dev[i], np.float64) - ora_f["out"][i])
            ref = np.linalg.norm(ora_f["out"][i])
            worst = max(worst, err / bound)
            worst_rel = max(worst_rel, err / ref)
            bound_rel = max(bound_rel, bound / ref)
        res["end_to_end_ratio"] = float(worst)
        res["rel_l2_out_vs_rounded_coefficients"] = float(worst_rel)
        res["apriori_bound_rel"] = float(bound_rel)
    return res


def assert_within_rounding_bounds(y, K=1.0):
    """Every residual within K times its a-priori bound (K = 1: the bound itself)."""
    for key in ("encode_ratio", "rounds_ratio", "decode_ratio", "end_to_end_ratio"):
        if key in y:
            assert y[key] <= K, (key, y)
