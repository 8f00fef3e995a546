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


def run_library(plan, grads_np, scale=1.0, *, inplace=False, stepwise=True, sync_check=True):
    """grads_np: (N, d) fp32.  Returns dict(out (N,d) fp32, Delta, Y as numpy)."""
    import torch
    N, c, L = plan.N, plan.c, plan.L
    d = grads_np.shape[1]
    p = d // c
    dev = torch.device("cuda:0")
    ws = torch.zeros(N * (c + N) * p, dtype=torch.float32, device=dev)
    ws.fill_(float("nan"))          # anything the kernels forget to write shows up
    s = torch_stream()
    wstride = (c + N) * p
    if inplace:
        wv = ws.view(N, c + N, p)
        wv[:, N:, :] = torch.from_numpy(grads_np).to(dev).view(N, c, p)
        g_ptr, g_stride = ws.data_ptr() + 4 * N * p, wstride
    else:
        g = torch.from_numpy(grads_np).to(dev).contiguous()
        g_ptr, g_stride = g.data_ptr(), d
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
            o = torch.full((N, d), float("nan"), dtype=torch.float32, device=dev)
            plan.decode(ws, o, d, d, scale, s)
            out = o.cpu().numpy()
    else:
        if inplace:
            plan.allreduce_sim(g_ptr, g_stride, g_ptr, g_stride, ws, d, scale, s)
            out = ws_view(ws, N, c, p)[:, N:, :].reshape(N, d).copy()
        else:
            o = torch.full((N, d), float("nan"), dtype=torch.float32, device=dev)
            plan.allreduce_sim(g_ptr, g_stride, o, d, ws, d, scale, s)
            out = o.cpu().numpy()
    torch.cuda.synchronize()
    if sync_check:
        plan.device_status(s)
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
    return {"positions": int(idx.size), "rel_l2_Y": P.rel_l2(Y_dev, Y_ora),
            "rel_l2_out_max": max(P.rel_l2(out_dev[i], ora["out"][i]) for i in range(N)),
            "kappa_M": kap, "kappa_times_2^-24": kap * 2.0 ** -24,
            "rel_l2_oracle_vs_exact_mean": max(P.rel_l2(ora["out"][i], P.exact_sum(list(g_sub)) * scale)
                                               for i in range(N))}
