"""Seeded synthetic inputs shaped like the paper's workloads.

Nothing here knows anything about CERAR's arithmetic: only random gradients
(fp32, one independent stream per logical worker) and the random base matrix
B that the epsilon / kappa constructions draw.  The same arrays are handed to
the CUDA library and to the CPU oracle.

Workloads (the paper reduces fp32 gradient tensors of 1e8..2.4e10 entries and
Pythia-1.4B gradients; neither the model nor its data is available, so these
stand in with the same shapes and scales):
  "normal"   i.i.d. N(0, std^2)
  "blocks"   24 contiguous layer-shaped blocks over the flat vector, block
             std log-uniform in [1e-5, 1e-2], Gaussian inside a block
  "student"  Student-t with nu = 3, scaled by 1e-3 (heavy tails)
"""
from __future__ import annotations

import numpy as np

PYTHIA_1P4B_PARAMS = 1_414_647_808     # 2*50304*2048 + 24*(12*2048^2 + 13*2048) + 2*2048

CONFIGS = {
    # name: N, c, construction, param, d, workload, workload kwargs
    "cfg1": dict(N=4, c=8, kind="vandermonde", param=0.1, d=65_536, workload="normal", std=1.0),
    "cfg2": dict(N=4, c=16, kind="epsilon", param=1e-3, d=16_777_216, workload="normal", std=1e-2),
    "cfg3": dict(N=8, c=32, kind="epsilon", param=1e-2, d=PYTHIA_1P4B_PARAMS, workload="blocks"),
    "cfg4": dict(N=8, c=64, kind="kappa", param=1e4, d=268_435_456, workload="student"),
}


def base_matrix(N: int, c: int, seed: int = 0) -> np.ndarray:
    """The N x c matrix B of i.i.d. N(0,1) entries the constructions start from."""
    return np.random.default_rng(seed).standard_normal((N, c))


def block_stds(seed: int = 0, nblocks: int = 24) -> np.ndarray:
    rng = np.random.default_rng(10_000 + seed)
    return 10.0 ** rng.uniform(-5.0, -2.0, size=nblocks)


def block_edges(d: int, nblocks: int = 24) -> np.ndarray:
    return np.array([(b * d) // nblocks for b in range(nblocks + 1)], dtype=np.int64)


def gradients_numpy(N: int, d: int, workload: str = "normal", seed: int = 0, std: float = 1.0) -> np.ndarray:
    """N x d fp32 array, worker i drawn from its own stream (seed 1000*seed + i)."""
    out = np.empty((N, d), dtype=np.float32)
    for i in range(N):
        rng = np.random.default_rng(1000 * seed + i)
        if workload == "normal":
            out[i] = (std * rng.standard_normal(d)).astype(np.float32)
        elif workload == "blocks":
            g = rng.standard_normal(d)
            edges, stds = block_edges(d), block_stds(seed)
            for b in range(len(stds)):
                g[edges[b]:edges[b + 1]] *= stds[b]
            out[i] = g.astype(np.float32)
        elif workload == "student":
            out[i] = (1e-3 * rng.standard_t(3.0, size=d)).astype(np.float32)
        else:
            raise ValueError(workload)
    return out


def fill_gradients_torch(dst, workload: str = "normal", seed: int = 0, std: float = 1.0, chunk: int = 1 << 26):
    """Fill rows of `dst` (list of N 1-D fp32 CUDA tensors, or an N x d tensor)
    in place on the device, worker i from generator seed 1000*seed + i."""
    import torch
    rows = [dst[i] for i in range(len(dst))]
    for i, row in enumerate(rows):
        d = row.numel()
        gen = torch.Generator(device=row.device)
        gen.manual_seed(1000 * seed + i)
        if workload == "normal":
            for a in range(0, d, chunk):
                row[a:a + chunk].normal_(0.0, std, generator=gen)
        elif workload == "blocks":
            edges, stds = block_edges(d), block_stds(seed)
            for b in range(len(stds)):
                lo, hi = int(edges[b]), int(edges[b + 1])
                for a in range(lo, hi, chunk):
                    row[a:min(a + chunk, hi)].normal_(0.0, float(stds[b]), generator=gen)
        elif workload == "student":
            # t_3 = z / sqrt(chi2_3 / 3), chi2_3 = sum of three squared normals
            for a in range(0, d, chunk):
                seg = row[a:a + chunk]
                seg.normal_(0.0, 1.0, generator=gen)
                chi = torch.zeros_like(seg)
                tmp = torch.empty_like(seg)
                for _ in range(3):
                    tmp.normal_(0.0, 1.0, generator=gen)
                    chi.addcmul_(tmp, tmp)
                seg.div_(chi.div_(3.0).sqrt_()).mul_(1e-3)
                del chi, tmp
        else:
            raise ValueError(workload)
    return dst


def structured_base(N: int, c: int, seed: int = 0):
    """(B, h) for a block-structured design: row r of the N x c base matrix is non-zero on its own c/N
    columns only (i.i.d. N(0,1) there), and the diagonal h repeats c/N equally spaced values of [-1, 1] in
    every block.  Needs N | c.  Seeded input data only: what the design does with them is the library's
    (and, separately, the oracle's) business."""
    if c % N:
        raise ValueError("a block-structured base matrix needs N | c")
    beta = c // N
    rng = np.random.default_rng(77000 + seed)
    B = np.zeros((N, c))
    for r in range(N):
        B[r, r * beta:(r + 1) * beta] = rng.standard_normal(beta)
    hb = np.linspace(-1.0, 1.0, beta) if beta > 1 else np.ones(1)
    return B, np.tile(hb, N)

