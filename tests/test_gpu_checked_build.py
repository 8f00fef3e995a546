"""The checked build of the library (libcerar_checked.so: the same sources compiled with
-DCERAR_BOUNDS_CHECK) stands in for a memory checker: its kernels compare every address they form
for a plain load, store or 1-D bulk copy with the extent of the buffer it belongs to, skip an
access that falls outside and report it through the status word.  The tests run in a child process,
because the binding loads one library per process (CERAR_LIBRARY=checked selects this one)."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
import numpy as np, torch
sys.path.insert(0, %(root)r)
from paper_2609_23898_b200 import cerar, inputs
from oracle import designs as Dz, protocol as P
assert cerar.lib.cerar_build_is_checked() == 1
s = torch.cuda.current_stream().cuda_stream
worst = 0.0
# FMA contractions (staged, tiled for unaligned rows, plain), the tensor-core kernel's row-by-row copies for
# unaligned rows, every form of the rounds, ragged tails
cases = [(4, 8, 4096 + 64, 0), (8, 16, 2052, 0), (5, 7, 1031, 0), (3, 5, 37, 1), (16, 20, 1028, 0), (8, 32, 516, 0),
         (32, 32, 260, 0), (33, 34, 36, 0), (8, 8, 151556, 0), (8, 32, 517, 0), (4, 64, 1030, 0), (4, 8, 4099, 0)]
for N, c, p, mode in cases:
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(N + c))
    g = inputs.gradients_numpy(N, d, "normal", seed=1)
    ora = P.allreduce([x.astype(np.float64) for x in g], des.U, des.R, 0.5) if N * d < 3e6 else None
    for one_call in (False, True):
        plan = cerar.Plan.create_custom(N, c, des.U, des.R)
        plan.set_kernel_mode(mode)
        dev_g = torch.from_numpy(g).cuda()
        out = torch.full((N, d), float("nan"), device="cuda")
        ws = torch.full((plan.workspace_bytes(d) // 4,), float("nan"), device="cuda")
        if one_call:
            plan.allreduce_sim(dev_g, d, out, d, ws, d, 0.5, s)
        else:
            plan.encode(dev_g, d, ws, d, s)
            for k in range(1, c + N - 1):
                plan.ring_round(ws, d, k, s)
            plan.decode(ws, out, d, d, 0.5, s)
        torch.cuda.synchronize()
        plan.device_status(s)                          # raises CerarError(BOUNDS) if any check fired
        if ora is not None:
            got = out.cpu().numpy()
            worst = max(worst, max(P.rel_l2(got[i], ora["out"][i]) for i in range(N)))
assert worst < 1e-5, worst
# the mechanism itself, without a single access out of range: the checks are told that the buffers end
# 8 floats early, so a kernel that touches the last positions (the encode writes the last row of the
# last worker) must skip those accesses and say so
N, c, p = 8, 16, 2052
d = c * p
des = Dz.custom_orthogonal(N, c, np.random.default_rng(0))
plan = cerar.Plan.create_custom(N, c, des.U, des.R)
dev_g = torch.randn(N * d, device="cuda")
ws = torch.zeros(plan.workspace_bytes(d) // 4, device="cuda")
plan.encode(dev_g, d, ws, d, s)
plan.device_status(s)
assert cerar.cerar_set_tuning("checked_shrink", 8) == 0
plan.encode(dev_g, d, ws, d, s)
try:
    plan.device_status(s)
    raise SystemExit("the shortened extent was not noticed")
except cerar.CerarError as e:
    assert e.status == 10, e
assert cerar.cerar_set_tuning("checked_shrink", 0) == 0
plan.device_status(s)                                  # reported once, then clear
print("CHECKED-BUILD-OK", worst)
'''


@pytest.mark.gpu
def test_checked_build_runs_the_pipeline_without_a_single_address_out_of_range():
    env = dict(os.environ, CERAR_LIBRARY="checked")
    res = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], env=env, capture_output=True, text=True,
                         timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "CHECKED-BUILD-OK" in res.stdout
