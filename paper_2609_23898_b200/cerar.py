"""ctypes binding of libcerar.so: same names as the C ABI (include/cerar.h).

Only marshals arguments: every step of the data path runs in the library's
CUDA kernels.  torch is used by callers for device memory and streams; this
module itself needs only pointers (ints) and never falls back to a CPU path:
if the library cannot be loaded, importing fails.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

VANDERMONDE, EPSILON, KAPPA = 0, 1, 2
KERNEL_AUTO, KERNEL_REF, KERNEL_STAGED, KERNEL_TC = 0, 1, 2, 3

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "SINGULAR", 4: "NOT_CONVERGED",
                5: "STATE", 6: "CUDA", 7: "NOMEM", 8: "TIMEOUT", 9: "TOO_LARGE", 10: "BOUNDS"}


class CerarError(RuntimeError):
    def __init__(self, status: int, detail: str):
        self.status = status
        super().__init__(f"cerar status {status} ({STATUS_NAMES.get(status, '?')}): {detail}")


class Options(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("B", C.POINTER(C.c_double)), ("h", C.POINTER(C.c_double)),
                ("eps_init", C.c_double), ("als_iters", C.c_int), ("als_tol", C.c_double),
                ("host_only", C.c_int)]


class PlanInfo(C.Structure):
    _fields_ = [("N", C.c_int), ("c", C.c_int), ("L", C.c_int), ("construction", C.c_int),
                ("param", C.c_double), ("phi", C.c_double), ("kappa_U_max", C.c_double),
                ("kappa_M_max", C.c_double), ("inv_residual_max", C.c_double),
                ("abs_U_max", C.c_double), ("abs_R_max", C.c_double),
                ("als_iters_done", C.c_int), ("on_device", C.c_int)]


class Counters(C.Structure):
    _fields_ = [("encoded", C.c_int), ("rounds_done", C.c_int),
                ("bytes_forwarded_per_worker", C.c_uint64), ("bytes_forwarded_last_round", C.c_uint64),
                ("bytes_stored_per_worker", C.c_uint64), ("bytes_gradient", C.c_uint64)]


def _load() -> C.CDLL:
    # CERAR_LIBRARY=checked selects the build whose kernels check every address they form (tests)
    checked = os.environ.get("CERAR_LIBRARY", "") == "checked"
    path = _build.CHECKED_LIB_PATH if checked else _build.LIB_PATH
    if _build.is_stale(path):
        path = _build.build(checked=checked)
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing and could not be built")
    return C.CDLL(path)


lib = _load()
_vp, _i64, _f32p = C.c_void_p, C.c_int64, C.c_void_p

lib.cerar_plan_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_double, C.POINTER(_vp)]
lib.cerar_plan_create_ex.argtypes = [C.c_int, C.c_int, C.c_int, C.c_double, C.POINTER(Options), C.POINTER(_vp)]
lib.cerar_plan_create_custom.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                         C.c_int, C.POINTER(_vp)]
lib.cerar_plan_destroy.argtypes = [_vp]
lib.cerar_plan_destroy.restype = None
lib.cerar_plan_get_U.argtypes = [_vp, C.c_int, C.POINTER(C.c_double)]
lib.cerar_plan_get_R.argtypes = [_vp, C.c_int, C.POINTER(C.c_double)]
lib.cerar_plan_info.argtypes = [_vp, C.POINTER(PlanInfo)]
lib.cerar_design_gamma.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_double), C.c_uint64, C.POINTER(C.c_double),
                                   C.POINTER(C.c_double)]
lib.cerar_design_optimize_h.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_uint64, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                        C.POINTER(C.c_double), C.POINTER(C.c_int)]
lib.cerar_padded_length.argtypes = [_vp, _i64]
lib.cerar_padded_length.restype = _i64
lib.cerar_workspace_bytes.argtypes = [_vp, _i64]
lib.cerar_workspace_bytes.restype = C.c_size_t
lib.cerar_encode.argtypes = [_vp, _f32p, _i64, _f32p, _i64, _vp]
lib.cerar_ring_round.argtypes = [_vp, _f32p, _i64, C.c_int, _vp]
lib.cerar_ring_rounds.argtypes = [_vp, _f32p, _i64, C.c_int, C.c_int, _vp]
lib.cerar_decode.argtypes = [_vp, _f32p, _f32p, _i64, _i64, C.c_float, _vp]
lib.cerar_allreduce_sim.argtypes = [_vp, _f32p, _i64, _f32p, _i64, _f32p, _i64, C.c_float, _vp]
lib.cerar_allreduce_sim_host.argtypes = [_vp, _f32p, _i64, _f32p, _i64, _f32p, _i64, C.c_float, _vp]
lib.cerar_allreduce_sim_static.argtypes = [_vp, _f32p, _i64, _f32p, _i64, _i64, C.c_float, _vp]
lib.cerar_allreduce_fused.argtypes = [_vp, _f32p, _i64, _f32p, _i64, _i64, C.c_float, _vp]
lib.cerar_fused_supported.argtypes = [_vp]
lib.cerar_rank_workspace_bytes.argtypes = [_vp, _i64]
lib.cerar_rank_workspace_bytes.restype = C.c_size_t
lib.cerar_rank_round_slots.argtypes = [_vp, C.c_int] + [C.POINTER(C.c_int)] * 4
lib.cerar_rank_encode.argtypes = [_vp, C.c_int, _f32p, _f32p, _i64, _vp]
lib.cerar_rank_round.argtypes = [_vp, C.c_int, _f32p, _f32p, _i64, C.c_int, _vp]
lib.cerar_rank_decode.argtypes = [_vp, C.c_int, _f32p, _f32p, _i64, C.c_float, _vp]
lib.cerar_rank_round_msg.argtypes = [_vp, C.c_int, _f32p, _f32p, _i64, C.c_int, _vp]
lib.cerar_rank_round_msg_bf16.argtypes = [_vp, C.c_int, _f32p, _vp, _i64, C.c_int, _vp]
lib.cerar_rank_recv_bf16.argtypes = [_vp, C.c_int, _f32p, _vp, _i64, C.c_int, _vp]
lib.cerar_fp8_message_bytes.argtypes = [_vp, _i64]
lib.cerar_fp8_message_bytes.restype = C.c_size_t
lib.cerar_rank_round_msg_fp8.argtypes = [_vp, C.c_int, _f32p, _vp, _i64, C.c_int, _vp]
lib.cerar_rank_recv_fp8.argtypes = [_vp, C.c_int, _f32p, _vp, _i64, C.c_int, _vp]
lib.cerar_ring_tiles.argtypes = [_vp, _i64]
lib.cerar_ring_tiles.restype = _i64
lib.cerar_rank_rounds_fused.argtypes = [_vp, C.c_int, _f32p, _f32p, _vp, _vp, _vp, _vp, _i64, C.c_uint, _vp]
lib.cerar_ring_rounds_fused_local.argtypes = [_vp, C.POINTER(C.c_void_p), _vp, _i64, C.c_uint, _vp]
lib.cerar_get_counters.argtypes = [_vp, C.POINTER(Counters)]
lib.cerar_launch_count.argtypes = [_vp]
lib.cerar_launch_count.restype = C.c_uint64
lib.cerar_set_kernel_mode.argtypes = [_vp, C.c_int]
lib.cerar_device_status.argtypes = [_vp, _vp]
lib.cerar_selftest_wait_timeout.argtypes = [_vp, C.c_int, _vp]
lib.cerar_set_tuning.argtypes = [C.c_char_p, C.c_int]
lib.cerar_status_string.argtypes = [C.c_int]
lib.cerar_status_string.restype = C.c_char_p
lib.cerar_last_error.restype = C.c_char_p
lib.cerar_build_is_checked.restype = C.c_int


def _check(status: int):
    if status != 0:
        raise CerarError(status, lib.cerar_last_error().decode())


def _dptr(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64).ctypes.data_as(C.POINTER(C.c_double))


def _ptr(t) -> int:
    """Device (or host) address of a torch tensor / numpy array / int."""
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def design_gamma(N: int, c: int, B=None, h=None, seed: int = 0) -> float:
    """cerar_design_gamma: min_l sigma_min(K^(l)(B, diag(h))) (Sec. II-C)."""
    import numpy as np
    Ba = None if B is None else np.ascontiguousarray(B, dtype=np.float64)
    ha = None if h is None else np.ascontiguousarray(h, dtype=np.float64)
    dp = C.POINTER(C.c_double)
    out = C.c_double()
    _check(lib.cerar_design_gamma(N, c, Ba.ctypes.data_as(dp) if Ba is not None else None, seed,
                                  ha.ctypes.data_as(dp) if ha is not None else None, C.byref(out)))
    return out.value


def optimize_h(N: int, c: int, B=None, h0=None, sweeps: int = 2, grid: int = 17, seed: int = 0):
    """cerar_design_optimize_h: coordinate ascent on gamma(B, H).  Returns (h, gamma, moves)."""
    import numpy as np
    Ba = None if B is None else np.ascontiguousarray(B, dtype=np.float64)
    h = np.zeros(c, dtype=np.float64) if h0 is None else np.array(h0, dtype=np.float64)
    g, m = C.c_double(0.0), C.c_int(0)
    _check(lib.cerar_design_optimize_h(N, c, None if Ba is None else Ba.ctypes.data, seed, h.ctypes.data,
                                       0 if h0 is None else 1, sweeps, grid, C.byref(g), C.byref(m)))
    return h, g.value, m.value


def select_h(N: int, c: int, B, candidates):
    """H picked among several trials (Sec. II-C allows that): of the candidate diagonals, the one with
    the largest gamma(B, H).  Returns (index, gammas)."""
    gammas = [design_gamma(N, c, B, h) for h in candidates]
    best = max(range(len(gammas)), key=lambda i: gammas[i])
    return best, gammas


def cerar_set_tuning(name: str, value: int) -> int:
    return lib.cerar_set_tuning(name.encode(), int(value))


class Plan:
    """Owns a cerar_plan_t*.  Methods are the C calls with the plan bound."""

    def __init__(self, handle: int, N: int, c: int):
        self._h = C.c_void_p(handle)
        self.N, self.c, self.L = N, c, c + N - 2

    # ---- creation
    @staticmethod
    def create(N, c, kind, param, *, seed=0, B=None, h=None, eps_init=0.0, als_iters=0,
               als_tol=0.0, host_only=False) -> "Plan":
        keep = [None if B is None else np.ascontiguousarray(B, dtype=np.float64),
                None if h is None else np.ascontiguousarray(h, dtype=np.float64)]
        opt = Options()
        opt.seed = seed
        opt.B = keep[0].ctypes.data_as(C.POINTER(C.c_double)) if keep[0] is not None else None
        opt.h = keep[1].ctypes.data_as(C.POINTER(C.c_double)) if keep[1] is not None else None
        opt.eps_init, opt.als_iters, opt.als_tol, opt.host_only = eps_init, als_iters, als_tol, int(host_only)
        out = C.c_void_p()
        _check(lib.cerar_plan_create_ex(N, c, kind, float(param), C.byref(opt), C.byref(out)))
        return Plan(out.value, N, c)

    @staticmethod
    def create_custom(N, c, U, R, host_only=False) -> "Plan":
        L = c + N - 2
        Ua = np.ascontiguousarray(np.stack([np.asarray(u, np.float64) for u in U]))
        Ra = np.ascontiguousarray(np.stack([np.asarray(r, np.float64) for r in R]))
        assert Ua.shape == (N, c, c) and Ra.shape == (N, L + 1, c)
        out = C.c_void_p()
        _check(lib.cerar_plan_create_custom(N, c, Ua.ctypes.data_as(C.POINTER(C.c_double)),
                                            Ra.ctypes.data_as(C.POINTER(C.c_double)), int(host_only), C.byref(out)))
        return Plan(out.value, N, c)

    def destroy(self):
        if self._h:
            lib.cerar_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # ---- host queries
    def get_U(self, worker: int) -> np.ndarray:
        out = np.empty((self.c, self.c), dtype=np.float64)
        _check(lib.cerar_plan_get_U(self._h, worker, out.ctypes.data_as(C.POINTER(C.c_double))))
        return out

    def get_R(self, worker: int) -> np.ndarray:
        out = np.empty((self.L + 1, self.c), dtype=np.float64)
        _check(lib.cerar_plan_get_R(self._h, worker, out.ctypes.data_as(C.POINTER(C.c_double))))
        return out

    def info(self) -> dict:
        s = PlanInfo()
        _check(lib.cerar_plan_info(self._h, C.byref(s)))
        return {f: getattr(s, f) for f, _ in PlanInfo._fields_}

    def padded_length(self, d: int) -> int:
        """Smallest d' >= d with 4c | d' (what the fast kernels want; pad the gradient with zeros)."""
        return int(lib.cerar_padded_length(self._h, d))

    def workspace_bytes(self, d: int) -> int:
        return lib.cerar_workspace_bytes(self._h, d)

    def counters(self) -> dict:
        s = Counters()
        _check(lib.cerar_get_counters(self._h, C.byref(s)))
        return {f: getattr(s, f) for f, _ in Counters._fields_}

    def launch_count(self) -> int:
        return lib.cerar_launch_count(self._h)

    def set_kernel_mode(self, mode: int) -> int:
        return lib.cerar_set_kernel_mode(self._h, mode)

    def device_status(self, stream=0):
        _check(lib.cerar_device_status(self._h, stream))

    def selftest_wait_timeout(self, limit_ms=20, stream=0):
        _check(lib.cerar_selftest_wait_timeout(self._h, limit_ms, stream))

    # ---- data path (device pointers; stream = a cudaStream_t handle as int)
    def encode(self, grads, grads_stride, ws, d, stream=0):
        _check(lib.cerar_encode(self._h, _ptr(grads), grads_stride, _ptr(ws), d, stream))

    def ring_round(self, ws, d, k, stream=0):
        _check(lib.cerar_ring_round(self._h, _ptr(ws), d, k, stream))

    def ring_rounds(self, ws, d, k_first, k_last, stream=0):
        """cerar_ring_rounds: rounds k_first..k_last in one launch."""
        _check(lib.cerar_ring_rounds(self._h, _ptr(ws), d, k_first, k_last, stream))

    def decode(self, ws, out, out_stride, d, scale=1.0, stream=0):
        _check(lib.cerar_decode(self._h, _ptr(ws), _ptr(out), out_stride, d, scale, stream))

    def allreduce_sim(self, grads, grads_stride, out, out_stride, ws, d, scale=1.0, stream=0):
        _check(lib.cerar_allreduce_sim(self._h, _ptr(grads), grads_stride, _ptr(out), out_stride,
                                       _ptr(ws), d, scale, stream))

    def allreduce_fused(self, grads, grads_stride, out, out_stride, d, scale=1.0, stream=0):
        """cerar_allreduce_fused: whole protocol in one launch, slots in shared memory (small N (c+N))."""
        _check(lib.cerar_allreduce_fused(self._h, _ptr(grads), grads_stride, _ptr(out), out_stride,
                                         d, scale, stream))

    def fused_supported(self) -> bool:
        return bool(lib.cerar_fused_supported(self._h))

    # ---- one worker per GPU
    def rank_workspace_bytes(self, d: int) -> int:
        return int(lib.cerar_rank_workspace_bytes(self._h, d))

    def rank_round_slots(self, k: int):
        """(slot_prev, slot_cancel, slot_add, slot_land) of round k; -1 where the term is absent."""
        v = [C.c_int() for _ in range(4)]
        _check(lib.cerar_rank_round_slots(self._h, k, *[C.byref(x) for x in v]))
        return tuple(x.value for x in v)

    def rank_encode(self, rank, grad, ws, d, stream=0):
        _check(lib.cerar_rank_encode(self._h, rank, _ptr(grad), _ptr(ws), d, stream))

    def rank_round(self, rank, ws, peer_ws, d, k, stream=0):
        _check(lib.cerar_rank_round(self._h, rank, _ptr(ws), _ptr(peer_ws), d, k, stream))

    def rank_round_msg(self, rank, ws, msg, d, k, stream=0):
        _check(lib.cerar_rank_round_msg(self._h, rank, _ptr(ws), _ptr(msg), d, k, stream))

    def rank_round_msg_bf16(self, rank, ws, msg, d, k, stream=0):
        _check(lib.cerar_rank_round_msg_bf16(self._h, rank, _ptr(ws), _ptr(msg), d, k, stream))

    def rank_recv_bf16(self, rank, ws, msg, d, k, stream=0):
        _check(lib.cerar_rank_recv_bf16(self._h, rank, _ptr(ws), _ptr(msg), d, k, stream))

    def fp8_message_bytes(self, d: int) -> int:
        return int(lib.cerar_fp8_message_bytes(self._h, d))

    def rank_round_msg_fp8(self, rank, ws, msg, d, k, stream=0):
        _check(lib.cerar_rank_round_msg_fp8(self._h, rank, _ptr(ws), _ptr(msg), d, k, stream))

    def rank_recv_fp8(self, rank, ws, msg, d, k, stream=0):
        _check(lib.cerar_rank_recv_fp8(self._h, rank, _ptr(ws), _ptr(msg), d, k, stream))

    def ring_tiles(self, d: int) -> int:
        return int(lib.cerar_ring_tiles(self._h, d))

    def rank_rounds_fused(self, rank, ws, peer_ws, landed_local, freed_local, landed_next, freed_prev, d, epoch,
                          stream=0):
        _check(lib.cerar_rank_rounds_fused(self._h, rank, _ptr(ws), _ptr(peer_ws), _ptr(landed_local),
                                           _ptr(freed_local), _ptr(landed_next), _ptr(freed_prev), d, epoch, stream))

    def ring_rounds_fused_local(self, ws_list, counters, d, epoch, stream=0):
        arr = (C.c_void_p * len(ws_list))(*[_ptr(w) for w in ws_list])
        _check(lib.cerar_ring_rounds_fused_local(self._h, arr, _ptr(counters), d, epoch, stream))

    def rank_decode(self, rank, ws, out, d, scale=1.0, stream=0):
        _check(lib.cerar_rank_decode(self._h, rank, _ptr(ws), _ptr(out), d, scale, stream))

    def allreduce_sim_static(self, grads, grads_stride, out, out_stride, d, scale=1.0, stream=0):
        """cerar_allreduce_sim_static: same pipeline, workspace built into the library (<= 64 MiB)."""
        _check(lib.cerar_allreduce_sim_static(self._h, _ptr(grads), grads_stride, _ptr(out), out_stride,
                                              d, scale, stream))

    def allreduce_sim_host(self, h_grads, h_grads_stride, h_out, h_out_stride, ws, d, scale=1.0, stream=0):
        _check(lib.cerar_allreduce_sim_host(self._h, _ptr(h_grads), h_grads_stride, _ptr(h_out),
                                            h_out_stride, _ptr(ws), d, scale, stream))


def cerar_plan_create(N, c, kind, param, **kw) -> Plan:
    return Plan.create(N, c, kind, param, **kw)


def cerar_plan_create_custom(N, c, U, R, host_only=False) -> Plan:
    return Plan.create_custom(N, c, U, R, host_only)
