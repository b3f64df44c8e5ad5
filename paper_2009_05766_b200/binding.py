"""Thin ctypes binding of libnetmax.so: argument marshalling only.

Function names mirror include/netmax.h.  Every step of a round runs inside the CUDA
library; there is no Python or CPU fallback -- if the library is missing or cannot be
loaded, importing a function from here raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

from . import build as _build

NETMAX_OK = 0
STATUS = {0: "OK", -1: "INVALID_ARG", -2: "BAD_PROB_ROW", -3: "OOM", -4: "CUDA_ERROR", -5: "TRACE_RANGE",
          -6: "NOT_CONNECTED", -7: "INFEASIBLE"}

EXPORTS = [
    "netmax_config_init", "netmax_workspace_size", "netmax_create_ex", "netmax_create", "netmax_destroy",
    "netmax_set_policy", "netmax_get_policy", "netmax_set_replicas", "netmax_set_centres", "netmax_round",
    "netmax_round_from_host",
    "netmax_rounds_done", "netmax_set_fuse_rounds", "netmax_read_replicas", "netmax_read_centres", "netmax_read_columns",
    "netmax_read_columns_static",
    "netmax_peer_trace", "netmax_telemetry", "netmax_replicas_device", "netmax_sample_peers",
    "netmax_measure", "netmax_async_begin", "netmax_async_set_times", "netmax_async_steps", "netmax_async_time",
    "netmax_async_trace", "netmax_async_ema", "netmax_async_monitor", "netmax_async_monitor_refreshes",
    "netmax_iteration_times", "netmax_policy_generate", "netmax_policy_generate_ex", "netmax_policy_generate_device", "netmax_policy_generate_fixed_weight", "netmax_policy_fixed_weight_at", "netmax_debug_absent_ctas", "netmax_kernel_launches", "netmax_last_error",
]


class NetmaxError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"netmax: {STATUS.get(code, code)}: {message}")
        self.code = code


class Config(C.Structure):
    _fields_ = [
        ("M", C.c_int32), ("d", C.c_int64), ("element_offset", C.c_int64), ("link_speed_gbps", C.c_void_p), ("prob", C.c_void_p),
        ("lr", C.c_double), ("rho", C.c_double), ("pull_weight", C.c_double), ("sigma", C.c_double), ("x0_std", C.c_double),
        ("c_std", C.c_double), ("objective", C.c_int32), ("seed", C.c_uint64), ("device", C.c_int32),
        ("stream", C.c_void_p), ("trace_rounds", C.c_int64), ("policy_K", C.c_int32), ("policy_R", C.c_int32), ("policy_rho_upper", C.c_double),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("storage", C.c_int32),
        ("fuse_rounds", C.c_int32), ("first_round", C.c_int64),
    ]

STORAGE = {"f32": 0, "bf16": 1}


_lib = None


def library_path() -> str:
    return _build.LIB


def lib():
    """Loads (building first if the sources are newer) the CUDA library; raises if it cannot."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.is_stale():
            path = _build.build()
        L = C.CDLL(path)
        vp, i32, i64, u64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_double
        sig = {
            "netmax_config_init": ([vp], C.c_int),
            "netmax_workspace_size": ([vp, vp], C.c_int),
            "netmax_create_ex": ([vp, vp], C.c_int),
            "netmax_create": ([i32, i64, vp, vp, dbl, u64, vp], C.c_int),
            "netmax_destroy": ([vp], None),
            "netmax_set_policy": ([vp, vp, vp, dbl], C.c_int),
            "netmax_get_policy": ([vp, vp, vp], C.c_int),
            "netmax_set_replicas": ([vp, vp], C.c_int),
            "netmax_set_centres": ([vp, vp], C.c_int),
            "netmax_round": ([vp, i64], C.c_int),
            "netmax_round_from_host": ([vp, vp, vp, i64, vp, i32], C.c_int),
            "netmax_rounds_done": ([vp], i64),
            "netmax_set_fuse_rounds": ([vp, i32], C.c_int),
            "netmax_read_replicas": ([vp, vp], C.c_int),
            "netmax_read_centres": ([vp, vp], C.c_int),
            "netmax_read_columns": ([vp, vp, i64, vp], C.c_int),
            "netmax_read_columns_static": ([vp, vp, i64, vp], C.c_int),
            "netmax_peer_trace": ([vp, i64, i64, vp], C.c_int),
            "netmax_telemetry": ([vp, i64, i64, vp, vp], C.c_int),
            "netmax_replicas_device": ([vp, vp, vp], C.c_int),
            "netmax_sample_peers": ([vp, i64, i64, vp], C.c_int),
            "netmax_measure": ([vp, vp, vp], C.c_int),
            "netmax_async_begin": ([vp, vp, dbl], C.c_int),
            "netmax_async_set_times": ([vp, vp], C.c_int),
            "netmax_async_steps": ([vp, i64], C.c_int),
            "netmax_async_time": ([vp, vp, vp], C.c_int),
            "netmax_async_trace": ([vp, i64, i64, vp, vp, vp, vp], C.c_int),
            "netmax_async_ema": ([vp, vp, vp], C.c_int),
            "netmax_async_monitor": ([vp, dbl], C.c_int),
            "netmax_async_monitor_refreshes": ([vp], i64),
            "netmax_iteration_times": ([i32, i64, vp, vp, vp], C.c_int),
            "netmax_policy_generate": ([i32, vp, vp, dbl, i32, i32, vp, vp, vp], C.c_int),
            "netmax_policy_generate_ex": ([i32, vp, vp, dbl, i32, i32, dbl, vp, vp, vp], C.c_int),
            "netmax_policy_generate_device": ([i32, vp, vp, dbl, i32, i32, dbl, i32, vp, vp, vp, vp], C.c_int),
            "netmax_policy_generate_fixed_weight": ([i32, vp, vp, dbl, i32, i32, dbl, vp, vp, vp], C.c_int),
            "netmax_policy_fixed_weight_at": ([i32, vp, vp, dbl, dbl, vp], C.c_int),
            "netmax_debug_absent_ctas": ([vp, i32], C.c_int),
            "netmax_kernel_launches": ([vp], i64),
            "netmax_last_error": ([vp], C.c_char_p),
        }
        for name, (args, res) in sig.items():
            fn = getattr(L, name)
            fn.argtypes, fn.restype = args, res
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f64(a, shape=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float64)
    if shape is not None and a.shape != shape:
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def _check(code: int, handle=None):
    if code != NETMAX_OK:
        msg = lib().netmax_last_error(handle)
        raise NetmaxError(code, msg.decode() if msg else "")


def netmax_iteration_times(link_speed_gbps, d: int):
    s = _f64(link_speed_gbps)
    M = s.shape[0]
    t = np.empty((M, M), dtype=np.float64)
    adj = np.empty((M, M), dtype=np.uint8)
    _check(lib().netmax_iteration_times(M, int(d), _p(s), _p(t), _p(adj)))
    return t, adj


def netmax_policy_generate(t_iter, adj, lr: float, K: int, R: int, rho_upper: float = 0.0):
    t = _f64(t_iter)
    M = t.shape[0]
    adj = np.ascontiguousarray(adj, dtype=np.uint8)
    P = np.empty((M, M), dtype=np.float64)
    rho = C.c_double()
    info = np.empty(5, dtype=np.float64)
    _check(lib().netmax_policy_generate_ex(M, _p(t), _p(adj), float(lr), int(K), int(R), float(rho_upper), _p(P),
                                           C.byref(rho), _p(info)))
    return P, rho.value, dict(lam2=info[0], tbar=info[1], t_conv=info[2], k=int(info[3]), r=int(info[4]))


def netmax_policy_generate_fixed_weight(t_iter, adj, pull_weight: float, K: int, R: int, floor_upper: float = 0.0):
    t = _f64(t_iter)
    M = t.shape[0]
    adj = np.ascontiguousarray(adj, dtype=np.uint8)
    P = np.empty((M, M), dtype=np.float64)
    floor = C.c_double()
    info = np.empty(5, dtype=np.float64)
    _check(lib().netmax_policy_generate_fixed_weight(M, _p(t), _p(adj), float(pull_weight), int(K), int(R), float(floor_upper),
                                                     _p(P), C.byref(floor), _p(info)))
    return P, floor.value, dict(lam2=info[0], tbar=info[1], t_conv=info[2], k=int(info[3]), r=int(info[4]))


def netmax_policy_fixed_weight_at(t_iter, adj, floor: float, t_bar: float):
    t = _f64(t_iter)
    M = t.shape[0]
    adj = np.ascontiguousarray(adj, dtype=np.uint8)
    P = np.empty((M, M), dtype=np.float64)
    _check(lib().netmax_policy_fixed_weight_at(M, _p(t), _p(adj), float(floor), float(t_bar), _p(P)))
    return P


def netmax_policy_generate_device(t_iter, adj, lr: float, K: int, R: int, device: int = 0, stream=None,
                                  rho_upper: float = 0.0):
    t = _f64(t_iter)
    M = t.shape[0]
    adj = np.ascontiguousarray(adj, dtype=np.uint8)
    P = np.empty((M, M), dtype=np.float64)
    rho = C.c_double()
    info = np.empty(5, dtype=np.float64)
    _check(lib().netmax_policy_generate_device(M, _p(t), _p(adj), float(lr), int(K), int(R), float(rho_upper), int(device), stream,
                                               _p(P), C.byref(rho), _p(info)))
    return P, rho.value, dict(lam2=info[0], tbar=info[1], t_conv=info[2], k=int(info[3]), r=int(info[4]))


class Netmax:
    """One simulator context (netmax_create_ex ... netmax_destroy)."""

    def __init__(self, M: int, d: int, lr: float, link_speed_gbps=None, prob=None, rho: float = 0.0,
                 sigma: float = 0.0, x0_std: float = 0.0, c_std: float = 0.0, objective: int = 1, seed: int = 0,
                 device: int = 0, stream: Optional[int] = None, trace_rounds: int = 1024, policy_K: int = 20,
                 policy_R: int = 20, workspace: Optional[int] = None, workspace_bytes: int = 0,
                 element_offset: int = 0, pull_weight: float = 0.0, policy_rho_upper: float = 0.0,
                 storage: str = "f32", fuse_rounds: int = 0, first_round: int = 0):
        L = lib()
        cfg = Config()
        _check(L.netmax_config_init(C.byref(cfg)))
        self._speed = _f64(link_speed_gbps, (M, M)) if link_speed_gbps is not None else None
        self._prob = _f64(prob, (M, M)) if prob is not None else None
        cfg.M, cfg.d, cfg.element_offset = int(M), int(d), int(element_offset)
        cfg.link_speed_gbps = self._speed.ctypes.data if self._speed is not None else None
        cfg.prob = self._prob.ctypes.data if self._prob is not None else None
        cfg.lr, cfg.rho, cfg.sigma = float(lr), float(rho), float(sigma)
        cfg.pull_weight = float(pull_weight)
        cfg.x0_std, cfg.c_std = float(x0_std), float(c_std)
        cfg.objective, cfg.seed, cfg.device = int(objective), int(seed), int(device)
        cfg.stream = stream
        cfg.trace_rounds = int(trace_rounds)
        cfg.policy_K, cfg.policy_R = int(policy_K), int(policy_R)
        cfg.policy_rho_upper = float(policy_rho_upper)
        cfg.workspace, cfg.workspace_bytes = workspace, int(workspace_bytes)
        cfg.storage = STORAGE[storage]
        cfg.fuse_rounds = int(fuse_rounds)
        cfg.first_round = int(first_round)
        self.first_round = int(first_round)
        self.storage = storage
        self.M, self.d = int(M), int(d)
        self._h = C.c_void_p()
        _check(L.netmax_create_ex(C.byref(cfg), C.byref(self._h)))

    @staticmethod
    def workspace_size(M: int, d: int, trace_rounds: int = 1024, storage: str = "f32") -> int:
        cfg = Config()
        _check(lib().netmax_config_init(C.byref(cfg)))
        cfg.M, cfg.d, cfg.trace_rounds = int(M), int(d), int(trace_rounds)
        cfg.storage = STORAGE[storage]
        out = C.c_size_t()
        _check(lib().netmax_workspace_size(C.byref(cfg), C.byref(out)))
        return out.value

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().netmax_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def set_policy(self, link_speed_gbps=None, prob=None, rho: float = 0.0):
        s = _f64(link_speed_gbps, (self.M, self.M)) if link_speed_gbps is not None else None
        p = _f64(prob, (self.M, self.M)) if prob is not None else None
        _check(lib().netmax_set_policy(self._h, _p(s), _p(p), float(rho)), self._h)

    def get_policy(self):
        P = np.empty((self.M, self.M), dtype=np.float64)
        rho = C.c_double()
        _check(lib().netmax_get_policy(self._h, _p(P), C.byref(rho)), self._h)
        return P, rho.value

    def set_replicas(self, x):
        _check(lib().netmax_set_replicas(self._h, self._host_plane(x)), self._h)

    def set_centres(self, c):
        _check(lib().netmax_set_centres(self._h, self._host_plane(c)), self._h)

    def _host_plane(self, a):
        """numpy array or host pointer (int) of M*d floats."""
        if isinstance(a, int):
            return C.c_void_p(a)
        a = np.ascontiguousarray(a, dtype=np.float32)
        if a.shape != (self.M, self.d):
            raise ValueError(f"expected shape {(self.M, self.d)}, got {a.shape}")
        self._keep = a
        return _p(a)

    def round(self, n_rounds: int = 1):
        _check(lib().netmax_round(self._h, int(n_rounds)), self._h)

    def round_from_host(self, x, c, n_rounds: int, out, n_chunks: int = 0):
        """netmax_round_from_host: x, c, out are numpy arrays (M, d) float32 or host pointers (int); x and c may be None."""
        def ptr(a):
            return None if a is None else self._host_plane(a)
        keep = [ptr(x), ptr(c)]
        if isinstance(out, int):
            po = C.c_void_p(out)
        else:
            assert out.dtype == np.float32 and out.shape == (self.M, self.d) and out.flags.c_contiguous
            po = _p(out)
        _check(lib().netmax_round_from_host(self._h, keep[0], keep[1], int(n_rounds), po, int(n_chunks)), self._h)
        return out

    def set_fuse_rounds(self, fuse_rounds: int):
        _check(lib().netmax_set_fuse_rounds(self._h, int(fuse_rounds)), self._h)

    @property
    def rounds_done(self) -> int:
        return int(lib().netmax_rounds_done(self._h))

    def read_replicas(self, out=None):
        if isinstance(out, int):
            _check(lib().netmax_read_replicas(self._h, C.c_void_p(out)), self._h)
            return None
        out = np.empty((self.M, self.d), dtype=np.float32) if out is None else out
        _check(lib().netmax_read_replicas(self._h, _p(out)), self._h)
        return out

    def read_centres(self):
        out = np.empty((self.M, self.d), dtype=np.float32)
        _check(lib().netmax_read_centres(self._h, _p(out)), self._h)
        return out

    def read_columns(self, cols):
        cols = np.ascontiguousarray(cols, dtype=np.int64)
        out = np.empty((self.M, cols.shape[0]), dtype=np.float32)
        _check(lib().netmax_read_columns(self._h, _p(cols), cols.shape[0], _p(out)), self._h)
        return out

    def read_columns_static(self, cols):
        """netmax_read_columns_static: the same read-back through the library's fixed staging
        array, for callers that must not allocate device memory (limits in the C header)."""
        cols = np.ascontiguousarray(cols, dtype=np.int64)
        out = np.empty((self.M, cols.shape[0]), dtype=np.float32)
        _check(lib().netmax_read_columns_static(self._h, _p(cols), cols.shape[0], _p(out)), self._h)
        return out

    def peer_trace(self, first_round: Optional[int] = None, n: Optional[int] = None):
        first_round = self.first_round if first_round is None else first_round
        n = self.rounds_done - first_round if n is None else n
        out = np.empty((n, self.M), dtype=np.int32)
        _check(lib().netmax_peer_trace(self._h, int(first_round), int(n), _p(out)), self._h)
        return out

    def telemetry(self, first_round: Optional[int] = None, n: Optional[int] = None):
        first_round = self.first_round if first_round is None else first_round
        n = self.rounds_done - first_round if n is None else n
        cons = np.empty(n, dtype=np.float64)
        loss = np.empty(n, dtype=np.float64)
        _check(lib().netmax_telemetry(self._h, int(first_round), int(n), _p(cons), _p(loss)), self._h)
        return cons, loss

    def replicas_device(self):
        ptr, ld = C.c_void_p(), C.c_int64()
        _check(lib().netmax_replicas_device(self._h, C.byref(ptr), C.byref(ld)), self._h)
        return ptr.value, ld.value

    def sample_peers(self, first_round: int, n_rounds: int, device_out: int):
        _check(lib().netmax_sample_peers(self._h, int(first_round), int(n_rounds), C.c_void_p(device_out)), self._h)

    def measure(self):
        cons, loss = C.c_double(), C.c_double()
        _check(lib().netmax_measure(self._h, C.byref(cons), C.byref(loss)), self._h)
        return cons.value, loss.value

    # ---- asynchronous timeline (one worker per global step)
    def async_begin(self, t_iter=None, beta: float = 0.9):
        t = _f64(t_iter, (self.M, self.M)) if t_iter is not None else None
        _check(lib().netmax_async_begin(self._h, _p(t), float(beta)), self._h)

    def async_set_times(self, t_iter):
        t = _f64(t_iter, (self.M, self.M))
        _check(lib().netmax_async_set_times(self._h, _p(t)), self._h)

    def async_steps(self, n_steps: int):
        _check(lib().netmax_async_steps(self._h, int(n_steps)), self._h)

    def async_monitor(self, period_s: float):
        _check(lib().netmax_async_monitor(self._h, float(period_s)), self._h)

    @property
    def async_monitor_refreshes(self) -> int:
        return int(lib().netmax_async_monitor_refreshes(self._h))

    def async_time(self):
        t, k = C.c_double(), C.c_int64()
        _check(lib().netmax_async_time(self._h, C.byref(t), C.byref(k)), self._h)
        return t.value, k.value

    def async_trace(self, first_step: int = 0, n: Optional[int] = None):
        n = self.async_time()[1] - first_step if n is None else n
        worker = np.empty(n, dtype=np.int32)
        peer = np.empty(n, dtype=np.int32)
        local_iter = np.empty(n, dtype=np.int64)
        time = np.empty(n, dtype=np.float64)
        _check(lib().netmax_async_trace(self._h, int(first_step), int(n), _p(worker), _p(peer), _p(local_iter),
                                        _p(time)), self._h)
        return worker, peer, local_iter, time

    def async_ema(self):
        ema = np.empty((self.M, self.M), dtype=np.float64)
        count = np.empty((self.M, self.M), dtype=np.int64)
        _check(lib().netmax_async_ema(self._h, _p(ema), _p(count)), self._h)
        return ema, count

    def debug_absent_ctas(self, n: int):
        _check(lib().netmax_debug_absent_ctas(self._h, int(n)), self._h)

    @property
    def kernel_launches(self) -> int:
        return int(lib().netmax_kernel_launches(self._h))
