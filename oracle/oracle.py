"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not the product).

Builds ``netmax_oracle.cpp`` with g++ on first use and exposes its functions with numpy
arrays.  Only tests, the smoke check and the benchmark's cpu_baseline / reference legs
may import this module; the CUDA library never does, and this module never imports it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "netmax_oracle.cpp")
_LIB = os.path.join(_HERE, "libnetmax_oracle.so")
_lock = threading.Lock()
_lib = None

TAG_PEER, TAG_NOISE, TAG_X0, TAG_C = 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile the oracle (plain g++, no fast-math, no FMA contraction)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-ffp-contract=off",
                   "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        vp, i32, i64, u32, u64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_double
        L.nmo_philox4x32_10.argtypes = [vp, vp, vp]
        L.nmo_philox_blocks.argtypes = [u64, u32, u32, u32, u32, i64, vp]
        L.nmo_noise.argtypes = [u64, i32, u64, i64, i64, vp]
        L.nmo_normals_from_words.argtypes = [vp, vp]
        L.nmo_build_thresholds.argtypes = [i32, vp, vp, vp]
        L.nmo_sample.argtypes = [vp, i32, i32, u32]
        L.nmo_sample.restype = i32
        L.nmo_build_weights.argtypes = [i32, vp, vp, dbl, dbl, vp]
        L.nmo_peer_draws.argtypes = [i32, vp, u64, u64, i64, vp]
        L.nmo_sim_create.argtypes = [i32, i64, vp, i64, vp, vp, dbl, dbl, dbl, i32, u64]
        L.nmo_sim_create.restype = vp
        L.nmo_sim_destroy.argtypes = [vp]
        L.nmo_sim_set_fixed_weight.argtypes = [vp, dbl]
        L.nmo_sim_set_policy.argtypes = [vp, vp, vp, dbl]
        L.nmo_sim_init.argtypes = [vp, dbl, dbl]
        for name in ("nmo_sim_set_x", "nmo_sim_set_c", "nmo_sim_get_x", "nmo_sim_get_c", "nmo_sim_get_unrounded"):
            getattr(L, name).argtypes = [vp, vp]
        L.nmo_sim_set_storage.argtypes = [vp, i32]
        L.nmo_bf16_round.argtypes = [vp, i64, vp]
        L.nmo_sim_round.argtypes = [vp, i64, i32]
        L.nmo_sim_rounds_done.argtypes = [vp]
        L.nmo_sim_rounds_done.restype = i64
        L.nmo_sim_set_first_round.argtypes = [vp, u64]
        L.nmo_sim_get_trace.argtypes = [vp, i64, i64, vp]
        L.nmo_sim_get_telemetry.argtypes = [vp, i64, i64, vp, vp]
        L.nmo_sim_telemetry_now.argtypes = [vp, vp, vp]
        L.nmo_async_begin.argtypes = [vp, vp, dbl]
        L.nmo_async_set_times.argtypes = [vp, vp]
        L.nmo_async_steps.argtypes = [vp, i64]
        L.nmo_async_steps_done.argtypes = [vp]
        L.nmo_async_steps_done.restype = i64
        L.nmo_async_now.argtypes = [vp]
        L.nmo_async_now.restype = dbl
        L.nmo_async_next_time.argtypes = [vp]
        L.nmo_async_next_time.restype = dbl
        L.nmo_async_trace.argtypes = [vp, i64, i64, vp, vp, vp, vp]
        L.nmo_async_ema.argtypes = [vp, vp, vp]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr = np.ascontiguousarray(ctr, dtype=np.uint32)
    key = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    lib().nmo_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def philox_blocks(seed: int, c0_first: int, c1: int, c2: int, c3: int, n: int) -> np.ndarray:
    out = np.empty((n, 4), dtype=np.uint32)
    lib().nmo_philox_blocks(seed, c0_first, c1, c2, c3, n, _p(out))
    return out


def noise(seed: int, worker: int, rnd: int, e0: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.float64)
    lib().nmo_noise(seed, worker, rnd, e0, n, _p(out))
    return out


def normals_from_words(words) -> np.ndarray:
    words = np.ascontiguousarray(words, dtype=np.uint32)
    out = np.empty(4, dtype=np.float64)
    lib().nmo_normals_from_words(_p(words), _p(out))
    return out


def bf16_round(values) -> np.ndarray:
    """fp32 values rounded to the nearest bfloat16 (ties to even), returned as fp32."""
    v = np.ascontiguousarray(values, dtype=np.float32)
    out = np.empty_like(v)
    lib().nmo_bf16_round(_p(v), v.size, _p(out))
    return out


def build_thresholds(P: np.ndarray):
    P = np.ascontiguousarray(P, dtype=np.float64)
    M = P.shape[0]
    T = np.empty((M, M), dtype=np.uint32)
    last = np.empty(M, dtype=np.int32)
    lib().nmo_build_thresholds(M, _p(P), _p(T), _p(last))
    return T, last


def sample(Trow: np.ndarray, last_nz: int, u: int) -> int:
    Trow = np.ascontiguousarray(Trow, dtype=np.uint32)
    return int(lib().nmo_sample(_p(Trow), Trow.shape[0], int(last_nz), int(u)))


def build_weights(P: np.ndarray, adj: np.ndarray, alpha: float, rho: float) -> np.ndarray:
    P = np.ascontiguousarray(P, dtype=np.float64)
    adj = np.ascontiguousarray(adj, dtype=np.uint8)
    M = P.shape[0]
    w = np.empty((M, M), dtype=np.float32)
    lib().nmo_build_weights(M, _p(P), _p(adj), float(alpha), float(rho), _p(w))
    return w


def peer_draws(P: np.ndarray, seed: int, first_round: int, n_rounds: int) -> np.ndarray:
    P = np.ascontiguousarray(P, dtype=np.float64)
    M = P.shape[0]
    out = np.empty((n_rounds, M), dtype=np.int32)
    lib().nmo_peer_draws(M, _p(P), seed, first_round, n_rounds, _p(out))
    return out


class Sim:
    """The round simulator: all M replicas (or a sample of their columns) on the CPU."""

    def __init__(self, M, d, P, adj, alpha, rho, sigma, objective, seed, cols=None, pull_weight=0.0, storage="f32",
                 first_round=0):
        self.M, self.d = int(M), int(d)
        self._P = np.ascontiguousarray(P, dtype=np.float64)
        self._adj = np.ascontiguousarray(adj, dtype=np.uint8)
        assert self._P.shape == (M, M) and self._adj.shape == (M, M)
        if cols is None:
            self.ncols, cptr = self.d, None
        else:
            self._cols = np.ascontiguousarray(cols, dtype=np.int64)
            self.ncols, cptr = int(self._cols.shape[0]), _p(self._cols)
        self._h = lib().nmo_sim_create(self.M, self.d, cptr, self.ncols, _p(self._P), _p(self._adj), float(alpha),
                                       float(rho), float(sigma), int(objective), int(seed))
        if pull_weight > 0.0:      # fixed pull weight (gossip / AD-PSGD style averaging)
            lib().nmo_sim_set_fixed_weight(self._h, float(pull_weight))
            lib().nmo_sim_set_policy(self._h, _p(self._P), _p(self._adj), float(rho))
        assert storage in ("f32", "bf16")
        self.storage = storage
        if storage == "bf16":      # bfloat16 state, fp32 arithmetic, one rounding per stored value
            lib().nmo_sim_set_storage(self._h, 1)
        if first_round:            # rounds numbered from here (trace and telemetry indices stay relative)
            lib().nmo_sim_set_first_round(self._h, int(first_round))

    def close(self):
        if self._h:
            lib().nmo_sim_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:       # (at interpreter exit the module's globals may already be gone)
            pass

    def set_policy(self, P, adj, rho):
        P = np.ascontiguousarray(P, dtype=np.float64)
        adj = np.ascontiguousarray(adj, dtype=np.uint8)
        lib().nmo_sim_set_policy(self._h, _p(P), _p(adj), float(rho))

    def init(self, x0_std, c_std):
        lib().nmo_sim_init(self._h, float(x0_std), float(c_std))

    def set_x(self, x):
        x = np.ascontiguousarray(x, dtype=np.float32)
        assert x.shape == (self.M, self.ncols)
        lib().nmo_sim_set_x(self._h, _p(x))

    def set_c(self, c):
        c = np.ascontiguousarray(c, dtype=np.float32)
        assert c.shape == (self.M, self.ncols)
        lib().nmo_sim_set_c(self._h, _p(c))

    def x(self) -> np.ndarray:
        out = np.empty((self.M, self.ncols), dtype=np.float32)
        lib().nmo_sim_get_x(self._h, _p(out))
        return out

    def c(self) -> np.ndarray:
        out = np.empty((self.M, self.ncols), dtype=np.float32)
        lib().nmo_sim_get_c(self._h, _p(out))
        return out

    def unrounded(self) -> np.ndarray:
        """bf16 storage: the last round's new parameters in fp32, before the rounding to bfloat16."""
        assert self.storage == "bf16"
        out = np.empty((self.M, self.ncols), dtype=np.float32)
        lib().nmo_sim_get_unrounded(self._h, _p(out))
        return out

    def round(self, n=1, threads=1):
        lib().nmo_sim_round(self._h, int(n), int(threads))

    @property
    def rounds_done(self) -> int:
        return int(lib().nmo_sim_rounds_done(self._h))

    def trace(self, first=0, n=None) -> np.ndarray:
        n = self.rounds_done - first if n is None else n
        out = np.empty((n, self.M), dtype=np.int32)
        lib().nmo_sim_get_trace(self._h, first, n, _p(out))
        return out

    def telemetry(self, first=0, n=None):
        n = self.rounds_done - first if n is None else n
        cons = np.empty(n, dtype=np.float64)
        loss = np.empty(n, dtype=np.float64)
        lib().nmo_sim_get_telemetry(self._h, first, n, _p(cons), _p(loss))
        return cons, loss

    # ---- asynchronous timeline (the paper's one-worker-per-global-step process)
    def async_begin(self, t_iter, beta):
        t = np.ascontiguousarray(t_iter, dtype=np.float64)
        assert t.shape == (self.M, self.M)
        lib().nmo_async_begin(self._h, _p(t), float(beta))

    def async_set_times(self, t_iter):
        t = np.ascontiguousarray(t_iter, dtype=np.float64)
        lib().nmo_async_set_times(self._h, _p(t))

    def async_steps(self, n):
        lib().nmo_async_steps(self._h, int(n))

    @property
    def async_steps_done(self) -> int:
        return int(lib().nmo_async_steps_done(self._h))

    @property
    def async_now(self) -> float:
        return float(lib().nmo_async_now(self._h))

    @property
    def async_next_time(self) -> float:
        return float(lib().nmo_async_next_time(self._h))

    def async_trace(self, first=0, n=None):
        n = self.async_steps_done - first if n is None else n
        worker = np.empty(n, dtype=np.int32)
        peer = np.empty(n, dtype=np.int32)
        local_iter = np.empty(n, dtype=np.int64)
        time = np.empty(n, dtype=np.float64)
        lib().nmo_async_trace(self._h, first, n, _p(worker), _p(peer), _p(local_iter), _p(time))
        return worker, peer, local_iter, time

    def async_ema(self):
        ema = np.empty((self.M, self.M), dtype=np.float64)
        count = np.empty((self.M, self.M), dtype=np.int64)
        lib().nmo_async_ema(self._h, _p(ema), _p(count))
        return ema, count

    def telemetry_now(self):
        a, b = C.c_double(), C.c_double()
        lib().nmo_sim_telemetry_now(self._h, C.byref(a), C.byref(b))
        return a.value, b.value
