"""ctypes wrapper around ``morphkv_oracle.c`` -- TEST INFRASTRUCTURE only.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It shares nothing with the CUDA path.  ``build()`` compiles the C
file with gcc next to this file; every other function marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "morphkv_oracle.c")
_LIB = os.path.join(_HERE, "libmorphkv_oracle.so")
_lock = threading.Lock()
_lib = None

SUM, MAX = 0, 1
FUSION = {"sum": SUM, "max": MAX}


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2, strict IEEE: no -ffast-math)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        dp, lp, ip = C.POINTER(C.c_double), C.POINTER(C.c_long), C.POINTER(C.c_int)
        lib.ora_create.restype = C.c_void_p
        lib.ora_create.argtypes = [C.c_int] * 7
        lib.ora_destroy.argtypes = [C.c_void_p]
        lib.ora_set_norm_mode.argtypes = [C.c_void_p, C.c_int]
        lib.ora_set_norm_mode.restype = None
        lib.ora_prefill.argtypes = [C.c_void_p, dp, dp, dp, C.c_int]
        lib.ora_prefill_forced.argtypes = [C.c_void_p, dp, dp, dp, C.c_int, lp, C.c_int]
        lib.ora_step.argtypes = [C.c_void_p, dp, dp, dp, dp, lp, C.c_int]
        lib.ora_count.argtypes = [C.c_void_p]
        lib.ora_next_pos.argtypes = [C.c_void_p]
        lib.ora_next_pos.restype = C.c_long
        lib.ora_cache_positions.argtypes = [C.c_void_p, lp]
        lib.ora_cache_row.argtypes = [C.c_void_p, C.c_long, dp, dp]
        lib.ora_last_scores.argtypes = [C.c_void_p, lp, dp]
        lib.ora_last_evicted.argtypes = [C.c_void_p, lp]
        lib.ora_last_boundary.argtypes = [C.c_void_p, dp, dp]
        lib.ora_window_stats.argtypes = [C.c_void_p, C.c_long, C.c_int, dp, dp]
        lib.ora_fuse_select.argtypes = [dp, C.c_int, C.c_int, C.c_int, C.c_int, dp, ip]
        _lib = lib
    return _lib


def _dp(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _lp(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_long))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


class Unit:
    """One MorphKV unit: a (layer, batch row, KV head) cache serving G query heads."""

    def __init__(self, G: int, d: int, C_: int, R: int, fusion, evict_interval: int = 1, recompute: bool = False,
                 norm: str = "frozen"):
        self.lib = _load()
        self.G, self.d, self.C, self.R, self.T = G, d, C_, R, evict_interval
        fusion = FUSION[fusion] if isinstance(fusion, str) else int(fusion)
        self.h = self.lib.ora_create(G, d, C_, R, fusion, evict_interval, int(recompute))
        if not self.h:
            raise ValueError("ora_create rejected the parameters")
        if norm not in ("frozen", "current"):
            raise ValueError(norm)
        self.lib.ora_set_norm_mode(self.h, int(norm == "current"))
        self.cap = C_ + R + evict_interval

    def __del__(self):
        h, self.h = getattr(self, "h", None), None
        if h:
            self.lib.ora_destroy(h)

    def prefill(self, k, v, q_window, forced=None) -> None:
        """k, v [P,d]; q_window [G, min(R,P), d] (last prompt positions, oldest first).  `forced`: the prompt
        positions to evict instead of the oracle's own choice (harness resync after a near tie)."""
        k, v, qw = _f64(k), _f64(v), _f64(q_window)
        P = k.shape[0]
        assert k.shape == (P, self.d) and v.shape == (P, self.d)
        assert qw.shape == (self.G, min(self.R, P), self.d), qw.shape
        self._scores_cap = max(self.cap, P)
        if forced is None or len(forced) == 0:
            rc = self.lib.ora_prefill(self.h, _dp(k), _dp(v), _dp(qw), P)
        else:
            farr = np.ascontiguousarray(np.asarray(forced, dtype=np.int64))
            rc = self.lib.ora_prefill_forced(self.h, _dp(k), _dp(v), _dp(qw), P, _lp(farr), len(farr))
        if rc:
            raise RuntimeError(f"ora_prefill failed ({rc})")

    def step(self, q, k_new, v_new, forced=None) -> np.ndarray:
        """q [G,d], k_new/v_new [d] -> attention output [G,d] (float64)."""
        q, k_new, v_new = _f64(q), _f64(k_new), _f64(v_new)
        assert q.shape == (self.G, self.d) and k_new.shape == (self.d,) and v_new.shape == (self.d,)
        out = np.empty((self.G, self.d), dtype=np.float64)
        if forced is None or len(forced) == 0:
            fptr, nf = None, 0
        else:
            farr = np.ascontiguousarray(np.asarray(forced, dtype=np.int64))
            fptr, nf = _lp(farr), len(farr)
        rc = self.lib.ora_step(self.h, _dp(q), _dp(k_new), _dp(v_new), _dp(out), fptr, nf)
        if rc:
            raise RuntimeError(f"ora_step failed ({rc})")
        return out

    @property
    def count(self) -> int:
        return self.lib.ora_count(self.h)

    @property
    def next_pos(self) -> int:
        return self.lib.ora_next_pos(self.h)

    def positions(self) -> np.ndarray:
        buf = np.empty(self.cap, dtype=np.int64)
        n = self.lib.ora_cache_positions(self.h, _lp(buf))
        return np.sort(buf[:n])

    def row(self, p: int):
        k = np.empty(self.d, dtype=np.float64)
        v = np.empty(self.d, dtype=np.float64)
        if self.lib.ora_cache_row(self.h, int(p), _dp(k), _dp(v)):
            raise KeyError(p)
        return k, v

    def last_scores(self):
        """Candidates of the last selection as (positions, F), sorted (F desc, pos asc)."""
        cap = max(self.cap, getattr(self, "_scores_cap", 0))      # a prompt can hold more candidates than slots
        p = np.empty(cap, dtype=np.int64)
        f = np.empty(cap, dtype=np.float64)
        n = self.lib.ora_last_scores(self.h, _lp(p), _dp(f))
        return p[:n].copy(), f[:n].copy()

    def last_evicted(self) -> np.ndarray:
        p = np.empty(self.cap, dtype=np.int64)
        n = self.lib.ora_last_evicted(self.h, _lp(p))
        return p[:n].copy()

    def last_boundary(self):
        """(C-th, (C+1)-th) largest fused score of the last selection; NaN when none ran."""
        a, b = C.c_double(), C.c_double()
        self.lib.ora_last_boundary(self.h, C.byref(a), C.byref(b))
        return a.value, b.value

    def window_stats(self, p: int, g: int):
        m, l = C.c_double(), C.c_double()
        if self.lib.ora_window_stats(self.h, int(p), g, C.byref(m), C.byref(l)):
            raise KeyError(p)
        return m.value, l.value


def fuse_select(S, C_: int, fusion):
    """Eq. 5/6 fusion of group-summed rows S [R,n] followed by Top_C -> (F [n], keep [n] bool)."""
    S = _f64(S)
    R, n = S.shape
    F = np.empty(n, dtype=np.float64)
    keep = np.empty(n, dtype=np.int32)
    fusion = FUSION[fusion] if isinstance(fusion, str) else int(fusion)
    _load().ora_fuse_select(_dp(S), R, n, C_, fusion, _dp(F), keep.ctypes.data_as(C.POINTER(C.c_int)))
    return F, keep.astype(bool)


def boundary_is_near_tie(kth: float, k1th: float, rel: float = 1e-3) -> bool:
    """True when the C-th and (C+1)-th fused scores are too close for the retained set to be unique:
    relative gap <= ``rel``."""
    if np.isnan(kth) or np.isnan(k1th):
        return False
    return abs(kth - k1th) <= rel * max(abs(kth), abs(k1th))
