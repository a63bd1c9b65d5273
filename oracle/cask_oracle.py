"""numpy front end of the CPU oracle (``cask_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu_baseline leg may import
this module; the CUDA library and its binding never do.  It compiles the C file
with gcc on first use (``build()``) and marshals numpy arrays; it adds no
arithmetic of its own.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cask_oracle.c")
_LIB = os.path.join(_HERE, "libcask_oracle.so")
_lib = None

NOOP_UNDER_BUDGET = 1
PREFIX_EVICTED = 2
DECODE_CONSOLIDATED = 4
PREFIX_BUDGET_EXHAUSTED = 8
MERGE_INACTIVE = 16

PLAN_FIELDS = ("B_p", "P_keep", "B_d", "r", "c", "m", "flags", "n_out")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.cask_oracle_threads.restype = C.c_int
    return _lib


def threads() -> int:
    return int(lib().cask_oracle_threads())


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def score(K, Q, causal: int = 1, lse_in=None):
    """K [T,d], Q [g,W,d] (float32 values) -> (s [T] float64, lse [g,W] float64)."""
    K, Q = _f32(K), _f32(Q)
    T, d = K.shape
    g, W, _ = Q.shape
    s = np.zeros(T, dtype=np.float64)
    lse = np.zeros((g, W), dtype=np.float64)
    li = None if lse_in is None else np.ascontiguousarray(lse_in, dtype=np.float64)
    lib().cask_oracle_score(_p(K, C.c_float), _p(Q, C.c_float), T, d, g, W, int(causal),
                            _p(li, C.c_double), _p(s, C.c_double), _p(lse, C.c_double))
    return s, lse


def plan(T: int, P: int, B: int, reserve: int, W: int, gamma: float = 0.5) -> np.ndarray:
    out = np.zeros(8, dtype=np.int32)
    lib().cask_oracle_plan(int(T), int(P), int(B), int(reserve), int(W), C.c_double(gamma), _p(out, C.c_int))
    return out


def prefix_evict(s, P: int, pl: np.ndarray, kind: np.ndarray) -> None:
    s = np.ascontiguousarray(s, dtype=np.float64)
    lib().cask_oracle_prefix_evict(_p(s, C.c_double), int(P), _p(pl, C.c_int), _p(kind, C.c_uint8))


def select_core(s, T: int, P: int, pl: np.ndarray, kind: np.ndarray) -> None:
    s = np.ascontiguousarray(s, dtype=np.float64)
    lib().cask_oracle_select_core(_p(s, C.c_double), int(T), int(P), _p(pl, C.c_int), _p(kind, C.c_uint8))


def consolidate(K, s, P: int, pl: np.ndarray, kind: np.ndarray, tau: float = 0.9, eps: float = 1e-9, mass_in=None,
                chan_w=None, band_w=None, band_layout: int = 0):
    """Updates ``kind`` in place; returns dict(seed_of, weight, sim, sim2, flags, lost_mass)."""
    K = _f32(K)
    T, d = K.shape
    s = np.ascontiguousarray(s, dtype=np.float64)
    seed_of = np.full(T, -1, dtype=np.int32)
    weight = np.zeros(T, dtype=np.float64)
    sim = np.zeros(T, dtype=np.float64)
    sim2 = np.zeros(T, dtype=np.float64)
    mass_in = None if mass_in is None else np.ascontiguousarray(mass_in, dtype=np.float64)
    chan_w = None if chan_w is None else np.ascontiguousarray(chan_w, dtype=np.float32)
    band_w = None if band_w is None else np.ascontiguousarray(band_w, dtype=np.float32)
    assert band_w is None or (chan_w is None and band_w.shape == (d // 2,))
    lost = C.c_double(0.0)
    fn = lib().cask_oracle_consolidate
    fn.restype = C.c_int
    fl = fn(_p(K, C.c_float), _p(s, C.c_double), T, int(P), d, _p(pl, C.c_int), C.c_double(tau),
            C.c_double(eps), _p(mass_in, C.c_double), _p(chan_w, C.c_float), _p(band_w, C.c_float), int(band_layout),
            _p(kind, C.c_uint8), _p(seed_of, C.c_int),
            _p(weight, C.c_double), _p(sim, C.c_double), _p(sim2, C.c_double), C.byref(lost))
    return dict(seed_of=seed_of, weight=weight, sim=sim, sim2=sim2, flags=int(fl), lost_mass=lost.value)


def compact(K, V, kind, seed_of, weight, s, eps: float = 1e-9, mass_in=None):
    """Returns dict(k_out, v_out [n_out,d] float64, n_out, slot_src, slot_kind, slot_mass, assign, weight)."""
    K, V = _f32(K), _f32(V)
    T, d = K.shape
    kind = np.ascontiguousarray(kind, dtype=np.uint8)
    seed_of = np.ascontiguousarray(seed_of, dtype=np.int32)
    weight = np.array(weight, dtype=np.float64, copy=True)
    s = np.ascontiguousarray(s, dtype=np.float64)
    cap = int(np.count_nonzero((kind >= 1) & (kind <= 4)))
    k_out = np.zeros((max(cap, 1), d), dtype=np.float64)
    v_out = np.zeros((max(cap, 1), d), dtype=np.float64)
    slot_src = np.zeros(max(cap, 1), dtype=np.int32)
    slot_kind = np.zeros(max(cap, 1), dtype=np.uint8)
    slot_mass = np.zeros(max(cap, 1), dtype=np.float64)
    assign = np.zeros(T, dtype=np.int32)
    mass_in = None if mass_in is None else np.ascontiguousarray(mass_in, dtype=np.float64)
    n_out = C.c_int(0)
    lib().cask_oracle_compact(_p(K, C.c_float), _p(V, C.c_float), T, d, _p(kind, C.c_uint8),
                              _p(seed_of, C.c_int), _p(weight, C.c_double), _p(s, C.c_double),
                              C.c_double(eps), _p(mass_in, C.c_double), _p(k_out, C.c_double), _p(v_out, C.c_double),
                              C.byref(n_out), _p(slot_src, C.c_int), _p(slot_kind, C.c_uint8),
                              _p(slot_mass, C.c_double), _p(assign, C.c_int))
    n = n_out.value
    return dict(k_out=k_out[:n], v_out=v_out[:n], n_out=n, slot_src=slot_src[:n], slot_kind=slot_kind[:n],
                slot_mass=slot_mass[:n], assign=assign, weight=weight)


def dispersion(K, s, kind, assign, k_rep, eps: float = 1e-9, mass_in=None, chan_w=None, band_w=None,
               band_layout: int = 0) -> float:
    """Within-group dispersion of one unit (Sec. 2.6): sum_i a_i ||k_i - k_rep[assign[i]]|| over the rows of kind 4/5.
    ``k_rep`` [n_out, d] holds the representatives as stored (rounded to the cache dtype by the caller)."""
    K = _f32(K)
    T, d = K.shape
    s = np.ascontiguousarray(s, dtype=np.float64)
    kind = np.ascontiguousarray(kind, dtype=np.uint8)
    assign = np.ascontiguousarray(assign, dtype=np.int32)
    k_rep = _f32(k_rep)
    mass_in = None if mass_in is None else np.ascontiguousarray(mass_in, dtype=np.float64)
    chan_w = None if chan_w is None else np.ascontiguousarray(chan_w, dtype=np.float32)
    band_w = None if band_w is None else np.ascontiguousarray(band_w, dtype=np.float32)
    fn = lib().cask_oracle_dispersion
    fn.restype = C.c_double
    return float(fn(_p(K, C.c_float), _p(s, C.c_double), T, d, C.c_double(eps), _p(mass_in, C.c_double),
                    _p(kind, C.c_uint8), _p(assign, C.c_int), _p(k_rep, C.c_float), _p(chan_w, C.c_float),
                    _p(band_w, C.c_float), int(band_layout)))


def event_batch(K, V, Q, tok_off, P, B, reserve, causal: int = 1, gamma: float = 0.5, tau: float = 0.9,
                eps: float = 1e-9, mass_in=None, chan_w=None, band_w=None, band_layout: int = 0) -> Dict[str, np.ndarray]:
    """Whole event for many contiguous units.  K, V [sum T, d]; Q [n, g, W, d] (float32 values)."""
    K, V, Q = _f32(K), _f32(V), _f32(Q)
    n, g, W, d = Q.shape
    tok_off = np.ascontiguousarray(tok_off, dtype=np.int64)
    P = np.ascontiguousarray(P, dtype=np.int32)
    B = np.ascontiguousarray(B, dtype=np.int32)
    reserve = np.ascontiguousarray(reserve, dtype=np.int32)
    Tt = int(tok_off[-1])
    Bmax = max(int(np.max(B)) if n else 1, 1)      # n_out <= B always (a unit under budget has T <= B)
    o = dict(
        s=np.zeros(Tt, np.float64), plan=np.zeros((n, 8), np.int32), kind=np.zeros(Tt, np.uint8),
        seed_of=np.zeros(Tt, np.int32), weight=np.zeros(Tt, np.float64), sim=np.zeros(Tt, np.float64),
        sim2=np.zeros(Tt, np.float64), k_out=np.zeros((n, Bmax, d), np.float64),
        v_out=np.zeros((n, Bmax, d), np.float64), n_out=np.zeros(n, np.int32),
        slot_src=np.zeros((n, Bmax), np.int32), slot_kind=np.zeros((n, Bmax), np.uint8),
        slot_mass=np.zeros((n, Bmax), np.float64), assign=np.zeros(Tt, np.int32),
        status=np.zeros(n, np.int32), lost_mass=np.zeros(n, np.float64), rho=np.zeros((n, 2), np.float64))
    mass_in = None if mass_in is None else np.ascontiguousarray(mass_in, dtype=np.float64)
    chan_w = None if chan_w is None else np.ascontiguousarray(chan_w, dtype=np.float32)
    band_w = None if band_w is None else np.ascontiguousarray(band_w, dtype=np.float32)
    assert band_w is None or (chan_w is None and band_w.shape == (d // 2,))
    lib().cask_oracle_event_batch(
        n, _p(K, C.c_float), _p(V, C.c_float), _p(Q, C.c_float), _p(tok_off, C.c_int64), _p(P, C.c_int),
        _p(B, C.c_int), _p(reserve, C.c_int), d, g, W, int(causal), C.c_double(gamma), C.c_double(tau),
        C.c_double(eps), _p(mass_in, C.c_double), _p(chan_w, C.c_float), _p(band_w, C.c_float), int(band_layout), Bmax,
        _p(o["s"], C.c_double), _p(o["plan"], C.c_int), _p(o["kind"], C.c_uint8),
        _p(o["seed_of"], C.c_int), _p(o["weight"], C.c_double), _p(o["sim"], C.c_double),
        _p(o["sim2"], C.c_double), _p(o["k_out"], C.c_double), _p(o["v_out"], C.c_double),
        _p(o["n_out"], C.c_int), _p(o["slot_src"], C.c_int), _p(o["slot_kind"], C.c_uint8),
        _p(o["slot_mass"], C.c_double), _p(o["assign"], C.c_int), _p(o["status"], C.c_int),
        _p(o["lost_mass"], C.c_double), _p(o["rho"], C.c_double))
    o["Bmax"] = Bmax
    o["rho_core"], o["rho_rep"] = o["rho"][:, 0].copy(), o["rho"][:, 1].copy()
    return o


def event(K, V, Q, P: int, B: int, reserve: int, **kw) -> Dict[str, np.ndarray]:
    """Whole event for one unit; same keys as ``event_batch`` with the unit axis removed."""
    K = _f32(K)
    T = K.shape[0]
    o = event_batch(K, V, _f32(Q)[None], np.array([0, T], np.int64), [P], [B], [reserve], **kw)
    n = int(o["n_out"][0])
    out = dict(o)
    for key in ("k_out", "v_out", "slot_src", "slot_kind", "slot_mass"):
        out[key] = o[key][0][:n]
    out["plan"] = o["plan"][0]
    out["n_out"] = n
    out["status"] = int(o["status"][0])
    out["lost_mass"] = float(o["lost_mass"][0])
    out["rho_core"], out["rho_rep"] = float(o["rho_core"][0]), float(o["rho_rep"][0])
    return out


def score_stats(K, mu, pi, delta_grid, omega, band_layout: int = 0, delta=None) -> np.ndarray:
    """Horizon-averaged mean score of one unit (App. B): K [T,d]; mu [g, d/2, 2]; pi [g, n_delta]; delta_grid
    [n_delta]; omega [d/2]; optional per-row offsets delta [T] (default T-1-i).  Returns s [T] float64."""
    K = _f32(K)
    T, d = K.shape
    mu = np.ascontiguousarray(mu, dtype=np.float32)
    g = mu.shape[0]
    pi = np.ascontiguousarray(pi, dtype=np.float64)
    delta_grid = np.ascontiguousarray(delta_grid, dtype=np.float64)
    omega = np.ascontiguousarray(omega, dtype=np.float64)
    assert mu.shape == (g, d // 2, 2) and pi.shape == (g, delta_grid.size) and omega.shape == (d // 2,)
    delta = None if delta is None else np.ascontiguousarray(delta, dtype=np.float64)
    s = np.zeros(T, np.float64)
    lib().cask_oracle_score_stats(_p(K, C.c_float), T, d, g, _p(mu, C.c_float), _p(pi, C.c_double),
                                  _p(delta_grid, C.c_double), int(delta_grid.size), _p(omega, C.c_double),
                                  int(band_layout), _p(delta, C.c_double), _p(s, C.c_double))
    return s


def score_batch(K, Q, tok_off, causal: int = 1):
    K, Q = _f32(K), _f32(Q)
    n, g, W, d = Q.shape
    tok_off = np.ascontiguousarray(tok_off, dtype=np.int64)
    s = np.zeros(int(tok_off[-1]), np.float64)
    lse = np.zeros((n, g, W), np.float64)
    lib().cask_oracle_score_batch(n, _p(K, C.c_float), _p(Q, C.c_float), _p(tok_off, C.c_int64), d, g, W,
                                  int(causal), _p(s, C.c_double), _p(lse, C.c_double))
    return s, lse


def round_bf16(x) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.zeros(x.shape, dtype=np.float32)
    lib().cask_oracle_round_bf16(_p(x, C.c_double), C.c_size_t(x.size), _p(out, C.c_float))
    return out
