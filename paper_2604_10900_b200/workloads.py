"""Seeded synthetic KV caches shaped like the reasoning and prompt-heavy workloads.

This module holds no arithmetic of the compression method: it only draws
keys, values and window queries with a stated distribution and rounds them to
the cache dtype.  It serves both the CPU oracle's tests and the CUDA path, so
both sides see byte-identical inputs.  It depends on numpy alone.

Recipe (one *unit* = one sequence x layer x KV head):

* generator ``numpy.random.Generator(PCG64(SeedSequence([2604, 10900, cfg,
  seq, layer, head])))``; the per-channel key scale is drawn from the stream
  ``[2604, 10900, cfg, seq, layer, 0xC5]`` so all heads of a layer share it;
* key channel scale ``sigma_c`` = 1 except ``ceil(0.1 d)`` random channels at 8
  (when ``outlier_channels`` is on); values are never scaled;
* prefix rows: ``k = sigma_c * N(0,1)``, ``v = N(0,1)`` i.i.d.;
* decode rows: a fraction ``cluster_frac`` belongs to near-duplicate clusters,
  either ``n_centres`` equiprobable centres (tiny config) or clusters of size
  ``1 + Geometric(p)`` (>= 2); a member is its centre plus ``noise * sigma_c *
  N(0,1)`` (keys) / ``noise * N(0,1)`` (values); members sit at uniformly
  random decode positions; the other decode rows are i.i.d. like prefix rows;
* window queries ``q ~ N(0,1)`` of shape ``[g, W, d]``.

These caches stand in for the reasoning-benchmark traces and long-document
prompt-heavy tasks the paper measured on; the datasets themselves are not used.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional, Tuple

import numpy as np

DTYPE_BF16 = 0
DTYPE_FP32 = 1


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and distribution of one benchmark configuration."""

    name: str
    cfg_id: int
    layers: int
    kv_heads: int
    group: int            # g: query heads per KV head
    head_dim: int         # d
    dtype: int            # DTYPE_BF16 | DTYPE_FP32
    prefix: int           # P
    decode: int           # N_d (or the maximum, when decode_min is set)
    window: int           # W
    budget: int           # B
    reserve: int          # slots held back for the decode region
    outlier_channels: bool = True
    cluster_frac: float = 0.6
    n_centres: int = 0    # >0: fixed number of equiprobable centres
    geometric_p: float = 0.1
    noise: float = 0.05
    n_seqs: int = 1
    decode_min: int = 0   # >0: N_d ~ U{decode_min..decode} per sequence
    carried_rows: int = 0     # >0: the first carried_rows rows are an earlier event's output and carry its masses
    layers_per_pass: int = 0  # >0: the benchmark holds this many layers of every sequence on the device at once

    @property
    def n_units(self) -> int:
        return self.n_seqs * self.layers * self.kv_heads

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _w(name, cfg_id, **kw) -> Workload:
    return Workload(name=name, cfg_id=cfg_id, **kw)


WORKLOADS: Dict[str, Workload] = {
    "tiny": _w("tiny", 1, layers=1, kv_heads=2, group=4, head_dim=64, dtype=DTYPE_FP32,
               prefix=128, decode=896, window=16, budget=128, reserve=64,
               outlier_channels=False, cluster_frac=1.0, n_centres=24),
    "reasoning8k_b384": _w("reasoning8k_b384", 2, layers=28, kv_heads=4, group=7, head_dim=128,
                           dtype=DTYPE_BF16, prefix=256, decode=8192, window=64, budget=384, reserve=192),
    "reasoning8k_b512": _w("reasoning8k_b512", 2, layers=28, kv_heads=4, group=7, head_dim=128,
                           dtype=DTYPE_BF16, prefix=256, decode=8192, window=64, budget=512, reserve=256),
    "reasoning32k_b384": _w("reasoning32k_b384", 3, layers=36, kv_heads=8, group=4, head_dim=128,
                            dtype=DTYPE_BF16, prefix=512, decode=32768, window=128, budget=384, reserve=192),
    "reasoning32k_b512": _w("reasoning32k_b512", 3, layers=36, kv_heads=8, group=4, head_dim=128,
                            dtype=DTYPE_BF16, prefix=512, decode=32768, window=128, budget=512, reserve=256),
    "reasoning32k_b1024": _w("reasoning32k_b1024", 3, layers=36, kv_heads=8, group=4, head_dim=128,
                             dtype=DTYPE_BF16, prefix=512, decode=32768, window=128, budget=1024, reserve=512),
    "prompt_heavy": _w("prompt_heavy", 4, layers=28, kv_heads=4, group=7, head_dim=128, dtype=DTYPE_BF16,
                       prefix=12288, decode=1024, window=64, budget=2048, reserve=512),
    "prompt_heavy_boundary": _w("prompt_heavy_boundary", 4, layers=28, kv_heads=4, group=7, head_dim=128,
                                dtype=DTYPE_BF16, prefix=16384, decode=1024, window=64, budget=1024,
                                reserve=256),
    "batched_serving": _w("batched_serving", 5, layers=36, kv_heads=8, group=4, head_dim=128,
                          dtype=DTYPE_BF16, prefix=512, decode=32768, window=128, budget=512, reserve=256,
                          n_seqs=64, decode_min=4096, layers_per_pass=6),
    # The serving sweep in its steady state: every cache was compacted to B = 512 rows by an earlier event
    # (256 prefix + 256 decode slots, carrying their group masses) and 128 decode steps have appended 128 rows.
    "serving_steady_b512": _w("serving_steady_b512", 6, layers=36, kv_heads=8, group=4, head_dim=128,
                              dtype=DTYPE_BF16, prefix=256, decode=384, window=128, budget=512, reserve=256,
                              n_seqs=64, carried_rows=512),
}


# ---------------------------------------------------------------------------
# dtype helpers (bit manipulation only)
# ---------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_cache_dtype(x: np.ndarray, dtype: int) -> np.ndarray:
    """float32 array -> storage array (uint16 bf16 bits, or float32 unchanged)."""
    if dtype == DTYPE_BF16:
        return f32_to_bf16_bits(x)
    return np.ascontiguousarray(x, dtype=np.float32)


def as_float32(x: np.ndarray, dtype: int) -> np.ndarray:
    """Storage array -> the exact float32 values it holds."""
    if dtype == DTYPE_BF16:
        return bf16_bits_to_f32(x)
    return np.ascontiguousarray(x, dtype=np.float32)


# ---------------------------------------------------------------------------
# unit generation
# ---------------------------------------------------------------------------

def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([2604, 10900, *key])))


def channel_scale(wl: Workload, seq: int, layer: int) -> np.ndarray:
    d = wl.head_dim
    sc = np.ones(d, dtype=np.float32)
    if wl.outlier_channels:
        r = _rng(wl.cfg_id, seq, layer, 0xC5)
        idx = r.choice(d, size=int(math.ceil(0.1 * d)), replace=False)
        sc[idx] = 8.0
    return sc


def decode_len(wl: Workload, seq: int) -> int:
    if wl.decode_min > 0:
        r = _rng(wl.cfg_id, seq, 0xD1)
        return int(r.integers(wl.decode_min, wl.decode + 1))
    return wl.decode


def make_unit(wl: Workload, seq: int, layer: int, head: int,
              decode: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Returns (K[T,d], V[T,d], Q[g,W,d]) in the cache dtype's storage type."""
    d, P = wl.head_dim, wl.prefix
    n_d = decode_len(wl, seq) if decode is None else decode
    T = P + n_d
    rng = _rng(wl.cfg_id, seq, layer, head)
    sc = channel_scale(wl, seq, layer)

    k = rng.standard_normal((T, d), dtype=np.float32)
    v = rng.standard_normal((T, d), dtype=np.float32)
    k *= sc

    n_cl_rows = int(round(wl.cluster_frac * n_d))
    if n_cl_rows > 0:
        if wl.n_centres > 0:
            n_c = wl.n_centres
            member_cluster = rng.integers(0, n_c, size=n_cl_rows)
        else:
            # draw sizes 1+Geometric(p) until they cover the clustered rows
            est = int(n_cl_rows / (1.0 + 1.0 / wl.geometric_p) * 1.5) + 16
            sizes = 1 + rng.geometric(wl.geometric_p, size=est)
            while sizes.sum() < n_cl_rows:
                sizes = np.concatenate([sizes, 1 + rng.geometric(wl.geometric_p, size=est)])
            csum = np.cumsum(sizes)
            n_c = int(np.searchsorted(csum, n_cl_rows, side="left")) + 1
            member_cluster = np.repeat(np.arange(n_c), sizes[:n_c])[:n_cl_rows]
        kc = rng.standard_normal((n_c, d), dtype=np.float32) * sc
        vc = rng.standard_normal((n_c, d), dtype=np.float32)
        pos = P + rng.permutation(n_d)[:n_cl_rows]
        # the i.i.d. draws already at these rows serve as the member noise
        k[pos] = kc[member_cluster] + np.float32(wl.noise) * k[pos]
        v[pos] = vc[member_cluster] + np.float32(wl.noise) * v[pos]

    q = rng.standard_normal((wl.group, wl.window, d), dtype=np.float32)
    return to_cache_dtype(k, wl.dtype), to_cache_dtype(v, wl.dtype), to_cache_dtype(q, wl.dtype)


def make_mass(wl: Workload, seq: int, layer: int, head: int, T: int) -> np.ndarray:
    """Carried masses of one unit: rows [0, carried_rows) hold the mass an earlier event left on them (a quarter
    of the decode slots stand for groups of 2 + Geometric(p) rows), the appended rows hold none."""
    rng = _rng(wl.cfg_id, seq, layer, head, 0xA5)
    n = min(wl.carried_rows, T)
    mass = np.zeros(T, dtype=np.float32)
    base = rng.uniform(0.5, 1.5, size=n) / max(n, 1)
    size = np.ones(n)
    rep = (np.arange(n) >= wl.prefix) & (rng.random(n) < 0.25)
    size[rep] = 2 + rng.geometric(wl.geometric_p, size=int(rep.sum()))
    mass[:n] = (base * size).astype(np.float32)
    return mass


@dataclasses.dataclass
class Batch:
    """A ragged batch of independent units, contiguous rows, host-resident."""

    wl: Workload
    k: np.ndarray            # [sum T, d] storage dtype
    v: np.ndarray            # [sum T, d]
    q: np.ndarray            # [n_units, g, W, d]
    T: np.ndarray            # int32 [n_units]
    P: np.ndarray            # int32 [n_units]
    B: np.ndarray            # int32 [n_units]
    reserve: np.ndarray      # int32 [n_units]
    tok_off: np.ndarray      # int64 [n_units+1]
    unit_ids: List[Tuple[int, int, int]]
    mass_in: Optional[np.ndarray] = None   # float32 [sum T] carried masses, when the workload has them

    @property
    def n_units(self) -> int:
        return len(self.unit_ids)

    def unit(self, u: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        a, b = int(self.tok_off[u]), int(self.tok_off[u + 1])
        return self.k[a:b], self.v[a:b], self.q[u]


def unit_list(wl: Workload, layers: Optional[range] = None, seqs: Optional[range] = None,
              heads: Optional[range] = None) -> List[Tuple[int, int, int]]:
    layers = range(wl.layers) if layers is None else layers
    seqs = range(wl.n_seqs) if seqs is None else seqs
    heads = range(wl.kv_heads) if heads is None else heads
    return [(s, l, h) for s in seqs for l in layers for h in heads]


def make_batch(wl: Workload, units: Optional[List[Tuple[int, int, int]]] = None,
               threads: int = 8, pinned_alloc=None) -> Batch:
    """Generate the listed units (default: all) into one contiguous host batch.

    ``pinned_alloc(shape, np_dtype) -> np.ndarray`` lets a caller place the arrays in
    page-locked memory; the default is ordinary numpy memory.
    """
    units = unit_list(wl) if units is None else units
    n = len(units)
    T = np.array([wl.prefix + decode_len(wl, s) for (s, _, _) in units], dtype=np.int32)
    tok_off = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(T, out=tok_off[1:])
    st = np.uint16 if wl.dtype == DTYPE_BF16 else np.float32
    alloc = pinned_alloc if pinned_alloc is not None else (lambda shape, dt: np.empty(shape, dtype=dt))
    k = alloc((int(tok_off[-1]), wl.head_dim), st)
    v = alloc((int(tok_off[-1]), wl.head_dim), st)
    q = alloc((n, wl.group, wl.window, wl.head_dim), st)
    mass = alloc((int(tok_off[-1]),), np.float32) if wl.carried_rows > 0 else None
    if mass is not None:
        mass[...] = 0.0

    def work(u: int) -> None:
        s, l, h = units[u]
        ku, vu, qu = make_unit(wl, s, l, h)
        a, b = int(tok_off[u]), int(tok_off[u + 1])
        k[a:b] = ku
        v[a:b] = vu
        q[u] = qu
        if mass is not None:
            mass[a:b] = make_mass(wl, s, l, h, b - a)

    if threads > 1 and n > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(n)))
    else:
        for u in range(n):
            work(u)
    return Batch(wl=wl, k=k, v=v, q=q, T=T,
                 P=np.full(n, wl.prefix, dtype=np.int32),
                 B=np.full(n, wl.budget, dtype=np.int32),
                 reserve=np.full(n, wl.reserve, dtype=np.int32),
                 tok_off=tok_off, unit_ids=list(units), mass_in=mass)


def shard_units(units: List[Tuple[int, int, int]], rank: int, world: int) -> List[Tuple[int, int, int]]:
    """Contiguous block partition of independent units over ranks (no exchange step)."""
    n = len(units)
    lo = (n * rank) // world
    hi = (n * (rank + 1)) // world
    return units[lo:hi]
