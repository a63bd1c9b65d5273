"""ctypes binding of libcask.so: the same entry points as ``include/cask.h``.

Argument marshalling only: every step of the compression event runs in the
CUDA kernels of the library.  torch is used for device memory and streams.
Loading fails loudly when the library has not been built; nothing here falls
back to a CPU implementation.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcask.so")

# mirrors of the header's constants
OK = 0
ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_WORKSPACE, ERR_UNSUPPORTED, ERR_CUDA, ERR_PARAM = -1, -2, -3, -4, -5, -6, -7
ERR_TOO_LARGE = -8
NOALLOC_SCRATCH_BYTES, NOALLOC_MAX_UNITS = 4 * 1024 * 1024, 64
ST_NOOP_UNDER_BUDGET, ST_PREFIX_EVICTED, ST_DECODE_CONSOLIDATED = 1, 2, 4
ST_PREFIX_BUDGET_EXHAUSTED, ST_MERGE_INACTIVE, ST_TIMEOUT, ST_BOUNDS = 8, 16, 32, 64
KIND_DROPPED, KIND_PREFIX, KIND_RECENT, KIND_CORE, KIND_SEED, KIND_MERGED = 0, 1, 2, 3, 4, 5
DTYPE_BF16, DTYPE_FP32 = 0, 1

EXPORTS = (
    "cask_create", "cask_destroy", "cask_set_stream", "cask_strerror", "cask_last_cuda_error",
    "cask_launch_count", "cask_last_score_path_tensor", "cask_last_device_flags", "cask_profile_enable", "cask_profile_read",
    "cask_kernel_count", "cask_kernel_name", "cask_workspace_bytes", "cask_plan_host",
    "cask_score", "cask_score_stats", "cask_prefix_evict", "cask_select_core", "cask_consolidate_scratch", "cask_compact",
    "cask_compress_event", "cask_writeback_paged", "cask_host_event_device_bytes", "cask_compress_event_host", "cask_score_noalloc",
    "cask_selftest_wait_timeout", "cask_selftest_exp_rate", "cask_last_score_clock_khz",
)


class CaskBatch(C.Structure):
    _fields_ = [
        ("n_units", C.c_int32), ("head_dim", C.c_int32), ("group", C.c_int32), ("window", C.c_int32),
        ("dtype", C.c_int32), ("page_size", C.c_int32),
        ("k", C.c_void_p), ("v", C.c_void_p),
        ("k_off", C.c_void_p), ("v_off", C.c_void_p), ("row_stride", C.c_int64),
        ("q", C.c_void_p), ("lse_in", C.c_void_p),
        ("T", C.c_void_p), ("P", C.c_void_p), ("B", C.c_void_p), ("reserve", C.c_void_p),
        ("tok_off", C.c_void_p),
        ("block_table", C.c_void_p), ("bt_off", C.c_void_p), ("n_pages", C.c_int64),
        ("mass_in", C.c_void_p), ("chan_w", C.c_void_p),
        ("band_w", C.c_void_p), ("band_layout", C.c_int32),
    ]


class CaskQueryStats(C.Structure):
    _fields_ = [
        ("mu", C.c_void_p), ("pi", C.c_void_p), ("delta_grid", C.c_void_p), ("n_delta", C.c_int32),
        ("omega", C.c_void_p), ("band_layout", C.c_int32), ("delta", C.c_void_p),
    ]


class CaskParams(C.Structure):
    _fields_ = [("gamma", C.c_float), ("tau", C.c_float), ("eps", C.c_float), ("causal", C.c_int32),
                ("score_path", C.c_int32)]


class CaskOutputs(C.Structure):
    _fields_ = [
        ("k_out", C.c_void_p), ("v_out", C.c_void_p), ("Bmax", C.c_int32),
        ("n_out", C.c_void_p), ("slot_src", C.c_void_p), ("slot_kind", C.c_void_p), ("slot_mass", C.c_void_p),
        ("assign", C.c_void_p), ("weight", C.c_void_p), ("kind", C.c_void_p), ("seed_of", C.c_void_p),
        ("plan", C.c_void_p), ("unit_status", C.c_void_p), ("lost_mass", C.c_void_p),
        ("s", C.c_void_p), ("lse", C.c_void_p), ("sim", C.c_void_p),
        ("rho_core", C.c_void_p), ("rho_rep", C.c_void_p), ("dispersion", C.c_void_p),
    ]


_lib = None


def lib():
    """The loaded library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2604_10900_b200.build` "
                "(the compression event has no CPU path)")
        L = C.CDLL(LIB_PATH)
        vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int
        PB, PP, PO = C.POINTER(CaskBatch), C.POINTER(CaskParams), C.POINTER(CaskOutputs)
        L.cask_create.argtypes = [C.POINTER(vp), i32, vp]
        L.cask_destroy.argtypes = [vp]
        L.cask_set_stream.argtypes = [vp, vp]
        L.cask_strerror.argtypes = [i32]
        L.cask_strerror.restype = C.c_char_p
        L.cask_last_cuda_error.argtypes = [vp]
        L.cask_last_cuda_error.restype = C.c_char_p
        L.cask_launch_count.argtypes = [vp]
        L.cask_launch_count.restype = C.c_int64
        L.cask_last_score_path_tensor.argtypes = [vp]
        L.cask_last_device_flags.argtypes = [vp, vp]
        L.cask_profile_enable.argtypes = [vp, i32]
        L.cask_profile_read.argtypes = [vp, vp, vp]
        L.cask_kernel_name.argtypes = [i32]
        L.cask_kernel_name.restype = C.c_char_p
        L.cask_workspace_bytes.argtypes = [PB, PP]
        L.cask_workspace_bytes.restype = sz
        L.cask_plan_host.argtypes = [PB, PP, vp]
        L.cask_score.argtypes = [vp, PB, PP, vp, vp, vp, sz]
        L.cask_score_stats.argtypes = [vp, PB, PP, C.POINTER(CaskQueryStats), vp, vp, sz]
        L.cask_prefix_evict.argtypes = [vp, PB, PP, vp, vp, vp, vp, sz]
        L.cask_select_core.argtypes = [vp, PB, PP, vp, vp, vp, vp, sz]
        L.cask_consolidate_scratch.argtypes = [vp, PB, PP, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz]
        L.cask_compact.argtypes = [vp, PB, PP, vp, vp, vp, vp, PO, vp, sz]
        L.cask_compress_event.argtypes = [vp, PB, PP, PO, vp, sz]
        L.cask_writeback_paged.argtypes = [vp, PB, PP, PO, vp, vp, vp, sz]
        L.cask_host_event_device_bytes.argtypes = [PB, PP, C.c_int32]
        L.cask_host_event_device_bytes.restype = sz
        L.cask_compress_event_host.argtypes = [vp, PB, PP, PO, vp, sz]
        L.cask_score_noalloc.argtypes = [i32, vp, PB, PP, vp, vp]
        L.cask_selftest_wait_timeout.argtypes = [vp, C.c_uint64, vp, sz, vp, vp]
        L.cask_selftest_exp_rate.argtypes = [vp, C.c_int32, vp, sz, vp]
        L.cask_last_score_clock_khz.argtypes = [vp, vp]
        _lib = L
    return _lib


def use_library(path: Optional[str] = None) -> str:
    """Loads another build of the library for every later call (contexts made before keep working only until then:
    make new ones).  ``None`` goes back to libcask.so.  Meant for the self-checking build, libcask_bounds.so."""
    global _lib, LIB_PATH
    LIB_PATH = os.path.join(_HERE, "libcask.so") if path is None else path
    _lib = None
    lib()
    return LIB_PATH


class CaskError(RuntimeError):
    def __init__(self, code: int, ctx=None):
        msg = lib().cask_strerror(code).decode()
        if code == ERR_CUDA and ctx is not None:
            msg += ": " + lib().cask_last_cuda_error(ctx).decode()
        super().__init__(f"cask error {code}: {msg}")
        self.code = code


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor, numpy array, int, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


def params(gamma: float = 0.5, tau: float = 0.9, eps: float = 1e-9, causal: int = 1,
           score_path: int = 0) -> CaskParams:
    return CaskParams(gamma, tau, eps, causal, score_path)


class HostArrays:
    """Keeps the host-side integer arrays of a batch alive next to the struct."""

    def __init__(self, T, P, B, reserve, tok_off, k_off, v_off):
        self.T = np.ascontiguousarray(T, np.int32)
        self.P = np.ascontiguousarray(P, np.int32)
        self.B = np.ascontiguousarray(B, np.int32)
        self.reserve = np.ascontiguousarray(reserve, np.int32)
        self.tok_off = np.ascontiguousarray(tok_off, np.int64)
        self.k_off = np.ascontiguousarray(k_off, np.int64)
        self.v_off = np.ascontiguousarray(v_off, np.int64)


def make_batch(k, v, q, T, P, B, reserve, tok_off, head_dim: int, group: int, window: int, dtype: int,
               k_off=None, v_off=None, row_stride: Optional[int] = None, lse_in=None, page_size: int = 0,
               block_table=None, bt_off=None, n_pages: int = 0, mass_in=None, chan_w=None, band_w=None,
               band_layout: int = 0):
    """Fills a cask_batch.  k, v, q, lse_in: tensors/arrays/addresses (device for the device calls,
    host for cask_compress_event_host).  Paged cache: page_size > 0, k and v the page pools,
    block_table a device int32 tensor, bt_off the host offsets of the units in it.
    Returns (struct, keepalive)."""
    tok_off = np.ascontiguousarray(tok_off, np.int64)
    if k_off is None:
        k_off = tok_off[:-1] * head_dim
    if v_off is None:
        v_off = k_off
    h = HostArrays(T, P, B, reserve, tok_off, k_off, v_off)
    b = CaskBatch()
    b.n_units = len(h.T)
    b.head_dim, b.group, b.window, b.dtype, b.page_size = head_dim, group, window, dtype, page_size
    b.k, b.v, b.q, b.lse_in = _ptr(k), _ptr(v), _ptr(q), _ptr(lse_in)
    b.k_off, b.v_off = h.k_off.ctypes.data, h.v_off.ctypes.data
    b.row_stride = head_dim if row_stride is None else row_stride
    b.T, b.P, b.B, b.reserve = h.T.ctypes.data, h.P.ctypes.data, h.B.ctypes.data, h.reserve.ctypes.data
    b.tok_off = h.tok_off.ctypes.data
    bt_host = None if bt_off is None else np.ascontiguousarray(bt_off, np.int64)
    b.block_table = _ptr(block_table)
    b.bt_off = None if bt_host is None else bt_host.ctypes.data
    b.n_pages = n_pages
    b.mass_in = _ptr(mass_in)
    b.chan_w = _ptr(chan_w)
    b.band_w = _ptr(band_w)
    b.band_layout = int(band_layout)
    return b, (h, k, v, q, lse_in, block_table, bt_host, mass_in, chan_w, band_w)


def make_outputs(d: Dict, Bmax: int) -> CaskOutputs:
    o = CaskOutputs()
    o.Bmax = Bmax
    for name, _ in CaskOutputs._fields_:
        if name == "Bmax":
            continue
        setattr(o, name, _ptr(d.get(name)))
    return o


class Context:
    """cask_create / cask_destroy around a CUDA device and stream."""

    def __init__(self, device: int = 0, stream: Optional[int] = None):
        self.handle = C.c_void_p()
        self._lib = lib()          # a context belongs to the build of the library that made it
        rc = self._lib.cask_create(C.byref(self.handle), device, stream)
        if rc != OK:
            raise CaskError(rc)

    def close(self):
        if self.handle:
            self._lib.cask_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stream(self, stream: Optional[int]):
        self._lib.cask_set_stream(self.handle, stream)

    @property
    def launches(self) -> int:
        return int(self._lib.cask_launch_count(self.handle))

    def profile_enable(self, on: bool = True):
        self._lib.cask_profile_enable(self.handle, int(on))

    def profile_read(self) -> Dict[str, Dict]:
        """{kernel name: {"ms": total, "launches": n}} since the last read."""
        n = self._lib.cask_kernel_count()
        ms = np.zeros(n, np.float32)
        cnt = np.zeros(n, np.int64)
        rc = self._lib.cask_profile_read(self.handle, ms.ctypes.data, cnt.ctypes.data)
        if rc != OK:
            raise CaskError(rc, self.handle)
        return {self._lib.cask_kernel_name(i).decode(): dict(ms=float(ms[i]), launches=int(cnt[i]))
                for i in range(n) if cnt[i]}

    @property
    def used_tensor_path(self) -> bool:
        return bool(self._lib.cask_last_score_path_tensor(self.handle))

    def score_clock_mhz(self):
        """(normaliser pass, score pass) SM clock in MHz of the last tensor-core scoring call (0: did not run)."""
        khz = (C.c_int32 * 2)(0, 0)
        rc = self._lib.cask_last_score_clock_khz(self.handle, C.addressof(khz))
        if rc != OK:
            raise CaskError(rc, self.handle)
        return khz[0] / 1e3, khz[1] / 1e3

    def device_flags(self) -> int:
        """CASK_ST_* bits raised on the device by the last call (waits for the stream)."""
        f = C.c_int32(0)
        rc = self._lib.cask_last_device_flags(self.handle, C.byref(f))
        if rc != OK:
            raise CaskError(rc, self.handle)
        return int(f.value)


def _check(rc: int, ctx: Optional[Context] = None):
    if rc != OK:
        raise CaskError(rc, ctx.handle if ctx is not None else None)


def cask_workspace_bytes(batch: CaskBatch, prm: CaskParams) -> int:
    return int(lib().cask_workspace_bytes(C.byref(batch), C.byref(prm)))


def cask_plan_host(batch: CaskBatch, prm: CaskParams) -> np.ndarray:
    out = np.zeros((batch.n_units, 8), np.int32)
    _check(lib().cask_plan_host(C.byref(batch), C.byref(prm), out.ctypes.data))
    return out


def cask_score(ctx: Context, batch, prm, s, lse_out, ws, ws_bytes: int, check: bool = True) -> int:
    rc = ctx._lib.cask_score(ctx.handle, C.byref(batch), C.byref(prm), _ptr(s), _ptr(lse_out), _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def make_query_stats(mu, pi, delta_grid, omega, band_layout: int = 0, delta=None):
    """(struct, keep-alive) for cask_score_stats; every array is a device tensor (float32)."""
    q = CaskQueryStats()
    q.mu, q.pi, q.delta_grid, q.omega, q.delta = _ptr(mu), _ptr(pi), _ptr(delta_grid), _ptr(omega), _ptr(delta)
    q.n_delta = int(delta_grid.shape[0])
    q.band_layout = int(band_layout)
    return q, (mu, pi, delta_grid, omega, delta)


def cask_score_stats(ctx: Context, batch, prm, stats: CaskQueryStats, s, ws, ws_bytes: int, check: bool = True) -> int:
    rc = ctx._lib.cask_score_stats(ctx.handle, C.byref(batch), C.byref(prm), C.byref(stats), _ptr(s), _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_prefix_evict(ctx, batch, prm, s, kind, plan, ws, ws_bytes: int, check: bool = True) -> int:
    rc = ctx._lib.cask_prefix_evict(ctx.handle, C.byref(batch), C.byref(prm), _ptr(s), _ptr(kind), _ptr(plan),
                                 _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_select_core(ctx, batch, prm, s, plan, kind, ws, ws_bytes: int, check: bool = True) -> int:
    rc = ctx._lib.cask_select_core(ctx.handle, C.byref(batch), C.byref(prm), _ptr(s), _ptr(plan), _ptr(kind),
                                _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_consolidate_scratch(ctx, batch, prm, s, plan, kind, seed_of, weight, sim, unit_status, lost_mass,
                             ws, ws_bytes: int, check: bool = True) -> int:
    rc = ctx._lib.cask_consolidate_scratch(ctx.handle, C.byref(batch), C.byref(prm), _ptr(s), _ptr(plan),
                                        _ptr(kind), _ptr(seed_of), _ptr(weight), _ptr(sim), _ptr(unit_status),
                                        _ptr(lost_mass), _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_compact(ctx, batch, prm, s, kind, seed_of, weight, out: CaskOutputs, ws, ws_bytes: int,
                 check: bool = True) -> int:
    rc = ctx._lib.cask_compact(ctx.handle, C.byref(batch), C.byref(prm), _ptr(s), _ptr(kind), _ptr(seed_of),
                            _ptr(weight), C.byref(out), _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_compress_event(ctx, batch, prm, out: CaskOutputs, ws, ws_bytes: int, check: bool = True) -> int:
    rc = ctx._lib.cask_compress_event(ctx.handle, C.byref(batch), C.byref(prm), C.byref(out), _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_writeback_paged(ctx, batch, prm, out: CaskOutputs, k_pool, v_pool, ws, ws_bytes: int, check: bool = True) -> int:
    rc = ctx._lib.cask_writeback_paged(ctx.handle, C.byref(batch), C.byref(prm), C.byref(out), _ptr(k_pool), _ptr(v_pool),
                                    _ptr(ws), ws_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_host_event_device_bytes(batch, prm, Bmax: int) -> int:
    return int(lib().cask_host_event_device_bytes(C.byref(batch), C.byref(prm), Bmax))


def cask_compress_event_host(ctx, host_batch, prm, host_out: CaskOutputs, dev_buf, dev_bytes: int,
                             check: bool = True) -> int:
    rc = ctx._lib.cask_compress_event_host(ctx.handle, C.byref(host_batch), C.byref(prm), C.byref(host_out),
                                        _ptr(dev_buf), dev_bytes)
    if check:
        _check(rc, ctx)
    return rc


def cask_score_noalloc(device: int, stream, batch, prm, s, lse_out=None, check: bool = True) -> int:
    """Scoring for callers that cannot allocate: the scratch is a fixed array inside the library
    (no context, no workspace).  See ``cask_score_noalloc`` in ``include/cask.h`` for the limits."""
    rc = lib().cask_score_noalloc(device, stream, C.byref(batch), C.byref(prm), _ptr(s), _ptr(lse_out))
    if check:
        _check(rc)
    return rc


def cask_selftest_wait_timeout(ctx: Context, limit_ns: int, ws, ws_bytes: int, check: bool = True):
    """Makes one bounded device wait run out (see ``cask_selftest_wait_timeout`` in ``include/cask.h``).
    Returns (return code, device flags, ns the waiting warp spent, ns the following warp spent)."""
    flags = C.c_int32(0)
    waited = (C.c_uint64 * 2)(0, 0)
    rc = ctx._lib.cask_selftest_wait_timeout(ctx.handle, limit_ns, _ptr(ws), ws_bytes, C.addressof(flags), C.addressof(waited))
    if check:
        _check(rc, ctx)
    return rc, int(flags.value), int(waited[0]), int(waited[1])


def cask_selftest_exp_rate(ctx: Context, iters: int, ws, ws_bytes: int) -> float:
    """Exponentials per clock per SM the special-function unit sustains in the scoring epilogue's instruction mix."""
    rate = C.c_double(0.0)
    _check(ctx._lib.cask_selftest_exp_rate(ctx.handle, iters, _ptr(ws), ws_bytes, C.addressof(rate)), ctx)
    return float(rate.value)


# ---- device-memory plumbing (torch): allocation of inputs, outputs and workspace -------------

def torch_storage_dtype(dtype: int):
    import torch
    return torch.bfloat16 if dtype == DTYPE_BF16 else torch.float32


def to_device(host_batch, device="cuda:0"):
    """workloads.Batch (numpy) -> dict of torch tensors on the device (k, v, q)."""
    import torch
    wl = host_batch.wl

    def up(a):
        t = torch.from_numpy(a)
        if wl.dtype == DTYPE_BF16:
            t = t.view(torch.bfloat16)
        return t.to(device)

    return dict(k=up(host_batch.k), v=up(host_batch.v), q=up(host_batch.q))


def alloc_outputs(n_units: int, sum_T: int, Bmax: int, d: int, rows: int, dtype: int, device="cuda:0",
                  optional: bool = True) -> Dict:
    import torch
    st = torch_storage_dtype(dtype)
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
    o = dict(
        k_out=z((n_units, Bmax, d), st), v_out=z((n_units, Bmax, d), st),
        n_out=z((n_units,), torch.int32), slot_src=z((n_units, Bmax), torch.int32),
        slot_kind=z((n_units, Bmax), torch.uint8), slot_mass=z((n_units, Bmax), torch.float32),
        assign=z((sum_T,), torch.int32), weight=z((sum_T,), torch.float32), kind=z((sum_T,), torch.uint8),
        seed_of=z((sum_T,), torch.int32), plan=z((n_units, 8), torch.int32),
        unit_status=z((n_units,), torch.int32), lost_mass=z((n_units,), torch.float32))
    if optional:
        o.update(s=z((sum_T,), torch.float32), lse=z((n_units, rows), torch.float32),
                 sim=z((sum_T,), torch.float32), rho_core=z((n_units,), torch.float32),
                 rho_rep=z((n_units,), torch.float32), dispersion=z((n_units,), torch.float32))
    return o


def alloc_workspace(batch: CaskBatch, prm: CaskParams, device="cuda:0"):
    import torch
    n = cask_workspace_bytes(batch, prm)
    if n == 0:
        n = 256
    return torch.empty(n, dtype=torch.uint8, device=device), n
