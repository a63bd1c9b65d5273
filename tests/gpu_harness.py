"""Helpers for the GPU parity tests: run the library and the oracle on one seeded batch and compare.

Comparison rules
  * integer/byte/index results must match exactly, except rows whose oracle score lies within
    REL_BAND (1e-5 relative) of a selection threshold, or whose best cosine similarity lies within
    SIM_BAND of tau or of the runner-up (the floating-point decision may legitimately flip there);
  * when such a flip changes a unit's kept set, seed set or a row's group, the unit is counted in ``cascaded``:
    its slot numbering and every group the flipped rows touch legitimately differ, but every group with the same
    seed and the same members on both sides is still compared (weights, group mass, merged K/V rows), and so is
    every row kept as a singleton on both sides (byte-identical copy);
  * copied rows are bit-identical to the input rows;
  * merged rows: bf16 |gpu - oracle| <= max(2e-2, 2^-7 |oracle|) (half a bf16 ulp exceeds 2e-2 once
    |x| >= 8), the strict 2e-2 pass rate is reported; fp32: |gpu - oracle| <= 1e-4 |oracle| + 1e-6.
"""
from __future__ import annotations

from typing import Dict

import numpy as np

from oracle import cask_oracle as orc
from paper_2604_10900_b200 import workloads as wl

REL_BAND = 1e-5
SIM_BAND = 1e-5
SCORE_RTOL = 1e-5
WEIGHT_RTOL = 2e-5


def run_oracle(hb: wl.Batch, **kw) -> Dict:
    """kw: tau, gamma, causal, eps, mass_in (per-row carried masses), chan_w (similarity channel weights), band_w / band_layout (per-band distance)."""
    w = hb.wl
    if hb.mass_in is not None:
        kw.setdefault("mass_in", hb.mass_in)
    return orc.event_batch(wl.as_float32(hb.k, w.dtype), wl.as_float32(hb.v, w.dtype),
                           wl.as_float32(hb.q, w.dtype), hb.tok_off, hb.P, hb.B, hb.reserve, **kw)


class GpuRun:
    """Device copies of a host batch plus everything needed to call the library on it."""

    def __init__(self, hb: wl.Batch, device="cuda:0", row_stride=None, lse_in=None, page_size=0, bad_page=None,
                 mass_in=None, chan_w=None, band_w=None, band_layout=0, **prm_kw):
        import torch
        from paper_2604_10900_b200 import binding as cb
        self.cb, self.torch, self.hb = cb, torch, hb
        w = hb.wl
        if mass_in is None:
            mass_in = hb.mass_in
        self.device = device
        self.dev = cb.to_device(hb, device)
        d = w.head_dim
        k_off = None
        if row_stride is not None and row_stride != d:
            # re-lay the rows out with padding between them
            def pad(t):
                p = torch.zeros((t.shape[0], row_stride), dtype=t.dtype, device=device)
                p[:, :d] = t
                return p
            self.dev["k"], self.dev["v"] = pad(self.dev["k"]), pad(self.dev["v"])
            k_off = hb.tok_off[:-1] * row_stride
        paged = {}
        if page_size:
            # Scatter the rows into a pool of shuffled pages (plus a few unused ones); the unused tail of a
            # unit's last page and the spare pages hold a finite junk value that must never show up.
            ps = int(page_size)
            n_lp = [(int(t) + ps - 1) // ps for t in hb.T]
            bt_off = np.concatenate([[0], np.cumsum(n_lp)]).astype(np.int64)
            n_pages = int(bt_off[-1]) + 3
            perm = np.random.default_rng(1234).permutation(n_pages).astype(np.int32)
            table = perm[:int(bt_off[-1])].copy()
            stride = d if row_stride is None else row_stride
            src = np.concatenate([np.arange(int(hb.tok_off[u]), int(hb.tok_off[u]) + int(hb.T[u])) for u in range(hb.n_units)])
            dst = np.concatenate([table[bt_off[u] + np.arange(int(hb.T[u])) // ps].astype(np.int64) * ps
                                  + np.arange(int(hb.T[u])) % ps for u in range(hb.n_units)])
            src_t, dst_t = torch.from_numpy(src).to(device), torch.from_numpy(dst).to(device)
            for name in ("k", "v"):
                pool = torch.full((n_pages * ps, stride), 768.0, dtype=torch.float32, device=device).to(self.dev[name].dtype)
                pool[dst_t, :d] = self.dev[name][src_t, :d]
                self.dev[name] = pool
            if bad_page is not None:
                table[bad_page] = n_pages + 5
            self.block_table = torch.from_numpy(table).to(device)
            paged = dict(page_size=ps, block_table=self.block_table, bt_off=bt_off, n_pages=n_pages)
            k_off = None
        self.mass_in = None if mass_in is None else torch.from_numpy(np.ascontiguousarray(mass_in, np.float32)).to(device)
        self.chan_w = None if chan_w is None else torch.from_numpy(np.ascontiguousarray(chan_w, np.float32)).to(device)
        self.band_w = None if band_w is None else torch.from_numpy(np.ascontiguousarray(band_w, np.float32)).to(device)
        self.lse_in = None if lse_in is None else torch.from_numpy(np.ascontiguousarray(lse_in, np.float32)).to(device)
        self.batch, self._keep = cb.make_batch(
            self.dev["k"], self.dev["v"], self.dev["q"], hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, d, w.group,
            w.window, w.dtype, k_off=k_off, row_stride=row_stride, lse_in=self.lse_in, mass_in=self.mass_in, chan_w=self.chan_w,
            band_w=self.band_w, band_layout=band_layout, **paged)
        self.prm = cb.params(**prm_kw)
        self.ctx = cb.Context(torch.device(device).index or 0, torch.cuda.current_stream(device).cuda_stream)
        self.ws, self.ws_bytes = cb.alloc_workspace(self.batch, self.prm, device)
        self.Bmax = int(hb.B.max())
        self.sum_T = int(hb.tok_off[-1])
        self.out = cb.alloc_outputs(hb.n_units, self.sum_T, self.Bmax, d, w.group * w.window, w.dtype, device)
        self.out_struct = cb.make_outputs(self.out, self.Bmax)

    def event(self) -> Dict:
        self.cb.cask_compress_event(self.ctx, self.batch, self.prm, self.out_struct, self.ws, self.ws_bytes)
        self.torch.cuda.synchronize()
        return self.numpy_outputs()

    def numpy_outputs(self) -> Dict:
        torch = self.torch
        o = {}
        for k, t in self.out.items():
            if t.dtype == torch.bfloat16:
                o[k] = wl.bf16_bits_to_f32(t.view(torch.uint16).cpu().numpy())
            else:
                o[k] = t.cpu().numpy()
        return o

    def dev_f32(self, a):
        return self.torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(self.device)

    def dev_arr(self, a, dt):
        return self.torch.from_numpy(np.ascontiguousarray(a, dt)).to(self.device)


def _kth_desc(vals: np.ndarray, k: int) -> float:
    """k-th greatest value (1-based); +inf if k == 0, -inf if k > len."""
    if k <= 0:
        return np.inf
    if k > len(vals):
        return -np.inf
    return float(np.partition(vals, len(vals) - k)[len(vals) - k])


def exempt_rows(o: Dict, u: int, a: int, T: int, P: int, tau: float) -> np.ndarray:
    """Rows of unit u whose selection may flip under floating-point error (see module docstring)."""
    s = o["s"][a:a + T]
    pl = o["plan"][u]
    pkeep, r, c, m, flags = int(pl[1]), int(pl[3]), int(pl[4]), int(pl[5]), int(pl[6])
    ex = np.zeros(T, bool)

    def band(lo, hi, k):
        n = hi - lo
        if 0 < k < n:
            thr = _kth_desc(s[lo:hi], k)
            nxt = _kth_desc(s[lo:hi], k + 1)
            for t in (thr, nxt):
                ex[lo:hi] |= np.abs(s[lo:hi] - t) <= REL_BAND * abs(t)

    if flags & orc.PREFIX_EVICTED:
        band(0, P, pkeep)
    band(P, T - r, c)
    if m > 0:
        band(P, T - r, c + m)
        sim, sim2 = o["sim"][a:a + T], o["sim2"][a:a + T]
        has = sim > -1.5
        ex |= has & (np.abs(sim - tau) <= SIM_BAND)
        ex |= has & (sim2 > -1.5) & (sim - sim2 <= SIM_BAND)
    return ex


def _merged_rows_check(st: Dict, w, name: str, u: int, mg: np.ndarray, mo: np.ndarray):
    """Merged rows of the GPU (mg) against the oracle's fp64 rows (mo) under the merged-row tolerance; counts them."""
    if not mg.size:
        return
    err = np.abs(mg.astype(np.float64) - mo)
    st["max_merge_abs"] = max(st["max_merge_abs"], float(err.max()))
    st["merged_elems"] += mg.size
    if w.dtype == wl.DTYPE_BF16:
        st["strict_ok"] += int((err <= 2e-2).sum())
        assert (err <= np.maximum(2e-2, 2.0 ** -7 * np.abs(mo))).all(), f"unit {u}: {name} merged rows"
    else:
        st["strict_ok"] += int((err <= 1e-4 * np.abs(mo) + 1e-6).sum())
        assert (err <= 1e-4 * np.abs(mo) + 1e-6).all(), f"unit {u}: {name} merged rows"


def _compare_unaffected(st: Dict, hb: wl.Batch, g: Dict, o: Dict, u: int, kf: np.ndarray, vf: np.ndarray):
    """A unit whose exempt rows flipped: the slot numbering and the groups those rows touch differ, everything else
    must still agree.  Compared here: every group with the same seed and the same member set on both sides
    (weights, group mass, merged rows) and every row that is a singleton slot on both sides (byte copy)."""
    w = hb.wl
    a, T = int(hb.tok_off[u]), int(hb.T[u])
    sl = slice(a, a + T)
    kg, ko = g["kind"][sl], o["kind"][sl]
    sg, so = g["seed_of"][sl], o["seed_of"][sl]
    ag, ao = g["assign"][sl], o["assign"][sl]
    wg, wo = g["weight"][sl], o["weight"][sl]
    n_g, n_o = int(g["n_out"][u]), int(o["n_out"][u])
    cnt_g = np.bincount(ag[ag >= 0], minlength=n_g)
    cnt_o = np.bincount(ao[ao >= 0], minlength=n_o)
    # singleton slots on both sides: bit-identical copies of the input row
    both_single = np.zeros(T, bool)
    kept = (ag >= 0) & (ao >= 0) & np.isin(kg, (1, 2, 3, 4)) & np.isin(ko, (1, 2, 3, 4))
    rows = np.nonzero(kept)[0]
    rows = rows[(cnt_g[ag[rows]] == 1) & (cnt_o[ao[rows]] == 1)]
    both_single[rows] = True
    for name, inp in (("k_out", kf), ("v_out", vf)):
        assert np.array_equal(g[name][u][ag[rows]], inp[a + rows]), f"unit {u}: {name} copies not bit-identical"
    # groups: same seed row, same members
    seeds = np.nonzero((kg == 4) & (ko == 4))[0]
    order_g, order_o = np.argsort(sg, kind="stable"), np.argsort(so, kind="stable")
    lo_g, hi_g = np.searchsorted(sg[order_g], seeds, "left"), np.searchsorted(sg[order_g], seeds, "right")
    lo_o, hi_o = np.searchsorted(so[order_o], seeds, "left"), np.searchsorted(so[order_o], seeds, "right")
    same = 0
    for j, sd in enumerate(seeds):
        mg_, mo_ = order_g[lo_g[j]:hi_g[j]], order_o[lo_o[j]:hi_o[j]]
        if len(mg_) != len(mo_) or not np.array_equal(mg_, mo_):
            continue
        same += 1
        assert np.allclose(wg[mg_], wo[mo_], rtol=WEIGHT_RTOL, atol=1e-9), f"unit {u}: weights of group {sd}"
        tg, to = int(ag[sd]), int(ao[sd])
        assert (ag[mg_] == tg).all() and (ao[mo_] == to).all()
        assert np.isclose(g["slot_mass"][u][tg], o["slot_mass"][u][to], rtol=WEIGHT_RTOL, atol=1e-12)
        if len(mg_) > 1:
            for name in ("k_out", "v_out"):
                _merged_rows_check(st, w, name, u, g[name][u][tg], o[name][u][to])
    st["groups_compared_in_cascaded"] = st.get("groups_compared_in_cascaded", 0) + same
    st["groups_in_cascaded"] = st.get("groups_in_cascaded", 0) + len(seeds)


def compare_event(hb: wl.Batch, g: Dict, o: Dict, tau: float = 0.9, eps: float = 1e-9,
                  check_scores: bool = True, geom: Dict = None) -> Dict:
    """Asserts parity of a GPU event `g` with the oracle event `o`; returns statistics.  `geom`: what the event was
    run with beyond the defaults (mass_in, chan_w, band_w, band_layout, eps), for the dispersion diagnostic."""
    w = hb.wl
    disp_kw = dict(geom or {})
    if hb.mass_in is not None:
        disp_kw.setdefault("mass_in", hb.mass_in)
    d = w.head_dim
    kf, vf = wl.as_float32(hb.k, w.dtype), wl.as_float32(hb.v, w.dtype)
    st = dict(units=hb.n_units, exempt_rows=0, flipped_rows=0, cascaded=0, merged_elems=0, strict_ok=0,
              max_score_rel=0.0, max_merge_abs=0.0, rows=0)
    assert np.array_equal(g["plan"], o["plan"]), "plan differs"
    assert np.array_equal(g["n_out"], o["n_out"]), "n_out differs"
    for u in range(hb.n_units):
        a, T, P = int(hb.tok_off[u]), int(hb.T[u]), int(hb.P[u])
        sl = slice(a, a + T)
        st["rows"] += T
        so, sg = o["s"][sl], g["s"][sl]
        if check_scores:
            rel = np.abs(sg - so) / np.maximum(so, 1e-30)
            big = so > 1e-12
            if big.any():
                st["max_score_rel"] = max(st["max_score_rel"], float(rel[big].max()))
            assert (rel[big] <= SCORE_RTOL).all(), f"unit {u}: score rel err {rel[big].max():.3e}"
            assert np.abs(sg[~big] - so[~big]).max(initial=0.0) <= 1e-12
        ex = exempt_rows(o, u, a, T, P, tau)
        st["exempt_rows"] += int(ex.sum())
        kg, ko = g["kind"][sl], o["kind"][sl]
        diff = kg != ko
        n_out = int(o["n_out"][u])
        if diff.any():
            st["flipped_rows"] += int(diff.sum())
            seeds_same = np.array_equal(kg == 4, ko == 4)
            core_same = np.array_equal(np.isin(kg, (1, 2, 3)), np.isin(ko, (1, 2, 3)))
            if seeds_same and core_same:
                # only join/drop decisions differ: each must be exempt
                assert ex[diff].all(), f"unit {u}: non-exempt join/drop flips at rows {np.nonzero(diff & ~ex)[0][:8]}"
            else:
                sel_diff = (np.isin(kg, (1, 2, 3, 4)) != np.isin(ko, (1, 2, 3, 4))) | ((kg == 4) != (ko == 4)) | \
                           (np.isin(kg, (1, 2, 3)) != np.isin(ko, (1, 2, 3)))
                assert ex[sel_diff].all(), \
                    f"unit {u}: non-exempt selection flips at rows {np.nonzero(sel_diff & ~ex)[0][:8]}"
            st["cascaded"] += 1
            assert int(g["n_out"][u]) == n_out
            _compare_unaffected(st, hb, g, o, u, kf, vf)
            continue
        # identical kinds: everything downstream must agree
        assert int(g["unit_status"][u]) == int(o["status"][u]), (u, g["unit_status"][u], o["status"][u])
        assert np.array_equal(g["slot_src"][u][:n_out], o["slot_src"][u][:n_out])
        assert np.array_equal(g["slot_kind"][u][:n_out], o["slot_kind"][u][:n_out])
        assert (g["slot_src"][u][n_out:] == -1).all() and (g["slot_kind"][u][n_out:] == 0).all()
        so_, sg_ = o["seed_of"][sl], g["seed_of"][sl]
        sd = so_ != sg_
        if sd.any():
            assert ex[sd].all(), f"unit {u}: non-exempt seed_of flips"
            st["cascaded"] += 1
            _compare_unaffected(st, hb, g, o, u, kf, vf)
            continue
        assert np.array_equal(g["assign"][sl], o["assign"][sl])
        wo, wg = o["weight"][sl], g["weight"][sl]
        assert np.allclose(wg, wo, rtol=WEIGHT_RTOL, atol=1e-9), f"unit {u}: weights"
        assert np.allclose(g["slot_mass"][u][:n_out], o["slot_mass"][u][:n_out], rtol=WEIGHT_RTOL, atol=1e-12)
        assert np.isclose(g["lost_mass"][u], o["lost_mass"][u], rtol=1e-4, atol=1e-9)
        if "rho_core" in g and "rho_core" in o:      # Sec. 2.6 diagnostics
            assert np.isclose(g["rho_core"][u], o["rho_core"][u], rtol=2e-5, atol=1e-7), (u, g["rho_core"][u], o["rho_core"][u])
            assert np.isclose(g["rho_rep"][u], o["rho_rep"][u], rtol=2e-5, atol=1e-7), (u, g["rho_rep"][u], o["rho_rep"][u])
        if "dispersion" in g:                        # Sec. 2.6: within-group dispersion against the stored representatives
            krep = o["k_out"][u][:n_out]
            krep = orc.round_bf16(krep) if w.dtype == wl.DTYPE_BF16 else krep.astype(np.float32)
            want = orc.dispersion(kf[sl], o["s"][sl], o["kind"][sl], o["assign"][sl], krep, eps=disp_kw.get("eps", 1e-9),
                                  mass_in=None if disp_kw.get("mass_in") is None else np.asarray(disp_kw["mass_in"])[sl],
                                  chan_w=disp_kw.get("chan_w"), band_w=disp_kw.get("band_w"),
                                  band_layout=disp_kw.get("band_layout", 0))
            # a representative may differ from the oracle's by one unit in the last place of the cache dtype
            assert np.isclose(g["dispersion"][u], want, rtol=2e-3, atol=1e-9), (u, g["dispersion"][u], want)
            st["dispersion_checked"] = st.get("dispersion_checked", 0) + 1
        # per-slot weight sums (Sec. 2.4: a convex combination)
        sums = np.bincount(g["assign"][sl][g["assign"][sl] >= 0], weights=wg[g["assign"][sl] >= 0], minlength=n_out)
        assert np.allclose(sums, 1.0, atol=1e-5)
        src = o["slot_src"][u][:n_out]
        counts = np.bincount(o["assign"][sl][o["assign"][sl] >= 0], minlength=n_out)
        single = counts == 1
        for name, inp in (("k_out", kf), ("v_out", vf)):
            go, oo = g[name][u][:n_out], o[name][u][:n_out]
            assert np.array_equal(go[single], inp[a + src[single]]), f"unit {u}: {name} copies not bit-identical"
            _merged_rows_check(st, w, name, u, go[~single], oo[~single])
    return st
