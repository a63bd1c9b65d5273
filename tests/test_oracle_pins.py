"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle's own code.

Each test names the passage it leans on.  None of them needs a GPU.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest

from oracle import cask_oracle as orc
from paper_2604_10900_b200 import workloads as wl

import bruteforce_event as bf

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand_unit(rng, T, d, g, W):
    K = rng.standard_normal((T, d)).astype(np.float32)
    V = rng.standard_normal((T, d)).astype(np.float32)
    Q = rng.standard_normal((g, W, d)).astype(np.float32)
    return K, V, Q


# ---- score -----------------------------------------------------------------

def test_score_is_a_distribution():
    """Mean of softmax rows: s_i >= 0 and sum_i s_i = 1 (softmax, by construction)."""
    rng = np.random.default_rng(1)
    for T, d, g, W in [(40, 8, 2, 5), (257, 64, 4, 16), (33, 16, 1, 33)]:
        K, _, Q = _rand_unit(rng, T, d, g, W)
        for causal in (0, 1):
            s, _ = orc.score(K, Q, causal=causal)
            assert (s >= 0).all()
            assert abs(s.sum() - 1.0) < 1e-12


def test_score_reduces_to_library_softmax():
    """W = 1, g = 1, non-causal: s = softmax(q K^T / sqrt(d)), checked against torch's CPU softmax."""
    import torch
    rng = np.random.default_rng(2)
    K, _, Q = _rand_unit(rng, 300, 32, 1, 1)
    s, lse = orc.score(K, Q, causal=0)
    x = torch.from_numpy(K.astype(np.float64)) @ torch.from_numpy(Q[0, 0].astype(np.float64)) / math.sqrt(32)
    ref = torch.softmax(x, dim=0).numpy()
    assert np.allclose(s, ref, rtol=1e-12, atol=1e-15)
    assert abs(lse[0, 0] - torch.logsumexp(x, 0).item()) < 1e-12


def test_score_multi_row_against_library_softmax_with_mask():
    """g, W > 1 causal: the same thing written with a masked library softmax (mask: key i <= T-W+j)."""
    import torch
    rng = np.random.default_rng(3)
    T, d, g, W = 90, 16, 3, 7
    K, _, Q = _rand_unit(rng, T, d, g, W)
    s, _ = orc.score(K, Q, causal=1)
    x = torch.einsum("hjc,ic->hji", torch.from_numpy(Q).double(), torch.from_numpy(K).double()) / math.sqrt(d)
    i = torch.arange(T)[None, None, :]
    j = torch.arange(W)[None, :, None]
    x = x.masked_fill(i > T - W + j, float("-inf"))
    ref = torch.softmax(x, dim=-1).mean(dim=(0, 1)).numpy()
    assert np.allclose(s, ref, rtol=1e-12, atol=1e-15)


def test_score_identical_keys_closed_form_golden():
    """All keys equal: every visible key gets 1/(number visible); hand-worked fixture."""
    g_ = json.load(open(os.path.join(GOLD, "identical_keys_score.json")))
    T, W, g = g_["T"], g_["W"], g_["g"]
    K = np.tile(np.array([[0.5, -1.25, 2.0]], np.float32), (T, 1))
    Q = np.random.default_rng(4).standard_normal((g, W, 3)).astype(np.float32)
    s, _ = orc.score(K, Q, causal=1)
    ref = np.array(g_["s_num"], np.float64) / g_["s_den"]
    assert np.allclose(s, ref, rtol=1e-13)


def test_score_identical_keys_closed_form_general():
    T, W, g, d = 57, 9, 2, 4
    K = np.tile(np.array([[1.0, 2.0, -3.0, 0.25]], np.float32), (T, 1))
    Q = np.random.default_rng(5).standard_normal((g, W, d)).astype(np.float32)
    s, _ = orc.score(K, Q, causal=1)
    ref = np.array([sum(1.0 / (T - W + j + 1) for j in range(W) if i <= T - W + j) / W for i in range(T)])
    assert np.allclose(s, ref, rtol=1e-12)


def test_score_supplied_lse_matches_computed():
    rng = np.random.default_rng(6)
    K, _, Q = _rand_unit(rng, 120, 16, 2, 8)
    s0, lse = orc.score(K, Q, causal=1)
    s1, _ = orc.score(K, Q, causal=1, lse_in=lse)
    assert np.allclose(s0, s1, rtol=1e-13)


# ---- budget split ----------------------------------------------------------

def test_budget_split_golden_table():
    """Hand-worked rows for every benchmark shape and both sides of the exhausted boundary (Sec. 2.2, 2.3, 5.2)."""
    tab = json.load(open(os.path.join(GOLD, "budget_split_table.json")))
    for T, P, B, res, W, Bp, Pk, Bd, r, c, m, exh, nout in tab["rows"]:
        pl = orc.plan(T, P, B, res, W, 0.5)
        assert list(pl[:6]) == [Bp, Pk, Bd, r, c, m], (T, P, B, res)
        assert bool(pl[6] & orc.PREFIX_BUDGET_EXHAUSTED) == bool(exh)
        assert pl[7] == nout


def test_budget_respected_exactly_everywhere():
    """n_out = min(P,B_p) + min(N_d, B - min(P,B_p)); equals B when T > B and N_d >= B_d; identity when T <= B."""
    for T in range(1, 15):
        for P in range(0, T + 1):
            for B in range(1, 16):
                for res in range(0, B + 1):
                    for W in (1, 2, 3, 5):
                        if W > T:
                            continue
                        pl = orc.plan(T, P, B, res, W, 0.5)
                        Nd = T - P
                        if T <= B:
                            assert pl[6] & orc.NOOP_UNDER_BUDGET and pl[7] == T
                            continue
                        Pk = min(P, B - res)
                        want = Pk + min(Nd, B - Pk)
                        assert pl[7] == want <= B
                        if Nd >= B - Pk:
                            assert pl[7] == B
                        # slots add up: kept prefix + recent + core + reps = n_out
                        assert pl[1] + pl[3] + pl[4] + pl[5] == pl[7]
                        if pl[6] & orc.DECODE_CONSOLIDATED:
                            assert pl[5] >= 1 and pl[2] >= pl[3] + 2
                        if pl[6] & orc.PREFIX_BUDGET_EXHAUSTED:
                            assert pl[5] == 0 and pl[2] < min(W, Nd) + 2 and Nd > pl[2]
                        assert bool(pl[6] & orc.PREFIX_EVICTED) == (P > B - res)


# ---- selections ------------------------------------------------------------

def test_prefix_eviction_is_brute_force_top_k():
    """Stage 1 (Sec. 2.2): evicted rows are exactly the P - B_p smallest under (score desc, row asc); untouched if P <= B_p."""
    rng = np.random.default_rng(7)
    for P, Bp in [(50, 20), (50, 50), (50, 70), (7, 0)]:
        s = rng.random(P + 30)
        s[3] = s[11] = s[12]          # exact ties resolve by row index
        pl = np.array([Bp, min(P, Bp), 0, 0, 0, 0, 0, 0], np.int32)
        kind = np.zeros(P + 30, np.uint8)
        orc.prefix_evict(s, P, pl, kind)
        order = sorted(range(P), key=lambda i: (-s[i], i))
        want = set(order[:min(P, Bp)])
        assert set(np.nonzero(kind[:P] == 1)[0].tolist()) == want
        assert (kind[P:] == 0).all()


def test_tau_above_one_is_plain_top_k_eviction():
    """tau > 1: nothing can join, so the decode keep-set is recent + top-(c+m) of the rest (textbook top-k)."""
    rng = np.random.default_rng(8)
    T, P, B, res, d, g, W = 200, 40, 64, 32, 16, 2, 8
    K, V, Q = _rand_unit(rng, T, d, g, W)
    o = orc.event(K, V, Q, P, B, res, tau=1.5)
    pl = o["plan"]
    r, c, m = pl[3], pl[4], pl[5]
    s = o["s"]
    rest = sorted(range(P, T - r), key=lambda i: (-s[i], i))[:c + m]
    kept_decode = set(np.nonzero(o["kind"][P:] >= 2)[0] + P)
    assert kept_decode == set(rest) | set(range(T - r, T))
    assert not (o["kind"] == 5).any()
    assert o["status"] & orc.MERGE_INACTIVE
    assert o["n_out"] == B


# ---- core / merge invariants -------------------------------------------------

def _event_tiny(head=0, **kw):
    w = wl.WORKLOADS["tiny"]
    k, v, q = wl.make_unit(w, 0, 0, head)
    return (k, v, q, w), orc.event(k, v, q, w.prefix, w.budget, w.reserve, **kw)


def test_core_is_never_merged_and_copied_bit_identically():
    """C subset R (Sec. 2.3); the core is not a merge target (Sec. 2.1)."""
    (k, v, q, w), o = _event_tiny()
    for t in range(o["n_out"]):
        src, kd = o["slot_src"][t], o["slot_kind"][t]
        members = np.nonzero(o["assign"] == t)[0]
        if kd in (1, 2, 3):
            assert members.tolist() == [src]
            assert o["weight"][src] == 1.0
            assert np.array_equal(o["k_out"][t], k[src].astype(np.float64))
            assert np.array_equal(o["v_out"][t], v[src].astype(np.float64))
    # all recent rows and exactly c core rows present
    pl = o["plan"]
    assert (o["kind"][-pl[3]:] == 2).all()
    assert np.count_nonzero(o["kind"] == 3) == pl[4]
    assert np.count_nonzero(o["kind"] == 4) == pl[5]


def test_merge_weights_and_mass():
    """Sec. 2.4: weights of a group sum to 1, slot mass is the sum of a_i; tau = -1 loses no mass."""
    (k, v, q, w), o = _event_tiny(tau=-1.0)
    eps = 1e-9
    a = o["s"] + eps
    for t in range(o["n_out"]):
        members = np.nonzero(o["assign"] == t)[0]
        assert abs(o["weight"][members].sum() - 1.0) < 1e-12
        assert abs(o["slot_mass"][t] - a[members].sum()) < 1e-15
    scratch = (o["kind"] == 4) | (o["kind"] == 5) | ((o["kind"] == 0) & (np.arange(len(a)) >= w.prefix))
    reps = o["slot_kind"] == 4
    assert abs(o["slot_mass"][reps].sum() - a[scratch].sum()) < 1e-12
    assert o["lost_mass"] == 0.0
    assert not (o["kind"][w.prefix:] == 0).any()


def test_lost_mass_is_dropped_scratch_mass():
    (k, v, q, w), o = _event_tiny()
    a = o["s"] + 1e-9
    dropped = (o["kind"] == 0) & (np.arange(len(a)) >= w.prefix)
    assert abs(o["lost_mass"] - a[dropped].sum()) < 1e-12


def test_merge_rule_worked_example_golden():
    """Sec. 2.4 equations on numbers worked by hand."""
    g_ = json.load(open(os.path.join(GOLD, "merge_rule_worked.json")))
    K = np.array(g_["k"], np.float32)
    V = np.array(g_["v"], np.float32)
    kind = np.array([4, 5], np.uint8)
    seed_of = np.array([0, 0], np.int32)
    o = orc.compact(K, V, kind, seed_of, np.array(g_["w"]), np.array(g_["a"]), eps=0.0)
    assert o["n_out"] == 1
    assert np.allclose(o["k_out"][0], g_["k_tilde"], rtol=1e-15)
    assert np.allclose(o["v_out"][0], g_["v_tilde"], rtol=1e-15)
    assert o["slot_mass"][0] == g_["m_G"]
    # and the weights consolidate() derives from scores are a_i / m_G
    K2 = np.array([[1, 0], [1, 0], [0, 1]], np.float32)         # rows 0,1 identical; row 2 is the recent row
    s = np.array([1.0, 3.0, 0.5])
    pl = np.array([0, 0, 2, 1, 0, 1, orc.DECODE_CONSOLIDATED, 2], np.int32)
    kind2 = np.zeros(3, np.uint8)
    orc.select_core(s, 3, 0, pl, kind2)
    c = orc.consolidate(K2, s, 0, pl, kind2, tau=0.9, eps=0.0)
    assert kind2.tolist() == [5, 4, 2]
    assert c["seed_of"].tolist() == [1, 1, -1]
    assert np.allclose(c["weight"][:2], [0.25, 0.75], rtol=1e-15)


def test_representative_is_the_exact_linear_surrogate():
    """Exact form of the diagnostic of Sec. 2.6: sum_i w_i <q,k_i> = <q,k~>; each coordinate inside the members' range."""
    (k, v, q, w), o = _event_tiny()
    rng = np.random.default_rng(9)
    probe = rng.standard_normal(w.head_dim)
    checked = 0
    for t in np.nonzero(o["slot_kind"] == 4)[0]:
        mem = np.nonzero(o["assign"] == t)[0]
        if len(mem) < 2:
            continue
        checked += 1
        lhs = (o["weight"][mem] * (k[mem].astype(np.float64) @ probe)).sum()
        assert abs(lhs - o["k_out"][t] @ probe) < 1e-10
        for src, out in ((k, o["k_out"]), (v, o["v_out"])):
            lo, hi = src[mem].min(0) - 1e-12, src[mem].max(0) + 1e-12
            assert ((out[t] >= lo) & (out[t] <= hi)).all()
    assert checked > 0


def test_exact_duplicates_merge_to_their_centre():
    """sigma = 0: members of a group are identical, so any convex combination equals the centre (to rounding of the weights); equal scores resolve by row."""
    w = wl.WORKLOADS["tiny"].with_(noise=0.0)
    k, v, q = wl.make_unit(w, 0, 0, 0)
    o = orc.event(k, v, q, w.prefix, w.budget, w.reserve)
    n_groups = 0
    for t in np.nonzero(o["slot_kind"] == 4)[0]:
        mem = np.nonzero(o["assign"] == t)[0]
        src = o["slot_src"][t]
        assert (k[mem] == k[src]).all()
        assert np.allclose(o["k_out"][t], k[src].astype(np.float64), rtol=1e-14, atol=0)
        assert np.allclose(o["v_out"][t], v[src].astype(np.float64), rtol=1e-14, atol=0)
        n_groups += len(mem) > 1
    assert n_groups > 0
    # duplicates below the window have identical scores: the earlier row must win the seed slot
    s = o["s"]
    for t in np.nonzero(o["slot_kind"] == 4)[0]:
        mem = np.nonzero(o["assign"] == t)[0]
        src = o["slot_src"][t]
        tied = [i for i in mem if s[i] == s[src]]
        assert src == min(tied)


def test_planted_clusters_are_recovered_with_full_purity():
    """Tiny config: 24 planted centres, noise 0.05: in-cluster cosine ~0.9975 vs cross-cluster far below tau."""
    w = wl.WORKLOADS["tiny"]
    for head in (0, 1):
        k, v, q = wl.make_unit(w, 0, 0, head)
        o = orc.event(k, v, q, w.prefix, w.budget, w.reserve)
        kn = k / np.linalg.norm(k, axis=1, keepdims=True)
        joiners = np.nonzero(o["kind"] == 5)[0]
        assert len(joiners) > 0
        for j in joiners:
            assert kn[j] @ kn[o["seed_of"][j]] > 0.99          # same planted cluster
        # a dropped scratch row has no seed in its own cluster
        seeds = np.nonzero(o["kind"] == 4)[0]
        dropped = np.nonzero((o["kind"] == 0) & (np.arange(len(k)) >= w.prefix))[0]
        assert (kn[dropped] @ kn[seeds].T).max() < 0.9


# ---- whole event vs the separately written brute force -----------------------

def _cmp_with_bruteforce(K, V, Q, P, B, res, tau, mass_in=None, chan_w=None, band_w=None, band_layout=0):
    o = orc.event(K, V, Q, P, B, res, tau=tau, mass_in=mass_in, chan_w=chan_w, band_w=band_w, band_layout=band_layout)
    b = bf.event(K.tolist(), V.tolist(), Q.tolist(), P, B, res, tau=tau,
                 mass_in=None if mass_in is None else list(mass_in),
                 chan_w=None if chan_w is None else [float(x) for x in chan_w],
                 band_w=None if band_w is None else [float(x) for x in band_w], band_layout=band_layout)
    assert abs(o["rho_core"] - b["rho_core"]) < 1e-12 and abs(o["rho_rep"] - b["rho_rep"]) < 1e-12
    assert np.allclose(o["s"], b["s"], rtol=1e-12, atol=1e-300)
    assert o["kind"].tolist() == b["kind"]
    assert o["slot_src"].tolist() == b["slots"]
    assert o["assign"].tolist() == b["assign"]
    assert o["n_out"] == b["n_out"]
    assert o["status"] == b["flags"], (o["status"], b["flags"], P, B, res)
    assert np.allclose(o["weight"], b["weight"], rtol=1e-12, atol=0)
    assert np.allclose(o["slot_mass"], b["mass"], rtol=1e-12)
    assert abs(o["lost_mass"] - b["lost"]) < 1e-12
    if o["n_out"]:
        assert np.allclose(o["k_out"], np.array(b["k_out"]), rtol=1e-12, atol=1e-14)
        assert np.allclose(o["v_out"], np.array(b["v_out"]), rtol=1e-12, atol=1e-14)


def test_whole_event_against_bruteforce_all_small_shapes():
    """Every (T, P, B, reserve, W) with T <= 12 on clustered rows, including both sides of B_d = r + 2."""
    rng = np.random.default_rng(10)
    n = 0
    for T in (5, 9, 12):
        centres = rng.standard_normal((3, 4))
        K = (centres[rng.integers(0, 3, T)] + 0.05 * rng.standard_normal((T, 4))).astype(np.float32)
        V = rng.standard_normal((T, 4)).astype(np.float32)
        for W in (1, 2, 4):
            Q = rng.standard_normal((2, W, 4)).astype(np.float32)
            for P, B in itertools.product(range(0, T + 1), range(1, T + 2)):
                for res in range(0, B + 1):
                    _cmp_with_bruteforce(K, V, Q, P, B, res, tau=0.9 if (P + B) % 2 else -1.0)
                    n += 1
    assert n > 1500


def test_carried_mass_and_diagnostics_against_bruteforce_and_closed_forms():
    """Rows that already carry group mass (representatives of an earlier event) fold with a_i = s_i + eps +
    carried mass (Sec. 2.4: the fold preserves group mass); rho_core / rho_rep of Sec. 2.6."""
    rng = np.random.default_rng(12)
    T, d, W = 14, 4, 2
    centres = rng.standard_normal((3, d))
    K = (centres[rng.integers(0, 3, T)] + 0.05 * rng.standard_normal((T, d))).astype(np.float32)
    V = rng.standard_normal((T, d)).astype(np.float32)
    Q = rng.standard_normal((2, W, d)).astype(np.float32)
    mass = np.where(rng.random(T) < 0.4, rng.random(T) * 0.5, 0.0)
    for P, B, res in [(0, 6, 6), (3, 8, 5), (4, 9, 6), (0, 5, 5), (2, 7, 4)]:
        for tau in (-1.0, 0.9):
            _cmp_with_bruteforce(K, V, Q, P, B, res, tau, mass_in=mass)
    # zero carried mass is the plain event
    a = orc.event(K, V, Q, 3, 8, 5, tau=-1.0)
    b = orc.event(K, V, Q, 3, 8, 5, tau=-1.0, mass_in=np.zeros(T))
    for k in ("kind", "weight", "slot_mass", "k_out", "rho_rep"):
        assert np.array_equal(a[k], b[k])
    # tau = -1 loses nothing: the slots hold the a_i of every kept or merged row; selections ignore the mass
    c = orc.event(K, V, Q, 0, 6, 6, tau=-1.0, mass_in=mass)
    a0 = orc.event(K, V, Q, 0, 6, 6, tau=-1.0)
    assert np.array_equal(c["kind"], a0["kind"]) and c["lost_mass"] == 0.0
    assert np.isclose(c["slot_mass"].sum(), (c["s"] + 1e-9 + mass).sum(), rtol=1e-12)
    # a heavy member pulls the representative towards itself: weights are a_i / m_G
    grp = np.flatnonzero(c["assign"] == c["assign"][np.flatnonzero(c["kind"] == 5)[0]])
    aw = c["s"][grp] + 1e-9 + mass[grp]
    assert np.allclose(c["weight"][grp], aw / aw.sum(), rtol=1e-12)
    # diagnostics: C is part of R, so rho_core <= rho_rep; with nothing lost and no prefix R carries all the
    # mass, which is at least the mass of the best B rows; a cache under budget keeps everything
    assert c["rho_core"] <= c["rho_rep"] and a0["rho_rep"] >= 1.0 - 1e-12
    u = orc.event(K, V, Q, 2, T + 1, 3)
    assert abs(u["rho_rep"] - (1.0 + T * 1e-9)) < 1e-12 and u["rho_core"] <= 1.0


def test_channel_weighted_similarity():
    """Sec. 2.5: channels (frequency bands) weigh differently in the merge geometry.  Unit weights are the plain
    cosine; 0/1 weights are the cosine of the selected channels (numpy); a common factor changes nothing."""
    rng = np.random.default_rng(13)
    T, d, W, P, B, res = 40, 8, 2, 0, 12, 12
    centres = rng.standard_normal((4, d))
    K = (centres[rng.integers(0, 4, T)] + 0.2 * rng.standard_normal((T, d))).astype(np.float32)
    V = rng.standard_normal((T, d)).astype(np.float32)
    Q = rng.standard_normal((2, W, d)).astype(np.float32)
    plain = orc.event(K, V, Q, P, B, res, tau=0.8)
    ones = orc.event(K, V, Q, P, B, res, tau=0.8, chan_w=np.ones(d))
    assert np.array_equal(plain["kind"], ones["kind"]) and np.array_equal(plain["sim"], ones["sim"])
    w = rng.random(d).astype(np.float32) + 0.1
    a = orc.event(K, V, Q, P, B, res, tau=0.8, chan_w=w)
    b = orc.event(K, V, Q, P, B, res, tau=0.8, chan_w=4.0 * w)
    assert np.array_equal(a["kind"], b["kind"]) and np.allclose(a["sim"], b["sim"], rtol=1e-12)
    assert not np.array_equal(a["sim"], plain["sim"])
    mask = np.array([1, 1, 0, 0, 1, 0, 1, 1], np.float32)
    m = orc.event(K, V, Q, P, B, res, tau=0.8, chan_w=mask)
    seeds = np.flatnonzero(m["kind"] == 4)
    Ks = K[:, mask > 0].astype(np.float64)
    for j in np.flatnonzero(m["sim"] > -1.5):
        cs = Ks[seeds] @ Ks[j] / (np.linalg.norm(Ks[seeds], axis=1) * np.linalg.norm(Ks[j]))
        assert abs(cs.max() - m["sim"][j]) < 1e-12
        if m["kind"][j] == 5:
            assert m["seed_of"][j] == seeds[int(np.argmax(cs))]
    for tau in (-1.0, 0.8):
        _cmp_with_bruteforce(K[:14], V[:14], Q, 2, 7, 4, tau, chan_w=w)


def test_band_distance_geometry():
    """Sec. 2.5, d_kappa = sum_f w_f ||k_if - k_jf||_2 over rotary bands f, read as the similarity
    1 - d_kappa / (D_i + D_j).  Closed forms: equal keys 1, opposite keys 0, orthogonal equal-norm bands
    1 - sqrt(2)/2; one band of weight one is numpy's Euclidean distance on that band's two channels; a common
    factor on the weights or on all keys changes nothing; the two band layouts pair different channels."""
    rng = np.random.default_rng(17)
    d, W = 8, 2
    # two-row closed forms through the whole event: one seed (row 1 scores higher), one candidate (row 0)
    def sim_of(k0, k1, bw, layout):
        K = np.array([k0, k1, k1, k1], np.float32)          # rows 2,3: the recent window (W = 2)
        K[2:] += 100.0                                       # keep them away from the seed choice
        V = np.zeros_like(K)
        Q = np.zeros((1, W, d), np.float32)
        pl = np.array([0, 0, 2, 0, 0, 1, 0, 0], np.int32)    # r = 0, c = 0, m = 1 over rows [0, 2)
        kind = np.zeros(4, np.uint8)
        s = np.array([0.1, 0.9, 0.0, 0.0])
        o = orc.consolidate(K[:2], s[:2], 0, pl, kind[:2], tau=2.0, band_w=bw, band_layout=layout)
        return o["sim"][0]
    k = rng.standard_normal(d).astype(np.float32)
    ones = np.ones(d // 2, np.float32)
    for layout in (0, 1):
        assert abs(sim_of(k, k, ones, layout) - 1.0) < 1e-15
        assert abs(sim_of(k, -k, ones, layout)) < 1e-15
        assert abs(sim_of(k, 4.0 * k, ones, layout) - 0.4) < 1e-12        # 1 - |1-4| / (1+4) in every band
    e = np.zeros(d, np.float32); e[0] = 2.0                                # band 0, first channel
    f0 = np.zeros(d, np.float32); f0[d // 2] = 2.0                         # layout 0: band 0, second channel
    f1 = np.zeros(d, np.float32); f1[1] = 2.0                              # layout 1: band 0, second channel
    assert abs(sim_of(e, f0, ones, 0) - (1.0 - math.sqrt(2.0) / 2.0)) < 1e-12
    assert abs(sim_of(e, f1, ones, 1) - (1.0 - math.sqrt(2.0) / 2.0)) < 1e-12
    assert abs(sim_of(e, f1, ones, 0)) < 1e-12      # layout 0 puts channels 0 and 1 in different bands: d = D_i + D_j
    # whole events: weights, scale invariance, one-band weights against numpy, brute force
    T, P, B, res = 40, 0, 12, 12
    centres = rng.standard_normal((4, d))
    K = (centres[rng.integers(0, 4, T)] + 0.2 * rng.standard_normal((T, d))).astype(np.float32)
    V = rng.standard_normal((T, d)).astype(np.float32)
    Q = rng.standard_normal((2, W, d)).astype(np.float32)
    bw = (rng.random(d // 2) + 0.1).astype(np.float32)
    plain = orc.event(K, V, Q, P, B, res, tau=0.6)
    a = orc.event(K, V, Q, P, B, res, tau=0.6, band_w=bw)
    b = orc.event(K, V, Q, P, B, res, tau=0.6, band_w=4.0 * bw)
    c = orc.event(2.0 * K, V, 0.5 * Q, P, B, res, tau=0.6, band_w=bw)      # same scores (q.k unchanged), keys doubled
    assert np.array_equal(a["kind"], b["kind"]) and np.allclose(a["sim"], b["sim"], rtol=1e-12)
    assert np.array_equal(a["kind"], c["kind"]) and np.allclose(a["sim"], c["sim"], rtol=1e-6, atol=1e-7)
    assert (a["kind"] == 5).any() and not np.array_equal(a["sim"], plain["sim"])
    cand = a["sim"] > -1.5
    assert (a["sim"][cand] >= 0.0).all() and (a["sim"][cand] <= 1.0).all()
    for layout, (c0, c1) in ((0, (1, 1 + d // 2)), (1, (2, 3))):
        one = np.zeros(d // 2, np.float32); one[1] = 1.0
        m = orc.event(K, V, Q, P, B, res, tau=0.6, band_w=one, band_layout=layout)
        seeds = np.flatnonzero(m["kind"] == 4)
        Kb = K[:, [c0, c1]].astype(np.float64)
        for j in np.flatnonzero(m["sim"] > -1.5):
            dist = np.linalg.norm(Kb[seeds] - Kb[j], axis=1)
            sm = 1.0 - dist / (np.linalg.norm(Kb[seeds], axis=1) + np.linalg.norm(Kb[j]))
            assert abs(sm.max() - m["sim"][j]) < 1e-12
            if m["kind"][j] == 5:
                assert m["seed_of"][j] == seeds[int(np.argmax(sm))]
    for layout in (0, 1):
        for tau in (-1.0, 0.6):
            _cmp_with_bruteforce(K[:14], V[:14], Q, 2, 7, 4, tau, band_w=bw, band_layout=layout)


def test_within_group_dispersion():
    """Sec. 2.6, first term of the bound: sum_i a_i ||k_i - k~_G|| over group members.  Hand-worked values for
    the three norms; exact duplicates have none; a two-member group with equal weights and the exact representative
    has a_1 |delta|/2 + a_2 |delta|/2; brute force over a whole event."""
    K = np.array([[1, 0, 0, 0], [3, 4, 0, 0], [0, 0, 0, 0]], np.float32)
    s = np.array([0.2, 0.3, 0.5])
    kind = np.array([4, 5, 0], np.uint8)
    asg = np.array([0, 0, -1], np.int32)
    rep = np.array([[1, 0, 0, 0]], np.float32)
    assert abs(orc.dispersion(K, s, kind, asg, rep, eps=0.0) - 0.3 * math.sqrt(20.0)) < 1e-15
    assert abs(orc.dispersion(K, s, kind, asg, rep, eps=0.0, chan_w=[4, 0.25, 1, 1]) - 0.3 * math.sqrt(16 + 4)) < 1e-15
    assert abs(orc.dispersion(K, s, kind, asg, rep, eps=0.0, band_w=[1, 2], band_layout=1) - 0.3 * math.sqrt(20.0)) < 1e-15
    assert abs(orc.dispersion(K, s, kind, asg, rep, eps=0.0, band_w=[1, 2], band_layout=0) - 0.3 * (2 + 2 * 4)) < 1e-15
    assert abs(orc.dispersion(K, s, kind, asg, rep, eps=0.0, mass_in=[0, 0.7, 0]) - 1.0 * math.sqrt(20.0)) < 1e-15
    # a whole event on exact duplicates: every representative equals its members
    rng = np.random.default_rng(23)
    T, d, W = 30, 8, 2
    centres = rng.standard_normal((3, d)).astype(np.float32)
    K = centres[rng.integers(0, 3, T)]
    V = rng.standard_normal((T, d)).astype(np.float32)
    Q = rng.standard_normal((2, W, d)).astype(np.float32)
    o = orc.event(K, V, Q, 0, 10, 10, tau=0.99)
    assert (o["kind"] == 5).any()
    assert orc.dispersion(K, o["s"], o["kind"], o["assign"], o["k_out"]) < 1e-12
    # noisy clusters: the definition written out with numpy on the oracle's own groups and representatives
    K = (centres[rng.integers(0, 3, T)] + 0.1 * rng.standard_normal((T, d))).astype(np.float32)
    o = orc.event(K, V, Q, 0, 10, 10, tau=0.8)
    mem = np.flatnonzero(np.isin(o["kind"], (4, 5)))
    a = o["s"][mem] + 1e-9
    want = float(np.sum(a * np.linalg.norm(K[mem].astype(np.float64) - o["k_out"][o["assign"][mem]], axis=1)))
    got = orc.dispersion(K, o["s"], o["kind"], o["assign"], o["k_out"].astype(np.float32))
    assert want > 0 and abs(got - want) < 1e-6 * want
    # two members, equal weights: each lies |delta|/2 from the mean
    K2 = np.array([[1, 1, 0, 0], [3, 1, 0, 0]], np.float32)
    d2 = orc.dispersion(K2, np.array([0.5, 0.5]), np.array([4, 5], np.uint8), np.array([0, 0], np.int32),
                        np.array([[2, 1, 0, 0]], np.float32), eps=0.0)
    assert abs(d2 - 1.0) < 1e-15


def test_query_statistics_scorer():
    """App. B: horizon kernel kappa = E_{delta~pi}[e^{i omega delta}] and mean score
    S = Re sum_f mu_f conj(k_f) kappa(omega_f) e^{i omega_f Delta}.  Closed forms: one band, mu = kappa = 1 gives
    k_x cos(omega Delta) + k_y sin(omega Delta); a point-mass horizon at delta_0 shifts Delta by delta_0; a uniform
    symmetric horizon gives the real Dirichlet kernel; the score is linear in mu; numpy complex arithmetic."""
    rng = np.random.default_rng(29)
    T, d, g = 9, 8, 3
    nb = d // 2
    K = rng.standard_normal((T, d)).astype(np.float32)
    om = 1.0 / (50.0 ** (np.arange(nb) / nb))
    # one band active, mu = 1, horizon = point mass at 0
    for layout, (c0, c1) in ((0, (2, 2 + nb)), (1, (4, 5))):
        mu = np.zeros((1, nb, 2), np.float32); mu[0, 2, 0] = 1.0
        s = orc.score_stats(K, mu, [[1.0]], [0.0], om, layout)
        D = T - 1 - np.arange(T)
        want = K[:, c0] * np.cos(om[2] * D) + K[:, c1] * np.sin(om[2] * D)
        assert np.abs(s - want).max() < 1e-12
        # point mass at delta_0 = 3: the same score three steps later
        s3 = orc.score_stats(K, mu, [[1.0]], [3.0], om, layout)
        want3 = K[:, c0] * np.cos(om[2] * (D + 3)) + K[:, c1] * np.sin(om[2] * (D + 3))
        assert np.abs(s3 - want3).max() < 1e-12
        # explicit offsets replace T-1-i
        sd = orc.score_stats(K, mu, [[1.0]], [0.0], om, layout, delta=np.full(T, 2.5))
        assert np.abs(sd - (K[:, c0] * np.cos(om[2] * 2.5) + K[:, c1] * np.sin(om[2] * 2.5))).max() < 1e-12
    # uniform horizon on {-a..a}: kappa is the Dirichlet kernel, real
    a = 4
    grid = np.arange(-a, a + 1, dtype=np.float64)
    mu = np.zeros((1, nb, 2), np.float32); mu[0, 1, 0] = 1.0
    s = orc.score_stats(K, mu, [np.full(2 * a + 1, 1.0 / (2 * a + 1))], grid, om, 0)
    dirichlet = np.sin((2 * a + 1) * om[1] / 2) / ((2 * a + 1) * np.sin(om[1] / 2))
    D = T - 1 - np.arange(T)
    assert np.abs(s - dirichlet * (K[:, 1] * np.cos(om[1] * D) + K[:, 1 + nb] * np.sin(om[1] * D))).max() < 1e-12
    # general case against numpy, linearity in mu, mean over heads
    mu = rng.standard_normal((g, nb, 2)).astype(np.float32)
    grid = np.array([0.0, 1.0, 2.0, 7.0])
    pi = rng.random((g, 4)); pi /= pi.sum(1, keepdims=True)
    for layout in (0, 1):
        c0 = np.arange(nb) if layout == 0 else 2 * np.arange(nb)
        c1 = c0 + (nb if layout == 0 else 1)
        kc = K[:, c0].astype(np.float64) + 1j * K[:, c1]
        muc = mu[..., 0].astype(np.float64) + 1j * mu[..., 1]
        kap = (pi[:, :, None] * np.exp(1j * om[None, None, :] * grid[None, :, None])).sum(1)
        want = np.real(np.einsum("hf,if,hf,if->i", muc, np.conj(kc), kap, np.exp(1j * om[None, :] * D[:, None]))) / g
        got = orc.score_stats(K, mu, pi, grid, om, layout)
        assert np.abs(got - want).max() < 1e-12
        heads = [orc.score_stats(K, mu[h:h + 1], pi[h:h + 1], grid, om, layout) for h in range(g)]
        assert np.abs(got - np.mean(heads, axis=0)).max() < 1e-12
        assert np.abs(orc.score_stats(K, 2.0 * mu, pi, grid, om, layout) - 2.0 * got).max() < 1e-12
    assert (got < 0).any() and (got > 0).any()


def test_whole_event_against_bruteforce_exhausted_boundary():
    rng = np.random.default_rng(11)
    T, P, W, d = 16, 10, 3, 4
    K, V, Q = _rand_unit(rng, T, d, 2, W)
    B = 9
    seen = set()
    for res in range(0, B + 1):
        o = orc.event(K, V, Q, P, B, res)
        seen.add(bool(o["status"] & orc.PREFIX_BUDGET_EXHAUSTED))
        _cmp_with_bruteforce(K, V, Q, P, B, res, tau=0.5)
        Bd = B - min(P, B - res)
        assert bool(o["status"] & orc.PREFIX_BUDGET_EXHAUSTED) == (T - P > Bd and Bd < W + 2)
    assert seen == {True, False}


def test_units_are_independent():
    """A unit's result does not depend on its neighbours in the batch or on their order."""
    w = wl.WORKLOADS["tiny"]
    b = wl.make_batch(w)
    full = orc.event_batch(wl.as_float32(b.k, w.dtype), b.v, b.q, b.tok_off, b.P, b.B, b.reserve)
    for u in range(b.n_units):
        k, v, q = b.unit(u)
        one = orc.event(k, v, q, w.prefix, w.budget, w.reserve)
        a, e = int(b.tok_off[u]), int(b.tok_off[u + 1])
        assert np.array_equal(full["s"][a:e], one["s"])
        assert np.array_equal(full["kind"][a:e], one["kind"])
        assert np.array_equal(full["k_out"][u][:one["n_out"]], one["k_out"])


def test_bf16_rounding_helper():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -3.14159, 1e-40, 0.0, 300.5])
    got = orc.round_bf16(x)
    ref = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x.astype(np.float32)))
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == np.float32(1.0 + 2 ** -6)   # ties to even
    assert np.array_equal(got[3:], ref[3:])
