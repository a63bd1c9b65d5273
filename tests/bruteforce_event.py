"""Pure-Python brute force of one compression event, for caches of a few rows.

Written separately from the C oracle (different language, different structure:
dict/sorted-based, math.fsum sums) so that the two can be compared on every
small (T, P, B, reserve, W) combination.  Definitions followed: score = mean
causal-softmax attention mass of the window queries (reading of Sec. 1);
two-stage split (Sec. 2.2); C subset R and |R| <= B (Sec. 2.3); merge rule
m_G, k~, v~ (Sec. 2.4); cosine grouping (Sec. 2.5).
"""
from __future__ import annotations

import math
from typing import Dict, List

NOOP, EVICTED, CONSOLIDATED, EXHAUSTED, INACTIVE = 1, 2, 4, 8, 16


def scores(K: List[List[float]], Q: List[List[List[float]]], causal: bool = True) -> List[float]:
    T, d = len(K), len(K[0])
    g, W = len(Q), len(Q[0])
    s = [[] for _ in range(T)]
    for h in range(g):
        for j in range(W):
            last = T - W + j if causal else T - 1
            vis = [i for i in range(T) if i <= last]
            x = {i: math.fsum(Q[h][j][c] * K[i][c] for c in range(d)) / math.sqrt(d) for i in vis}
            mx = max(x.values())
            z = math.fsum(math.exp(x[i] - mx) for i in vis)
            for i in vis:
                s[i].append(math.exp(x[i] - mx) / z)
    return [math.fsum(col) / (g * W) for col in s]


def top(rows: List[int], s: List[float], k: int) -> List[int]:
    return sorted(rows, key=lambda i: (-s[i], i))[:max(k, 0)]


def cosine(a: List[float], b: List[float], w=None) -> float:
    w = [1.0] * len(a) if w is None else w
    na = math.sqrt(math.fsum(c * x * x for c, x in zip(w, a)))
    nb = math.sqrt(math.fsum(c * x * x for c, x in zip(w, b)))
    if na == 0.0 or nb == 0.0:
        return 0.0
    return math.fsum(c * x * y for c, x, y in zip(w, a, b)) / (na * nb)


def band_similarity(a: List[float], b: List[float], bw: List[float], layout: int) -> float:
    """1 - d_kappa(a,b) / (D_a + D_b) with d_kappa = sum_f w_f ||a_f - b_f||, D_x = sum_f w_f ||x_f|| (Sec. 2.5)."""
    d = len(a)
    pairs = [(f, f + d // 2) if layout == 0 else (2 * f, 2 * f + 1) for f in range(d // 2)]
    Da = math.fsum(w * math.hypot(a[i], a[j]) for w, (i, j) in zip(bw, pairs))
    Db = math.fsum(w * math.hypot(b[i], b[j]) for w, (i, j) in zip(bw, pairs))
    if Da == 0.0 or Db == 0.0:
        return 0.0
    dist = math.fsum(w * math.hypot(a[i] - b[i], a[j] - b[j]) for w, (i, j) in zip(bw, pairs))
    return 1.0 - dist / (Da + Db)


def event(K, V, Q, P: int, B: int, reserve: int, gamma: float = 0.5, tau: float = 0.9,
          eps: float = 1e-9, causal: bool = True, mass_in=None, chan_w=None, band_w=None, band_layout: int = 0) -> Dict:
    T, d = len(K), len(K[0])
    W = len(Q[0])
    s = scores(K, Q, causal)
    a = [x + eps + (mass_in[i] if mass_in is not None else 0.0) for i, x in enumerate(s)]
    Nd = T - P
    prefix, decode = list(range(P)), list(range(P, T))
    flags = 0
    groups: Dict[int, List[int]] = {}
    lost = 0.0
    if T <= B:
        flags |= NOOP
        keep = {i: 1 for i in prefix}
        r = min(W, Nd)
        keep.update({i: (2 if i >= T - r else 3) for i in decode})
    else:
        Bp = B - reserve
        if P > Bp:
            flags |= EVICTED
            keep = {i: 1 for i in top(prefix, s, Bp)}
        else:
            keep = {i: 1 for i in prefix}
        Bd = B - len(keep)
        r = min(W, Nd)
        if Nd <= Bd:
            keep.update({i: (2 if i >= T - r else 3) for i in decode})
        elif Bd < r + 2:
            flags |= EXHAUSTED
            r = min(r, Bd)
            recent = [i for i in decode if i >= T - r]
            keep.update({i: 2 for i in recent})
            keep.update({i: 3 for i in top([i for i in decode if i < T - r], s, Bd - r)})
        else:
            flags |= CONSOLIDATED
            room = Bd - r
            c = min(math.ceil(gamma * room), room - 1)
            m = room - c
            recent = [i for i in decode if i >= T - r]
            rest = [i for i in decode if i < T - r]
            core = top(rest, s, c)
            scratch = [i for i in rest if i not in core]
            seeds = sorted(top(scratch, s, m))
            keep.update({i: 2 for i in recent})
            keep.update({i: 3 for i in core})
            keep.update({i: 4 for i in seeds})
            groups = {u: [u] for u in seeds}
            for j in scratch:
                if j in groups:
                    continue
                if band_w is not None:
                    sims = [(band_similarity(K[j], K[u], band_w, band_layout), -u) for u in seeds]
                else:
                    sims = [(cosine(K[j], K[u], chan_w), -u) for u in seeds]
                best, negu = max(sims)
                if best >= tau:
                    groups[-negu].append(j)
                else:
                    lost += a[j]
            if all(len(v) == 1 for v in groups.values()):
                flags |= INACTIVE
    slots = sorted(keep)
    weight = [0.0] * T
    assign = [-1] * T
    k_out, v_out, mass = [], [], []
    for t, i in enumerate(slots):
        members = sorted(groups.get(i, [i])) if keep[i] == 4 else [i]
        mG = math.fsum(a[x] for x in members)
        for x in members:
            weight[x] = a[x] / mG if keep[i] == 4 else 1.0
            assign[x] = t
        if len(members) == 1:
            k_out.append(list(K[i]))
            v_out.append(list(V[i]))
        else:
            k_out.append([math.fsum(weight[x] * K[x][c] for x in members) for c in range(d)])
            v_out.append([math.fsum(weight[x] * V[x][c] for x in members) for c in range(d)])
        mass.append(mG)
    kind = [0] * T
    for i, kd in keep.items():
        kind[i] = kd
    for u, mem in groups.items():
        for x in mem:
            if x != u:
                kind[x] = 5
    top_mass = math.fsum(sorted(s, reverse=True)[:B])
    rho_core = math.fsum(s[i] for i in range(T) if kind[i] in (2, 3)) / top_mass
    rho_rep = math.fsum(mass) / top_mass
    return dict(rho_core=rho_core, rho_rep=rho_rep, s=s, kind=kind, slots=slots, weight=weight, assign=assign, k_out=k_out, v_out=v_out,
                mass=mass, flags=flags, lost=lost, n_out=len(slots))
