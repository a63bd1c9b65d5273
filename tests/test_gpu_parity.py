"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C-ABI."""
import numpy as np
import pytest

from paper_2604_10900_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _small(name, **kw):
    """A benchmark-shaped workload cut down so the oracle finishes in seconds."""
    return wl.WORKLOADS[name].with_(**kw)


def _run(w, units=None, tau=0.9, **prm):
    import gpu_harness as gh
    hb = wl.make_batch(w, units)
    run = gh.GpuRun(hb, tau=tau, **prm)
    g = run.event()
    o = gh.run_oracle(hb, tau=tau, causal=prm.get("causal", 1), gamma=prm.get("gamma", 0.5))
    st = gh.compare_event(hb, g, o, tau=tau)
    return hb, run, g, o, st


def test_tiny_config_whole_event():
    """Config 1: fp32 cache, d=64, 1024 rows, budget 128 (both heads)."""
    hb, run, g, o, st = _run(wl.WORKLOADS["tiny"])
    assert st["cascaded"] == 0 and st["merged_elems"] > 0
    assert (g["n_out"] == 128).all()
    assert not run.ctx.used_tensor_path


@pytest.mark.parametrize("score_path", [0, 1])
def test_reasoning_shape_bf16(score_path):
    """Config-2 shape (d=128, g=7, W=64, bf16, outlier channels, geometric clusters), 2 layers, ragged tail."""
    w = _small("reasoning8k_b384", layers=2, decode=2048 + 37)
    hb, run, g, o, st = _run(w, score_path=score_path)
    assert st["cascaded"] <= 1
    assert st["merged_elems"] > 0
    assert st["max_score_rel"] < 1e-5
    assert run.ctx.used_tensor_path == (score_path == 0)


@pytest.mark.parametrize("score_path", [0, 1])
def test_long_reasoning_shape_bf16(score_path):
    """Config-3 shape (g=4, W=128 -> 512 query rows), several key tiles and a ragged last tile."""
    w = _small("reasoning32k_b512", layers=1, kv_heads=3, decode=4096 + 77)
    hb, run, g, o, st = _run(w, score_path=score_path)
    assert st["cascaded"] <= 1
    assert (g["n_out"] == 512).all()
    assert run.ctx.used_tensor_path == (score_path == 0)
    print("score path", score_path, "max rel err", st["max_score_rel"], "exempt rows", st["exempt_rows"], "flipped", st["flipped_rows"])


def test_many_seeds_share_accumulator_buffers():
    """Budget 1024 on the config-3 shape: m = 192 seeds, so two epilogue groups split the seed columns."""
    w = _small("reasoning32k_b1024", layers=1, kv_heads=2, decode=4096 + 77)
    hb, run, g, o, st = _run(w)
    assert (g["plan"][:, 5] == 192).all() and (g["n_out"] == 1024).all()
    assert st["cascaded"] <= 1 and st["merged_elems"] > 0


def _next_cache(w, hb, o, rng, n_new=128):
    """The cache a serving loop holds after an event and n_new more decode steps, built from the ORACLE's result of
    that event (rounded to the cache dtype): its compacted rows, then n_new appended rows of which half repeat kept
    rows with a little noise; representatives carry the group mass they were given."""
    from oracle import cask_oracle as orc
    d = w.head_dim
    k2, v2, mass, T2, P2 = [], [], [], [], []
    for u in range(hb.n_units):
        n = int(o["n_out"][u])
        ko = wl.to_cache_dtype(orc.round_bf16(o["k_out"][u][:n]), w.dtype)
        vo = wl.to_cache_dtype(orc.round_bf16(o["v_out"][u][:n]), w.dtype)
        pkeep = int(o["plan"][u][1])
        fresh_k = wl.to_cache_dtype(rng.standard_normal((n_new, d)).astype(np.float32) * wl.channel_scale(w, 0, 0), w.dtype)
        src = rng.integers(pkeep, n, n_new // 2)
        noisy = wl.as_float32(ko[src], w.dtype) + 0.05 * rng.standard_normal((n_new // 2, d)).astype(np.float32)
        fresh_k[: n_new // 2] = wl.to_cache_dtype(noisy, w.dtype)
        k2.append(np.concatenate([ko, fresh_k]))
        v2.append(np.concatenate([vo, wl.to_cache_dtype(rng.standard_normal((n_new, d)).astype(np.float32), w.dtype)]))
        mass.append(np.concatenate([np.where(o["slot_kind"][u][:n] == 4, o["slot_mass"][u][:n], 0.0), np.zeros(n_new)]))
        T2.append(n + n_new)
        P2.append(pkeep)
    T2 = np.array(T2, np.int32)
    hb2 = wl.Batch(wl=w, k=np.concatenate(k2), v=np.concatenate(v2), q=hb.q, T=T2, P=np.array(P2, np.int32), B=hb.B,
                   reserve=hb.reserve, tok_off=np.concatenate([[0], np.cumsum(T2)]).astype(np.int64),
                   unit_ids=hb.unit_ids, mass_in=np.concatenate(mass).astype(np.float32))
    return hb2


def test_carried_mass_trigger_loop_on_compacted_caches():
    """Steady state of a serving loop: the cache left by one event, grown by 128 new decode rows, is compressed
    again, three times over; representatives bring the group mass they were given (a_i = s_i + eps + carried mass).
    Every event's inputs are built from the oracle's previous result, identical bytes for both sides; the second
    event runs on a paged cache and is written back into its pages."""
    import gpu_harness as gh
    import torch
    w = _small("reasoning8k_b384", layers=1, kv_heads=3, decode=2048)
    hb, run, g, o, st = _run(w)
    rng = np.random.default_rng(77)
    B = w.budget
    for step in range(3):
        hb = _next_cache(w, hb, o, rng)
        assert (hb.mass_in > 0).any() and int(hb.T.max()) <= 1024          # the small-unit kernels serve it
        run = gh.GpuRun(hb, page_size=64 if step == 1 else 0)
        g = run.event()
        assert run.ctx.device_flags() == 0
        o = gh.run_oracle(hb)
        st = gh.compare_event(hb, g, o)
        assert st["dispersion_checked"] > 0
        assert (g["n_out"] == B).all() and st["merged_elems"] > 0 and st["cascaded"] <= 1
        if step == 1:
            cb = run.cb
            cb.cask_writeback_paged(run.ctx, run.batch, run.prm, run.out_struct, run.dev["k"], run.dev["v"], run.ws,
                                    run.ws_bytes)
            torch.cuda.synchronize()
            table = run.block_table.cpu().numpy().astype(np.int64)
            off = 0
            for u in range(hb.n_units):
                t = np.arange(int(g["n_out"][u]))
                rows = torch.from_numpy(table[off + t // 64] * 64 + t % 64).to(run.device)
                assert torch.equal(run.dev["k"][rows].view(torch.uint16), run.out["k_out"][u, :len(t)].view(torch.uint16))
                off += (int(hb.T[u]) + 63) // 64
    # the carried mass changes the fold: without it the merged rows come out differently
    plain = wl.Batch(wl=w, k=hb.k, v=hb.v, q=hb.q, T=hb.T, P=hb.P, B=hb.B, reserve=hb.reserve, tok_off=hb.tok_off,
                     unit_ids=hb.unit_ids)
    g3 = gh.GpuRun(plain).event()
    assert np.array_equal(g3["kind"], g["kind"]) and not np.array_equal(g3["weight"], g["weight"])


@pytest.mark.parametrize("name,kw,tensor_assign", [
    ("reasoning32k_b512", dict(layers=1, kv_heads=2, decode=4096 + 77), True),      # m = 64: hi/lo seed columns
    ("reasoning32k_b1024", dict(layers=1, kv_heads=2, decode=4096 + 77), False),    # m = 192: SIMT assignment
    ("tiny", dict(), False)])
def test_channel_weighted_similarity(name, kw, tensor_assign):
    """Sec. 2.5: per-channel (frequency band) weights in the merge similarity."""
    import gpu_harness as gh
    w = _small(name, **kw)
    hb = wl.make_batch(w)
    rng = np.random.default_rng(5)
    cw = (rng.random(w.head_dim) ** 2 + 0.02).astype(np.float32)
    cw[rng.random(w.head_dim) < 0.1] = 0.0                      # bands of no future relevance
    run = gh.GpuRun(hb, chan_w=cw)
    g = run.event()
    o = gh.run_oracle(hb, chan_w=cw)
    st = gh.compare_event(hb, g, o, geom=dict(chan_w=cw))
    assert st["cascaded"] <= 1 and st["merged_elems"] > 0
    plain = gh.run_oracle(hb)
    assert not np.array_equal(plain["sim"], o["sim"])


@pytest.mark.parametrize("name,kw,layout", [
    ("reasoning32k_b512", dict(layers=1, kv_heads=2, decode=2048 + 77), 0),
    ("reasoning32k_b1024", dict(layers=1, kv_heads=2, decode=2048 + 77), 1),       # m = 192: three seed steps
    ("serving_steady_b512", dict(layers=1, kv_heads=2, n_seqs=2), 0),              # short units, carried masses
    ("tiny", dict(), 1)])
def test_band_distance_similarity(name, kw, layout):
    """Sec. 2.5 in its own form: d_kappa = sum_f w_f ||k_if - k_jf|| over rotary bands, as the similarity
    1 - d_kappa / (D_i + D_j), in place of the cosine."""
    import gpu_harness as gh
    w = _small(name, **kw)
    hb = wl.make_batch(w)
    rng = np.random.default_rng(7)
    bw = (rng.random(w.head_dim // 2) ** 2 + 0.02).astype(np.float32)
    bw[rng.random(w.head_dim // 2) < 0.1] = 0.0                 # bands of no future relevance
    run = gh.GpuRun(hb, band_w=bw, band_layout=layout, tau=0.8)
    g = run.event()
    assert run.ctx.device_flags() == 0
    o = gh.run_oracle(hb, band_w=bw, band_layout=layout, tau=0.8)
    st = gh.compare_event(hb, g, o, tau=0.8, geom=dict(band_w=bw, band_layout=layout))
    assert st["dispersion_checked"] > 0
    assert st["cascaded"] <= 1 and st["merged_elems"] > 0
    other = gh.run_oracle(hb, band_w=bw, band_layout=1 - layout, tau=0.8)
    assert not np.array_equal(other["sim"], o["sim"])
    # both kinds of weights at once are refused before any launch
    cb = run.cb
    bad = gh.GpuRun(hb, band_w=bw, chan_w=np.ones(w.head_dim, np.float32))
    assert cb.cask_compress_event(bad.ctx, bad.batch, bad.prm, bad.out_struct, bad.ws, bad.ws_bytes, check=False) == cb.ERR_SHAPE


@pytest.mark.parametrize("group,window", [(1, 32), (3, 32), (1, 128), (2, 128), (3, 128), (5, 96)])
def test_query_row_counts_that_fill_one_to_four_accumulator_slots(group, window):
    """32 to 480 window-query rows: one, two, three and four 128-column slots, a ragged last slot, idle epilogue
    groups and warps (tensor-core scoring throughout)."""
    w = _small("reasoning32k_b512", layers=1, kv_heads=2, group=group, window=window, decode=2048 + 61, prefix=300,
               budget=512, reserve=256)
    hb, run, g, o, st = _run(w)
    assert run.ctx.used_tensor_path and run.ctx.device_flags() == 0
    assert st["max_score_rel"] < 1e-5 and st["cascaded"] <= 1
    assert (g["n_out"] == 512).all()


def test_prompt_heavy_two_stage():
    """Config-4 shape: prefix eviction fires before decode consolidation."""
    w = _small("prompt_heavy", layers=1, kv_heads=2, prefix=3072, decode=1024, budget=1024, reserve=256)
    hb, run, g, o, st = _run(w)
    from oracle import cask_oracle as orc
    assert (g["unit_status"] & orc.PREFIX_EVICTED).all() and (g["unit_status"] & orc.DECODE_CONSOLIDATED).all()
    assert (g["n_out"] == 1024).all()


@pytest.mark.parametrize("reserve,exhausted", [(66, False), (65, True), (64, True)])
def test_prefix_budget_exhausted_boundary(reserve, exhausted):
    """Config-4 variant around B_d = r + 2 (Sec. 5.2: the available slots collapse)."""
    w = _small("prompt_heavy_boundary", layers=1, kv_heads=1, prefix=2048, decode=512, budget=512, reserve=reserve)
    hb, run, g, o, st = _run(w)
    from oracle import cask_oracle as orc
    assert bool(g["unit_status"][0] & orc.PREFIX_BUDGET_EXHAUSTED) == exhausted
    assert g["n_out"][0] == 512
    if exhausted:
        assert not np.isin(g["kind"], (4, 5)).any()


def test_ragged_batch_mixed_outcomes():
    """Units of different length and budget in one call: under budget, prefix-only, decode-active."""
    base = wl.WORKLOADS["tiny"].with_(dtype=wl.DTYPE_BF16, head_dim=128, group=2, window=8)
    import gpu_harness as gh
    parts = []
    specs = [(128, 896, 128, 64), (16, 40, 64, 32), (300, 0, 128, 64), (64, 131, 96, 90), (10, 500, 700, 100)]
    ks, vs, qs, T, P, B, R = [], [], [], [], [], [], []
    for i, (p, nd, b, r) in enumerate(specs):
        w = base.with_(prefix=p, decode=nd, budget=b, reserve=r)
        k, v, q = wl.make_unit(w, i, 0, 0)
        ks.append(k); vs.append(v); qs.append(q[None])
        T.append(p + nd); P.append(p); B.append(b); R.append(r)
    tok = np.concatenate([[0], np.cumsum(T)]).astype(np.int64)
    hb = wl.Batch(wl=base, k=np.concatenate(ks), v=np.concatenate(vs), q=np.concatenate(qs),
                  T=np.array(T, np.int32), P=np.array(P, np.int32), B=np.array(B, np.int32),
                  reserve=np.array(R, np.int32), tok_off=tok, unit_ids=[(i, 0, 0) for i in range(len(T))])
    run = gh.GpuRun(hb)
    g = run.event()
    o = gh.run_oracle(hb)
    st = gh.compare_event(hb, g, o)
    from oracle import cask_oracle as orc
    assert g["unit_status"][1] & orc.NOOP_UNDER_BUDGET and g["n_out"][1] == 56
    assert g["unit_status"][4] & orc.NOOP_UNDER_BUDGET
    assert g["n_out"][2] == 64          # prefix-only event leaves the reserve free
    # unit independence: each unit alone gives the same bytes as inside the batch
    for u in (0, 3):
        one = wl.Batch(wl=base, k=ks[u], v=vs[u], q=qs[u], T=hb.T[u:u + 1], P=hb.P[u:u + 1], B=hb.B[u:u + 1],
                       reserve=hb.reserve[u:u + 1], tok_off=np.array([0, T[u]], np.int64), unit_ids=[(u, 0, 0)])
        g1 = gh.GpuRun(one).event()
        a = int(tok[u])
        assert np.array_equal(g1["s"], g["s"][a:a + T[u]])
        assert np.array_equal(g1["kind"], g["kind"][a:a + T[u]])
        n = int(g1["n_out"][0])
        assert np.array_equal(g1["k_out"][0][:n], g["k_out"][u][:n])
        assert np.array_equal(g1["v_out"][0][:n], g["v_out"][u][:n])


@pytest.mark.parametrize("seed,max_rows", [(1, 1024), (2, 1024), (3, 2600)])
def test_random_ragged_batches(seed, max_rows):
    """48 units of random length, prefix, budget and reserve in one call (all at most 1,024 rows: the short-unit
    kernels; or up to 2,600: the general ones), every one against the oracle.  Prefix-only units, units under budget,
    exhausted decode budgets and single-slot budgets all occur."""
    import gpu_harness as gh
    rng = np.random.default_rng(seed)
    base = wl.WORKLOADS["tiny"].with_(dtype=wl.DTYPE_BF16, head_dim=128, group=2, window=16, cluster_frac=0.6,
                                      n_centres=0)
    ks, vs, qs, T, P, B, R = [], [], [], [], [], [], []
    for i in range(48):
        t = int(rng.integers(16, max_rows + 1))
        p = int(rng.integers(0, t - 15)) if rng.random() < 0.8 else t       # a fifth are prefix-only caches
        b = int(rng.integers(1, min(t + 40, 700)))
        r = int(rng.integers(0, b + 1))
        w = base.with_(prefix=p, decode=t - p, budget=b, reserve=r)
        k, v, q = wl.make_unit(w, i, seed, 0)
        ks.append(k); vs.append(v); qs.append(q[None])
        T.append(t); P.append(p); B.append(b); R.append(r)
    hb = wl.Batch(wl=base, k=np.concatenate(ks), v=np.concatenate(vs), q=np.concatenate(qs),
                  T=np.array(T, np.int32), P=np.array(P, np.int32), B=np.array(B, np.int32),
                  reserve=np.array(R, np.int32), tok_off=np.concatenate([[0], np.cumsum(T)]).astype(np.int64),
                  unit_ids=[(i, 0, 0) for i in range(len(T))])
    run = gh.GpuRun(hb)
    g = run.event()
    assert run.ctx.device_flags() == 0
    o = gh.run_oracle(hb)
    st = gh.compare_event(hb, g, o)
    from oracle import cask_oracle as orc
    seen = np.bitwise_or.reduce(g["unit_status"])
    assert seen & orc.NOOP_UNDER_BUDGET and seen & orc.PREFIX_EVICTED and seen & orc.DECODE_CONSOLIDATED
    assert st["cascaded"] <= 4


def _query_stats(w, n_units, rng, n_delta=9):
    nb = w.head_dim // 2
    mu = rng.standard_normal((n_units, w.group, nb, 2)).astype(np.float32)
    pi = rng.random((n_units, w.group, n_delta)).astype(np.float32)
    pi /= pi.sum(-1, keepdims=True)
    grid = np.concatenate([[0.0], np.sort(rng.integers(1, 4096, n_delta - 1))]).astype(np.float32)
    omega = (1.0 / (10000.0 ** (np.arange(nb) / nb))).astype(np.float32)       # rotary-embedding frequencies
    return mu, pi, grid, omega


@pytest.mark.parametrize("name,kw,layout,paged", [
    ("reasoning32k_b512", dict(layers=1, kv_heads=2, decode=8192 + 77), 0, 0),
    ("reasoning8k_b384", dict(layers=1, kv_heads=2, decode=3000), 1, 64),
    ("tiny", dict(), 0, 0)])
def test_query_statistics_scorer(name, kw, layout, paged):
    """App. B: horizon kernel + horizon-averaged mean score, one pass over the keys, against the oracle.  The sum
    has d/2 terms of size |A_f||k_f|; single-precision sine, cosine and accumulation leave an error of a few 1e-7
    of sum_f |A_f||k_f| per row, so the bound is 2e-6 of that sum (about ten times what is seen)."""
    import gpu_harness as gh
    import torch
    from oracle import cask_oracle as orc
    w = _small(name, **kw)
    hb = wl.make_batch(w)
    rng = np.random.default_rng(41)
    mu, pi, grid, omega = _query_stats(w, hb.n_units, rng)
    run = gh.GpuRun(hb, page_size=paged)
    cb = run.cb
    dev = [torch.from_numpy(x).to(run.device) for x in (mu, pi, grid, omega)]
    for use_delta in (False, True):
        delta = rng.uniform(-5000.0, 40000.0, int(hb.tok_off[-1])).astype(np.float32) if use_delta else None
        ddev = None if delta is None else torch.from_numpy(delta).to(run.device)
        qs, keep = cb.make_query_stats(dev[0], dev[1], dev[2], dev[3], layout, ddev)
        s = torch.full((int(hb.tok_off[-1]),), float("nan"), dtype=torch.float32, device=run.device)
        cb.cask_score_stats(run.ctx, run.batch, run.prm, qs, s, run.ws, run.ws_bytes)
        torch.cuda.synchronize()
        assert run.ctx.device_flags() == 0
        got = s.cpu().numpy().astype(np.float64)
        kf = wl.as_float32(hb.k, w.dtype)
        nb = w.head_dim // 2
        c0 = np.arange(nb) if layout == 0 else 2 * np.arange(nb)
        c1 = c0 + (nb if layout == 0 else 1)
        worst = 0.0
        for u in range(hb.n_units):
            a, b = int(hb.tok_off[u]), int(hb.tok_off[u + 1])
            want = orc.score_stats(kf[a:b], mu[u], pi[u].astype(np.float64), grid.astype(np.float64),
                                   omega.astype(np.float64), layout, None if delta is None else delta[a:b].astype(np.float64))
            kap = (pi[u].astype(np.float64)[:, :, None] * np.exp(1j * omega[None, None, :].astype(np.float64) * grid[None, :, None])).sum(1)
            A = np.abs(((mu[u][..., 0] + 1j * mu[u][..., 1]) * kap).mean(0))
            scale = (np.hypot(kf[a:b][:, c0], kf[a:b][:, c1]) * A[None, :]).sum(1)
            err = np.abs(got[a:b] - want) / scale
            worst = max(worst, float(err.max()))
        assert worst < 2e-6, worst
        assert (got < 0).any() and (got > 0).any()
    # arguments are checked on the host
    bad, _ = cb.make_query_stats(dev[0], dev[1], dev[2], dev[3], 2)
    assert cb.cask_score_stats(run.ctx, run.batch, run.prm, bad, s, run.ws, run.ws_bytes, check=False) == cb.ERR_SHAPE


@pytest.mark.parametrize("decode", [600, 3000])
def test_exact_duplicates_tie_at_the_selection_thresholds(decode):
    """Decode rows that are exact copies of a few centres have exactly equal scores, so the core and seed thresholds
    fall inside runs of equal keys and the row index decides (short-unit ranking and two-threshold radix select,
    both through their tie paths); merged rows equal their centre."""
    import gpu_harness as gh
    w = _small("reasoning8k_b384", layers=1, kv_heads=2, decode=decode, noise=0.0, cluster_frac=1.0, n_centres=37)
    hb = wl.make_batch(w)
    run = gh.GpuRun(hb)
    g = run.event()
    o = gh.run_oracle(hb)
    # the duplicates really tie: far fewer distinct scores than rows in the decode region
    a, T, P = 0, int(hb.T[0]), int(hb.P[0])
    assert len(np.unique(o["s"][a + P:a + T - w.window])) < (T - P) // 4
    # Equal keys in differently masked tiles can come out one unit in the last place apart in fp32 (the masked and the
    # plain block forms add in a different order), so a unit may resolve a run of ties differently from the oracle;
    # compare_event accepts that only inside the tolerance band around a threshold.
    st = gh.compare_event(hb, g, o)
    assert st["exempt_rows"] > 0 and st["cascaded"] <= hb.n_units


@pytest.mark.parametrize("prefix,decode,budget,reserve", [
    (200, 230, 128, 64),        # prefix eviction and scratch selection over at most 256 rows: ranking by counting
    (700, 900, 256, 128),       # 257 .. 1,024 rows each: the sorted path
    (300, 650, 256, 128),       # the same in units of at most 1,024 rows, whose selection CTAs have 256 threads
    (1000, 1040, 384, 192),     # exactly 1,000 and 1,024 - 48 rows: the sorted path at its upper end, ragged
    (1500, 3000, 384, 192),     # above 1,024 rows: radix select (one and two thresholds)
])
def test_every_selection_path_with_injected_tied_scores(prefix, decode, budget, reserve):
    """Prefix eviction, core selection and seed selection on injected scores that take a dozen distinct values, so
    every threshold falls inside a long run of equal keys and the row index decides: the kinds must equal the
    oracle's on the same scores, through the staged calls, for ranges that take each of the three selection paths
    (counting, sorting network, radix select)."""
    import gpu_harness as gh
    import torch
    from oracle import cask_oracle as orc
    w = _small("reasoning8k_b384", layers=1, kv_heads=3, group=2, window=16, prefix=prefix, decode=decode,
               budget=budget, reserve=reserve)
    hb = wl.make_batch(w)
    run = gh.GpuRun(hb)
    cb, o = run.cb, run.out
    kf = wl.as_float32(hb.k, w.dtype)
    rng = np.random.default_rng(prefix * 7 + decode)
    n = int(hb.tok_off[-1])
    s32 = (rng.integers(1, 13, n) / np.float32(16.0)).astype(np.float32)
    s32[rng.random(n) < 0.02] += np.float32(1.0)           # a few rows clear of every tie
    sd = s32.astype(np.float64)
    s_dev = run.dev_f32(s32)
    cb.cask_prefix_evict(run.ctx, run.batch, run.prm, s_dev, o["kind"], o["plan"], run.ws, run.ws_bytes)
    cb.cask_select_core(run.ctx, run.batch, run.prm, s_dev, o["plan"], o["kind"], run.ws, run.ws_bytes)
    torch.cuda.synchronize()
    kind_g, plan_g = o["kind"].cpu().numpy(), o["plan"].cpu().numpy()
    want = []
    for u in range(hb.n_units):
        a, T, P = int(hb.tok_off[u]), int(hb.T[u]), int(hb.P[u])
        pl = orc.plan(T, P, int(hb.B[u]), int(hb.reserve[u]), w.window, 0.5)
        assert np.array_equal(plan_g[u], pl)
        kind = np.zeros(T, np.uint8)
        orc.prefix_evict(sd[a:a + T], P, pl, kind)
        orc.select_core(sd[a:a + T], T, P, pl, kind)
        assert np.array_equal(kind_g[a:a + T], kind), f"unit {u}"
        want.append(kind)
    cb.cask_consolidate_scratch(run.ctx, run.batch, run.prm, s_dev, o["plan"], o["kind"], o["seed_of"], o["weight"],
                                o["sim"], o["unit_status"], o["lost_mass"], run.ws, run.ws_bytes)
    torch.cuda.synchronize()
    kind_g2 = o["kind"].cpu().numpy()
    for u in range(hb.n_units):
        a, T, P = int(hb.tok_off[u]), int(hb.T[u]), int(hb.P[u])
        kind = want[u].copy()
        orc.consolidate(kf[a:a + T], sd[a:a + T], P, plan_g[u], kind, tau=0.9, eps=float(np.float32(1e-9)))
        assert (kind == 4).any()
        assert np.array_equal(kind == 4, kind_g2[a:a + T] == 4), f"unit {u}: seed rows"
    assert run.ctx.device_flags() == 0


@pytest.mark.parametrize("tau", [-1.0, 1.5])
def test_tau_extremes(tau):
    """tau = -1 merges every scratch row (no lost mass); tau > 1 is plain top-k eviction."""
    hb, run, g, o, st = _run(wl.WORKLOADS["tiny"], tau=tau)
    if tau < 0:
        assert (g["lost_mass"] == 0).all()
        assert not ((g["kind"] == 0) & (np.arange(len(g["kind"])) % 1024 >= 128)).any()
    else:
        from oracle import cask_oracle as orc
        assert (g["unit_status"] & orc.MERGE_INACTIVE).all() and not (g["kind"] == 5).any()


def test_non_causal_and_other_gamma():
    _run(wl.WORKLOADS["tiny"], causal=0)
    _run(wl.WORKLOADS["tiny"], gamma=0.25)


def test_strided_rows_and_fp32_d128():
    import gpu_harness as gh
    w = wl.WORKLOADS["tiny"].with_(head_dim=128)
    hb = wl.make_batch(w)
    g = gh.GpuRun(hb, row_stride=160).event()
    o = gh.run_oracle(hb)
    gh.compare_event(hb, g, o)
    wb = wl.WORKLOADS["tiny"].with_(dtype=wl.DTYPE_BF16)       # bf16 with d = 64: SIMT path
    hb = wl.make_batch(wb)
    run = gh.GpuRun(hb, row_stride=72)
    g = run.event()
    gh.compare_event(hb, g, gh.run_oracle(hb))


def test_supplied_normalisers():
    """lse_in from the oracle: the normaliser pass is skipped and scores still match."""
    import gpu_harness as gh
    w = wl.WORKLOADS["tiny"]
    hb = wl.make_batch(w)
    o = gh.run_oracle(hb)
    from oracle import cask_oracle as orc
    _, lse = orc.score_batch(hb.k, hb.q, hb.tok_off)
    run = gh.GpuRun(hb, lse_in=lse.reshape(hb.n_units, -1))
    n0 = run.ctx.launches
    g = run.event()
    gh.compare_event(hb, g, o)
    run2 = gh.GpuRun(hb)
    run2.event()
    assert run.ctx.launches - n0 < run2.ctx.launches       # one pass fewer


@pytest.mark.parametrize("name,kw", [
    ("reasoning8k_b384", dict(decode=1500)),
    # units of at most 1,024 rows: the event takes its fused selection kernel, the staged calls their own kernels
    ("reasoning8k_b384", dict(decode=600)),
    ("prompt_heavy", dict(prefix=700, decode=200, budget=512, reserve=160)),     # with prefix eviction
    # exact duplicates: runs of equal scores across the thresholds, the fused selections take their tie paths
    ("reasoning8k_b384", dict(decode=3000, noise=0.0, cluster_frac=1.0, n_centres=37)),
    ("reasoning8k_b384", dict(decode=600, noise=0.0, cluster_frac=1.0, n_centres=37)),
])
def test_deterministic_and_staged_equals_fused(name, kw):
    """Same inputs twice -> same bytes; the five staged calls give the event's bytes."""
    import gpu_harness as gh
    import torch
    w = _small(name, layers=1, kv_heads=2, **kw)
    hb = wl.make_batch(w)
    run = gh.GpuRun(hb)
    g1 = run.event()
    g2 = run.event()
    for k in g1:
        assert np.array_equal(g1[k], g2[k]), k
    cb = run.cb
    st = gh.GpuRun(hb)
    o = st.out
    cb.cask_score(st.ctx, st.batch, st.prm, o["s"], o["lse"], st.ws, st.ws_bytes)
    cb.cask_prefix_evict(st.ctx, st.batch, st.prm, o["s"], o["kind"], o["plan"], st.ws, st.ws_bytes)
    cb.cask_select_core(st.ctx, st.batch, st.prm, o["s"], o["plan"], o["kind"], st.ws, st.ws_bytes)
    cb.cask_consolidate_scratch(st.ctx, st.batch, st.prm, o["s"], o["plan"], o["kind"], o["seed_of"], o["weight"],
                                o["sim"], o["unit_status"], o["lost_mass"], st.ws, st.ws_bytes)
    cb.cask_compact(st.ctx, st.batch, st.prm, o["s"], o["kind"], o["seed_of"], o["weight"], st.out_struct, st.ws,
                    st.ws_bytes)
    torch.cuda.synchronize()
    g3 = st.numpy_outputs()
    for k in g1:
        assert np.array_equal(g1[k], g3[k]), k


def test_stages_with_oracle_intermediates_injected():
    """Each stage fed the oracle's upstream results (as fp32): selections must match with no exemption."""
    import gpu_harness as gh
    import torch
    from oracle import cask_oracle as orc
    w = _small("reasoning8k_b512", layers=1, kv_heads=2, decode=3000)
    hb = wl.make_batch(w)
    run = gh.GpuRun(hb)
    cb, o = run.cb, run.out
    kf, vf, qf = (wl.as_float32(x, w.dtype) for x in (hb.k, hb.v, hb.q))
    s64, _ = orc.score_batch(kf, qf, hb.tok_off)
    s32 = s64.astype(np.float32)
    sd = s32.astype(np.float64)              # the oracle works on exactly the values the GPU gets
    s_dev = run.dev_f32(s32)
    cb.cask_prefix_evict(run.ctx, run.batch, run.prm, s_dev, o["kind"], o["plan"], run.ws, run.ws_bytes)
    cb.cask_select_core(run.ctx, run.batch, run.prm, s_dev, o["plan"], o["kind"], run.ws, run.ws_bytes)
    torch.cuda.synchronize()
    kind_g = o["kind"].cpu().numpy()
    plan_g = o["plan"].cpu().numpy()
    for u in range(hb.n_units):
        a, T, P = int(hb.tok_off[u]), int(hb.T[u]), int(hb.P[u])
        pl = orc.plan(T, P, int(hb.B[u]), int(hb.reserve[u]), w.window, 0.5)
        assert np.array_equal(plan_g[u], pl)
        kind = np.zeros(T, np.uint8)
        orc.prefix_evict(sd[a:a + T], P, pl, kind)
        orc.select_core(sd[a:a + T], T, P, pl, kind)
        assert np.array_equal(kind_g[a:a + T], kind), f"unit {u}"
    # consolidation on the oracle's kinds
    cb.cask_consolidate_scratch(run.ctx, run.batch, run.prm, s_dev, o["plan"], o["kind"], o["seed_of"], o["weight"],
                                o["sim"], o["unit_status"], o["lost_mass"], run.ws, run.ws_bytes)
    torch.cuda.synchronize()
    kind_g2, seed_g, sim_g, w_g = (o[x].cpu().numpy() for x in ("kind", "seed_of", "sim", "weight"))
    inj_kind, inj_seed, inj_w = kind_g2.copy(), seed_g.copy(), w_g.astype(np.float64)
    for u in range(hb.n_units):
        a, T, P = int(hb.tok_off[u]), int(hb.T[u]), int(hb.P[u])
        kind = kind_g[a:a + T].copy()
        c = orc.consolidate(kf[a:a + T], sd[a:a + T], P, plan_g[u], kind, tau=0.9, eps=float(np.float32(1e-9)))
        assert np.array_equal(kind == 4, kind_g2[a:a + T] == 4), "seed sets (same scores) must match exactly"
        near = (np.abs(c["sim"] - 0.9) <= gh.SIM_BAND) | ((c["sim2"] > -1.5) & (c["sim"] - c["sim2"] <= gh.SIM_BAND))
        bad = (kind != kind_g2[a:a + T]) | (c["seed_of"] != seed_g[a:a + T])
        assert not (bad & ~near).any(), f"unit {u}: non-exempt assignment differences"
        has = c["sim"] > -1.5
        assert np.abs(sim_g[a:a + T][has] - c["sim"][has]).max() < 2e-6
        same = ~bad
        assert np.allclose(w_g[a:a + T][same], c["weight"][same], rtol=2e-5, atol=1e-9)
        inj_kind[a:a + T], inj_seed[a:a + T], inj_w[a:a + T] = kind, c["seed_of"], c["weight"]
    # compaction on the oracle's kinds / seeds / weights
    kd, so, wt = run.dev_arr(inj_kind, np.uint8), run.dev_arr(inj_seed, np.int32), run.dev_f32(inj_w)
    cb.cask_compact(run.ctx, run.batch, run.prm, s_dev, kd, so, wt, run.out_struct, run.ws, run.ws_bytes)
    torch.cuda.synchronize()
    g = run.numpy_outputs()
    for u in range(hb.n_units):
        a, T = int(hb.tok_off[u]), int(hb.T[u])
        oc = orc.compact(kf[a:a + T], vf[a:a + T], inj_kind[a:a + T], inj_seed[a:a + T],
                         inj_w[a:a + T].astype(np.float32).astype(np.float64), sd[a:a + T],
                         eps=float(np.float32(1e-9)))
        n = oc["n_out"]
        assert g["n_out"][u] == n
        assert np.array_equal(g["slot_src"][u][:n], oc["slot_src"])
        assert np.array_equal(g["slot_kind"][u][:n], oc["slot_kind"])
        assert np.array_equal(g["assign"][a:a + T], oc["assign"])
        assert np.allclose(g["slot_mass"][u][:n], oc["slot_mass"], rtol=2e-5)
        err = np.abs(g["k_out"][u][:n].astype(np.float64) - oc["k_out"])
        assert (err <= np.maximum(2e-2, 2.0 ** -7 * np.abs(oc["k_out"]))).all()
        errv = np.abs(g["v_out"][u][:n].astype(np.float64) - oc["v_out"])
        assert (errv <= np.maximum(2e-2, 2.0 ** -7 * np.abs(oc["v_out"]))).all()


def test_bad_arguments_are_refused_on_the_host_before_any_launch():
    import gpu_harness as gh
    hb = wl.make_batch(wl.WORKLOADS["tiny"])
    run = gh.GpuRun(hb)
    cb = run.cb
    n0 = run.ctx.launches

    def rc(**chg):
        b, keep = cb.make_batch(run.dev["k"], run.dev["v"], run.dev["q"],
                                chg.get("T", hb.T), chg.get("P", hb.P), chg.get("B", hb.B),
                                chg.get("reserve", hb.reserve), hb.tok_off, chg.get("d", 64), 4,
                                chg.get("W", 16), chg.get("dtype", 1), row_stride=chg.get("row_stride"),
                                page_size=chg.get("page_size", 0))
        if chg.get("null_k"):
            b.k = None
        return cb.cask_compress_event(run.ctx, b, chg.get("prm", run.prm), run.out_struct,
                                      chg.get("ws", run.ws), chg.get("ws_bytes", run.ws_bytes), check=False)

    assert rc() == cb.OK
    n1 = run.ctx.launches
    assert rc(null_k=True) == cb.ERR_NULL
    assert rc(B=np.array([0, 128], np.int32)) == cb.ERR_SHAPE
    assert rc(P=np.array([2000, 128], np.int32)) == cb.ERR_SHAPE
    assert rc(W=2000) == cb.ERR_SHAPE
    assert rc(reserve=np.array([129, 0], np.int32)) == cb.ERR_SHAPE
    assert rc(d=60) == cb.ERR_SHAPE
    assert rc(row_stride=66) == cb.ERR_ALIGN
    assert rc(page_size=16) == cb.ERR_NULL            # a paged batch without its block table
    assert rc(ws_bytes=1024) == cb.ERR_WORKSPACE
    assert rc(prm=cb.params(gamma=1.5)) == cb.ERR_PARAM
    assert rc(prm=cb.params(eps=0.0)) == cb.ERR_PARAM
    small = cb.make_outputs(run.out, 64)
    b, keep = cb.make_batch(run.dev["k"], run.dev["v"], run.dev["q"], hb.T, hb.P, hb.B, hb.reserve, hb.tok_off,
                            64, 4, 16, 1)
    assert cb.cask_compress_event(run.ctx, b, run.prm, small, run.ws, run.ws_bytes, check=False) == cb.ERR_SHAPE
    import torch
    torch.cuda.synchronize()
    assert run.ctx.launches == n1 > n0       # the refused calls launched nothing; the context is still usable
    run.event()


def test_a_bounded_device_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """Every barrier wait of the kernels gives up after a wall-time limit and ends the kernel with CASK_ST_TIMEOUT
    instead of hanging.  The self-test entry point makes one such wait run out (a barrier nobody arrives at, a limit
    of two milliseconds): the kernel must return by itself, the flag must show, a second warp waiting with the
    default one-second limit must follow the first out at once, and the context must still give a correct event."""
    import gpu_harness as gh
    import torch
    hb = wl.make_batch(wl.WORKLOADS["tiny"])
    run = gh.GpuRun(hb)
    cb = run.cb
    before = run.event()
    assert run.ctx.device_flags() == 0
    limit = 2_000_000
    rc, flags, waited, followed = cb.cask_selftest_wait_timeout(run.ctx, limit, run.ws, run.ws_bytes)
    assert rc == cb.OK and flags == cb.ST_TIMEOUT
    assert run.ctx.device_flags() == cb.ST_TIMEOUT
    assert limit <= waited < 50 * limit              # gave up after the limit, not after the default second
    assert 0 < followed < 50 * limit                 # the follower left on the abort flag
    # out-of-range limits and a missing workspace are refused on the host
    n0 = run.ctx.launches
    assert cb.cask_selftest_wait_timeout(run.ctx, 10, run.ws, run.ws_bytes, check=False)[0] == cb.ERR_PARAM
    assert cb.cask_selftest_wait_timeout(run.ctx, 10**10, run.ws, run.ws_bytes, check=False)[0] == cb.ERR_PARAM
    assert cb.cask_selftest_wait_timeout(run.ctx, limit, None, 0, check=False)[0] == cb.ERR_WORKSPACE
    assert run.ctx.launches == n0
    # the context and the device carry on: the same event, the same bytes, no flag
    after = run.event()
    assert run.ctx.device_flags() == 0
    for k in before:
        assert np.array_equal(before[k], after[k], equal_nan=True), k
    o = gh.run_oracle(hb)
    gh.compare_event(hb, after, o)
    torch.cuda.synchronize()


@pytest.mark.parametrize("extras", [0, 1, 2])
def test_host_buffer_entry_point_matches_device_entry_point(extras):
    """cask_compress_event_host (host K/V/Q and host outputs; only the value rows that are read go up) gives the
    bytes of the device call, also with carried masses and channel weights (1) or band weights (2) passed as host
    arrays."""
    import gpu_harness as gh
    import torch
    w = _small("reasoning8k_b384", layers=1, kv_heads=2, decode=1000)
    hb = wl.make_batch(w)
    rng = np.random.default_rng(3)
    mass = (np.where(rng.random(int(hb.tok_off[-1])) < 0.3, rng.random(int(hb.tok_off[-1])) * 1e-3, 0.0)
            .astype(np.float32)) if extras else None
    cw = (rng.random(w.head_dim) + 0.05).astype(np.float32) if extras == 1 else None
    bw = (rng.random(w.head_dim // 2) + 0.05).astype(np.float32) if extras == 2 else None
    run = gh.GpuRun(hb, mass_in=mass, chan_w=cw, band_w=bw, band_layout=1)
    g = run.event()
    cb = run.cb
    hbatch, keep = cb.make_batch(hb.k, hb.v, hb.q, hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, w.head_dim, w.group,
                                 w.window, w.dtype, mass_in=mass, chan_w=cw, band_w=bw, band_layout=1)
    nbytes = cb.cask_host_event_device_bytes(hbatch, run.prm, run.Bmax)
    assert nbytes > 0
    dev = torch.empty(nbytes, dtype=torch.uint8, device="cuda:0")
    ho = {k: (np.zeros(tuple(t.shape), np.uint16) if t.dtype == torch.bfloat16 else np.zeros(tuple(t.shape), t.cpu().numpy().dtype))
          for k, t in run.out.items()}
    cb.cask_compress_event_host(run.ctx, hbatch, run.prm, cb.make_outputs(ho, run.Bmax), dev, nbytes)
    for k in g:
        got = wl.bf16_bits_to_f32(ho[k]) if ho[k].dtype == np.uint16 else ho[k]
        assert np.array_equal(got, g[k]), k


@pytest.mark.parametrize("budgets", ["small", "near_full"])
def test_host_buffer_entry_point_in_slices(budgets):
    """A host batch of 60 MB of keys goes through the device in several slices of units (each with its own staging
    and workspace, uploads overlapping the slice before); 44 ragged units with odd lengths, carried masses and
    channel weights, every one against the oracle.  Against the device entry point on the whole batch only the
    last bits of the scores may differ (a unit's tiles are shared out between the CTAs differently).
    "near_full": budgets a few hundred rows short of the cache, so nearly every value row is needed and the pinned
    staging of the context has to grow while earlier slices are in flight."""
    import gpu_harness as gh
    import torch
    rng = np.random.default_rng(11)
    base = wl.WORKLOADS["tiny"].with_(dtype=wl.DTYPE_BF16, head_dim=128, group=2, window=16, cluster_frac=0.6,
                                      n_centres=0)
    ks, vs, qs, T, P, B, R = [], [], [], [], [], [], []
    for i in range(44):
        t = int(rng.integers(4000, 7001))
        p = int(rng.integers(0, 600))
        b = int(rng.integers(64, 385)) if budgets == "small" else t - int(rng.integers(50, 400))
        r = int(rng.integers(0, b + 1)) if budgets == "small" else b // 2
        w = base.with_(prefix=p, decode=t - p, budget=b, reserve=r)
        k, v, q = wl.make_unit(w, i, 5, 0)
        ks.append(k); vs.append(v); qs.append(q[None])
        T.append(t); P.append(p); B.append(b); R.append(r)
    hb = wl.Batch(wl=base, k=np.concatenate(ks), v=np.concatenate(vs), q=np.concatenate(qs),
                  T=np.array(T, np.int32), P=np.array(P, np.int32), B=np.array(B, np.int32),
                  reserve=np.array(R, np.int32), tok_off=np.concatenate([[0], np.cumsum(T)]).astype(np.int64),
                  unit_ids=[(i, 0, 0) for i in range(len(T))])
    sumT = int(hb.tok_off[-1])
    assert sumT * 256 > 3 * (16 << 20)           # enough keys for three slices or more
    mass = np.where(rng.random(sumT) < 0.3, rng.random(sumT) * 1e-3, 0.0).astype(np.float32)
    cw = (rng.random(128) + 0.05).astype(np.float32)
    run = gh.GpuRun(hb, mass_in=mass, chan_w=cw)
    whole = run.event()
    cb = run.cb
    hbatch, keep = cb.make_batch(hb.k, hb.v, hb.q, hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, 128, 2, 16,
                                 wl.DTYPE_BF16, mass_in=mass, chan_w=cw)
    nbytes = cb.cask_host_event_device_bytes(hbatch, run.prm, run.Bmax)
    assert nbytes > 0
    dev = torch.empty(nbytes, dtype=torch.uint8, device="cuda:0")
    ho = {k: (np.zeros(tuple(t.shape), np.uint16) if t.dtype == torch.bfloat16 else np.zeros(tuple(t.shape), t.cpu().numpy().dtype))
          for k, t in run.out.items()}
    assert cb.cask_compress_event_host(run.ctx, hbatch, run.prm, cb.make_outputs(ho, run.Bmax), dev, nbytes - 256,
                                       check=False) == cb.ERR_WORKSPACE
    cb.cask_compress_event_host(run.ctx, hbatch, run.prm, cb.make_outputs(ho, run.Bmax), dev, nbytes)
    assert run.ctx.device_flags() == 0
    g = {k: (wl.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a) for k, a in ho.items()}
    o = gh.run_oracle(hb, mass_in=mass, chan_w=cw)
    st = gh.compare_event(hb, g, o, geom=dict(mass_in=mass, chan_w=cw))
    assert st["units"] == 44
    assert np.allclose(g["s"], whole["s"], rtol=1e-5, atol=1e-12)
    assert np.array_equal(g["plan"], whole["plan"]) and np.array_equal(g["unit_status"], whole["unit_status"])
