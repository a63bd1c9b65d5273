#!/usr/bin/env python
"""Benchmark of the CASK compression event on B200.

One *step* is one whole compression event (score -> prefix eviction -> core
selection -> scratch consolidation -> compaction) over every unit (layer x KV
head) of one sequence of the named workload.  Default workload: the 32k-token
reasoning decode shape at budget 512 (36 layers x 8 KV heads, 33,280 rows per
unit, bf16, 4.9 GB of K/V), the shape the roofline target is quoted on.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
    python bench.py --impl reference ...        # the CPU oracle, timed as it stands

Multi-GPU: units are independent, so each rank runs the event on its own
sequence (weak scaling, no data-path collective); only the timing barrier and
the max over ranks use torch.distributed.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_10900_b200 import workloads as wl  # noqa: E402

METRIC = "kv_tokens_compressed_per_s"
UNIT = "tokens/s"

# DRAM bytes per cache row (dram__bytes_read.sum + dram__bytes_write.sum of one launch / rows streamed) from the
# ncu captures summarised under profiles/; traffic grows in proportion to the rows a launch streams.
NCU_TRAFFIC = {
    "score_norm": (268.0, "profiles/score_tc_reasoning32k_16units.txt"),
    "score_mass": (274.2, "profiles/score_tc_reasoning32k_16units.txt"),
    "assign": (264.9, "profiles/assign_tc_reasoning32k_16units.txt"),
}
# ex2 units: 16 results per clock per SM (special-function pipe), 148 SMs, 1.965 GHz maximum SM clock.
EX2_PEAK_T_PER_S = 148 * 16 * 1.965e9 / 1e12


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if ts < t0 - 0.05 or ts > t1 + 0.15:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:   # region shorter than one sample: fall back to everything seen
            for ts, line in self.lines:
                f = [x.strip() for x in line.split(",")]
                try:
                    sm.append(float(f[0])); mx.append(float(f[1]))
                except (ValueError, IndexError):
                    pass
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def _dist():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def algorithmic_bytes(hb: wl.Batch, n_out: np.ndarray, kind: np.ndarray) -> int:
    """Bytes the event must move: K once, Q, K and V of every contributing row (kept or merged),
    the compacted K/V written, and the per-row / per-slot index maps."""
    w = hb.wl
    e = 2 if w.dtype == wl.DTYPE_BF16 else 4
    d = w.head_dim
    sum_T = int(hb.T.sum())
    contributing = int(np.count_nonzero(kind != 0))
    rows = w.group * w.window
    return (sum_T * d * e + hb.n_units * rows * d * e + 2 * contributing * d * e
            + 2 * int(n_out.sum()) * d * e + 8 * sum_T + 12 * int(hb.B.sum()))


def run_ours(args):
    import torch
    from paper_2604_10900_b200 import binding as cb

    world, rank, local = _dist()
    if args.gpus != world:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torch.distributed.run for --gpus > 1")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))
    w = wl.WORKLOADS[args.workload]
    # A batch of many sequences does not fit one GPU with all its layers (64 sequences x 36 layers x 8 heads of
    # the serving sweep hold 179 GB of K/V): it runs on a slice of the layers, every sequence present.
    n_layers = min(w.layers, args.layer_slice or w.layers_per_pass or w.layers)
    units = wl.unit_list(w, seqs=range(rank, rank + 1)) if w.n_seqs == 1 else \
        wl.shard_units(wl.unit_list(w, layers=range(n_layers)), rank, world)
    if args.max_units:
        units = units[:args.max_units]

    def pinned(shape, dt):
        t = torch.empty(tuple(shape), dtype={np.dtype(np.uint16): torch.uint16, np.dtype(np.float32): torch.float32,
                                             np.dtype(np.int32): torch.int32, np.dtype(np.uint8): torch.uint8}[np.dtype(dt)],
                        pin_memory=True)
        return t.numpy()

    t_gen = time.time()
    hb = wl.make_batch(w, units, threads=min(16, os.cpu_count() or 8), pinned_alloc=pinned)
    t_gen = time.time() - t_gen
    sum_T = int(hb.tok_off[-1])
    d, rows = w.head_dim, w.group * w.window

    dev = cb.to_device(hb, device)
    mass_dev = None if hb.mass_in is None else torch.from_numpy(hb.mass_in).to(device)
    # merge similarity (Sec. 2.5): plain cosine, or synthetic weights |kappa| that fall off with the band index
    chan_host, band_host = similarity_weights(args.similarity, d)
    sim_dev = dict(chan_w=None if chan_host is None else torch.from_numpy(chan_host).to(device),
                   band_w=None if band_host is None else torch.from_numpy(band_host).to(device))
    sim_host = dict(chan_w=chan_host, band_w=band_host)
    batch, keep = cb.make_batch(dev["k"], dev["v"], dev["q"], hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, d, w.group,
                                w.window, w.dtype, mass_in=mass_dev, **sim_dev)
    prm = cb.params(score_path=args.score_path)
    stream = torch.cuda.current_stream(device)
    ctx = cb.Context(local, stream.cuda_stream)
    ws, ws_bytes = cb.alloc_workspace(batch, prm, device)
    Bmax = int(hb.B.max())
    out = cb.alloc_outputs(hb.n_units, sum_T, Bmax, d, rows, w.dtype, device, optional=False)
    out["lse"] = torch.zeros((hb.n_units, rows), dtype=torch.float32, device=device)   # normalisers used
    out_struct = cb.make_outputs(out, Bmax)

    def step():
        cb.cask_compress_event(ctx, batch, prm, out_struct, ws, ws_bytes)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    n_out = out["n_out"].cpu().numpy()
    kind = out["kind"].cpu().numpy()
    status = out["unit_status"].cpu().numpy()
    assert (n_out == np.minimum(hb.B, hb.T)).all() or (n_out <= hb.B).all()

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    ctx.profile_enable(True)
    ctx.profile_read()
    l0 = ctx.launches
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    t1 = time.time()
    ms_total = ev0.elapsed_time(ev1)
    launches = ctx.launches - l0
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    clocks = sampler.stop(t0, t1)

    # The same event when the caller hands over the window queries' softmax normalisers (a decode attention
    # kernel has them): the normaliser pass is skipped.  Reported beside the headline, never instead of it.
    batch_l, keep_l = cb.make_batch(dev["k"], dev["v"], dev["q"], hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, d, w.group,
                                    w.window, w.dtype, lse_in=out["lse"].clone(), mass_in=mass_dev, **sim_dev)
    cb.cask_compress_event(ctx, batch_l, prm, out_struct, ws, ws_bytes)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        cb.cask_compress_event(ctx, batch_l, prm, out_struct, ws, ws_bytes)
    ev1.record(stream)
    barrier()
    ms_lse = ev0.elapsed_time(ev1) / args.steps
    assert (out["n_out"].cpu().numpy() == n_out).all()

    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms_total], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
        tok = torch.tensor([float(sum_T)], device=device, dtype=torch.float64)
        dist.all_reduce(tok, op=dist.ReduceOp.SUM)
        total_tokens = float(tok.item())
    else:
        total_tokens = float(sum_T)
    ms_step = ms_total / args.steps
    value = total_tokens / (ms_step * 1e-3)

    # ---- end to end through the host-buffer entry point ---------------------------------------
    hbatch, hkeep = cb.make_batch(hb.k, hb.v, hb.q, hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, d, w.group, w.window,
                                  w.dtype, mass_in=hb.mass_in, **sim_host)
    dev_bytes = cb.cask_host_event_device_bytes(hbatch, prm, Bmax)
    del dev, out, out_struct, ws
    torch.cuda.empty_cache()
    dev_buf = torch.empty(dev_bytes, dtype=torch.uint8, device=device)
    e = 2 if w.dtype == wl.DTYPE_BF16 else 4
    st = np.uint16 if w.dtype == wl.DTYPE_BF16 else np.float32
    # every result lands in pinned memory: a copy into pageable memory would hold the host until it is done
    ho = dict(k_out=pinned((hb.n_units, Bmax, d), st), v_out=pinned((hb.n_units, Bmax, d), st),
              n_out=pinned((hb.n_units,), np.int32), slot_src=pinned((hb.n_units, Bmax), np.int32),
              slot_kind=pinned((hb.n_units, Bmax), np.uint8), slot_mass=pinned((hb.n_units, Bmax), np.float32),
              assign=pinned((sum_T,), np.int32), weight=pinned((sum_T,), np.float32),
              kind=pinned((sum_T,), np.uint8), seed_of=pinned((sum_T,), np.int32),
              plan=pinned((hb.n_units, 8), np.int32), unit_status=pinned((hb.n_units,), np.int32),
              lost_mass=pinned((hb.n_units,), np.float32))
    for a in ho.values():
        a[...] = 0
    ho_struct = cb.make_outputs(ho, Bmax)
    # The host entry point sends the keys and queries whole but only the value rows that are kept or merged
    # (counted from the row kinds of the device run); the row kinds come back once more in mid-call.
    h2d = hb.k.nbytes + hb.q.nbytes + int(np.count_nonzero(kind)) * d * (2 if w.dtype == wl.DTYPE_BF16 else 4) \
        + (0 if hb.mass_in is None else hb.mass_in.nbytes)
    d2h = sum(a.nbytes for a in ho.values()) + sum_T
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    cb.cask_compress_event_host(ctx, hbatch, prm, ho_struct, dev_buf, dev_bytes)   # warm-up
    barrier()
    ev0.record(stream)
    for _ in range(e2e_steps):
        cb.cask_compress_event_host(ctx, hbatch, prm, ho_struct, dev_buf, dev_bytes)
    ev1.record(stream)
    barrier()
    e2e_ms = ev0.elapsed_time(ev1) / e2e_steps
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([e2e_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    assert (ho["n_out"] == n_out).all()
    e2e_value = total_tokens / (e2e_ms * 1e-3)

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel -------------------------------------------------------
    ctx_tensor_path = ctx.used_tensor_path
    peaks = _peaks()
    per_kernel = {k: dict(ms_per_launch=v["ms"] / v["launches"], launches_per_step=v["launches"] / args.steps,
                          share=v["ms"] / max(sum(x["ms"] for x in prof.values()), 1e-9)) for k, v in prof.items()}
    top = max(prof, key=lambda k: prof[k]["ms"])
    top_ms = prof[top]["ms"] / prof[top]["launches"]
    flops_pass = 2.0 * rows * float(sum_T) * d        # one Q_w K^T contraction over every unit
    tensor_roof = None
    if top in ("score_norm", "score_mass"):
        # One exponential per (query row, key): the pass is bound by the ex2 pipe, not by the contraction that
        # feeds it (profiles/score_tc_*: ex2 pipe 65-72 % busy, tensor pipe 37-40 %, DRAM 17 %).
        exps = float(rows) * float(sum_T)
        achieved = exps / (top_ms * 1e-3) / 1e12
        roof = dict(kernel=top, bound="alu", achieved=achieved, peak=EX2_PEAK_T_PER_S, unit="Texp/s",
                    frac=achieved / EX2_PEAK_T_PER_S, traffic=None,
                    peak_source="148 SMs x 16 ex2/clk x 1.965 GHz", ms_per_launch=top_ms, exps_per_launch=exps)
        t_ach = flops_pass / (top_ms * 1e-3) / 1e12
        tensor_roof = dict(kernel=top, bound="tensor", achieved=t_ach, peak=peaks["bf16_tflops_sustained"],
                           unit="TFLOP/s", frac=t_ach / peaks["bf16_tflops_sustained"],
                           peak_source=peaks["source"] + " (sustained cuBLAS bf16)", flops_per_launch=flops_pass)
    else:
        byts = algorithmic_bytes(hb, n_out, kind)
        achieved = byts / (top_ms * 1e-3) / 1e9
        roof = dict(kernel=top, bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], traffic=None, peak_source=peaks["source"], ms_per_launch=top_ms)
    if top in NCU_TRAFFIC and ctx_tensor_path:
        roof["traffic"] = NCU_TRAFFIC[top][0] * float(sum_T)
        roof["traffic_source"] = NCU_TRAFFIC[top][1] + " (bytes per cache row x rows of this launch)"
    ev_bytes = algorithmic_bytes(hb, n_out, kind)
    t_hbm = ev_bytes / (peaks["hbm_gbs"] * 1e9)
    n_pass = 2          # normaliser pass + score pass (no caller-supplied normalisers here)
    t_tensor = n_pass * flops_pass / (peaks["bf16_tflops_sustained"] * 1e12)
    event = dict(algorithmic_bytes=ev_bytes, gbs=ev_bytes / (ms_step * 1e-3) / 1e9,
                 hbm_frac_measured_peak=ev_bytes / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
                 hbm_frac_nominal_8tbs=ev_bytes / (ms_step * 1e-3) / 1e9 / 8000.0,
                 composite_floor_ms=max(t_hbm, t_tensor) * 1e3,
                 composite_frac=max(t_hbm, t_tensor) * 1e3 / ms_step)

    # ---- the oracle on this machine's host cores, bounded sample ------------------------------------
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w, args.cpu_units, args.similarity)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak" if w.n_seqs == 1 else "strong", "vs_baseline": None, "dtype": "bf16" if w.dtype == wl.DTYPE_BF16 else "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "units_per_gpu": hb.n_units, "rows_per_unit": int(hb.T.max()), "head_dim": d,
                   "query_rows": rows, "budget": int(hb.B.max()), "tokens_per_step": total_tokens,
                   "l2": "inputs larger than L2: %.2f GB of K/V read per step" % ((hb.k.nbytes + hb.v.nbytes) / 1e9),
                   "score_path": "tcgen05" if ctx.used_tensor_path else "simt", "gen_seconds": round(t_gen, 1),
                   "reduced": bool(args.max_units),
                   **({"sequences": w.n_seqs, "layers_per_pass": n_layers, "layers": w.layers,
                       "events_per_s": w.n_seqs * n_layers / w.layers / (ms_step * 1e-3),
                       "events_per_s_note": "one event = all layers of one sequence; this pass held layers_per_pass of them"}
                      if w.n_seqs > 1 else {}),
                   **({"carried_mass_rows": w.carried_rows} if w.carried_rows else {}),
                   "similarity": args.similarity,
                   "status_bits_seen": int(np.bitwise_or.reduce(status))},
        "with_supplied_normalisers": {"ms_per_step": ms_lse, "value": total_tokens / (ms_lse * 1e-3), "unit": UNIT,
                                      "note": "lse_in given by the caller: one scoring pass instead of two (this rank)"},
        "roofline": roof, "tensor_roofline": tensor_roof, "event_roofline": event, "kernels": per_kernel,
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": e2e_ms, "steps": e2e_steps},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def similarity_weights(kind: str, d: int):
    """(chan_w [d], band_w [d/2]) for --similarity: None for the cosine; |kappa|-like weights 1 / (1 + f/8) on band
    f = channels (f, f + d/2) otherwise, per channel (inner-product form) or per band (distance form)."""
    if kind == "cosine":
        return None, None
    bw = (1.0 / (1.0 + np.arange(d // 2) / 8.0)).astype(np.float32)
    if kind == "channel":
        return np.concatenate([bw, bw]).astype(np.float32), None
    return None, bw


def cpu_baseline(w: wl.Workload, n_units: int, similarity: str = "cosine"):
    """The oracle, as it stands, on a bounded sample: the first `n_units` units of the workload."""
    from oracle import cask_oracle as orc
    n_units = n_units or max(1, min(w.n_units, (96 * 33280) // (w.prefix + w.decode)))
    units = wl.unit_list(w)[:n_units]
    hb = wl.make_batch(w, units)
    kf, vf, qf = (wl.as_float32(x, w.dtype) for x in (hb.k, hb.v, hb.q))
    orc.lib()
    t = time.time()
    cw, bw = similarity_weights(similarity, w.head_dim)
    orc.event_batch(kf, vf, qf, hb.tok_off, hb.P, hb.B, hb.reserve, mass_in=hb.mass_in, chan_w=cw, band_w=bw)
    dt = time.time() - t
    return {"value": float(hb.T.sum()) / dt, "unit": UNIT, "cores": orc.threads(), "kind": "oracle",
            "sample": f"{len(units)} of {w.n_units} units of {w.name} (whole event, fp64), {dt:.1f} s",
            "seconds": dt}


def run_reference(args):
    """The CPU oracle timed as the reference arm: each step is the event on a bounded sample."""
    world, rank, local = _dist()
    if rank != 0:
        return
    from oracle import cask_oracle as orc
    w = wl.WORKLOADS[args.workload]
    n_units = min(args.cpu_units, 16) if args.cpu_units else max(1, min(w.n_units, (16 * 33280) // (w.prefix + w.decode)))
    units = wl.unit_list(w)[:n_units]
    hb = wl.make_batch(w, units)
    kf, vf, qf = (wl.as_float32(x, w.dtype) for x in (hb.k, hb.v, hb.q))
    orc.lib()

    def step():
        orc.event_batch(kf, vf, qf, hb.tok_off, hb.P, hb.B, hb.reserve, mass_in=hb.mass_in, chan_w=cw, band_w=bw)

    cw, bw = similarity_weights(args.similarity, w.head_dim)
    for _ in range(args.warmup):
        step()
    t = time.time()
    for _ in range(args.steps):
        step()
    dt = (time.time() - t) / args.steps
    value = float(hb.T.sum()) / dt
    sample = f"{len(units)} of {w.n_units} units of {w.name} per step (whole event, fp64 oracle)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "units_per_step": len(units), "rows_per_unit": int(hb.T.max())},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_stats_scorer(args):
    """Times the query-statistics scorer (App. B) alone: one pass over the keys, reported against HBM bandwidth."""
    import torch
    from paper_2604_10900_b200 import binding as cb
    world, rank, local = _dist()
    if rank != 0:
        return
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    w = wl.WORKLOADS[args.workload]
    n_layers = min(w.layers, args.layer_slice or w.layers_per_pass or w.layers)
    units = wl.unit_list(w, layers=range(n_layers))
    if args.max_units:
        units = units[:args.max_units]
    hb = wl.make_batch(w, units, threads=min(16, os.cpu_count() or 8))
    d, nb, sum_T = w.head_dim, w.head_dim // 2, int(hb.tok_off[-1])
    dev = cb.to_device(hb, device)
    batch, keep = cb.make_batch(dev["k"], dev["v"], dev["q"], hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, d, w.group,
                                w.window, w.dtype)
    prm = cb.params()
    stream = torch.cuda.current_stream(device)
    ctx = cb.Context(local, stream.cuda_stream)
    ws, ws_bytes = cb.alloc_workspace(batch, prm, device)
    rng = np.random.default_rng(2604)
    n_delta = 64
    mu = torch.from_numpy(rng.standard_normal((hb.n_units, w.group, nb, 2)).astype(np.float32)).to(device)
    pi = rng.random((hb.n_units, w.group, n_delta)).astype(np.float32)
    pi = torch.from_numpy(pi / pi.sum(-1, keepdims=True)).to(device)
    grid = torch.arange(n_delta, dtype=torch.float32, device=device) * 16.0
    omega = torch.from_numpy((1.0 / (10000.0 ** (np.arange(nb) / nb))).astype(np.float32)).to(device)
    # "stats_offsets": every row brings its own (fractional, signed) offset instead of Delta_i = T - 1 - i
    offsets = args.scorer == "stats_offsets"
    delta = (torch.rand(sum_T, dtype=torch.float32, device=device) * 45000.0 - 5000.0) if offsets else None
    qs, keep2 = cb.make_query_stats(mu, pi, grid, omega, 0, delta)
    s = torch.empty(sum_T, dtype=torch.float32, device=device)
    for _ in range(max(args.warmup, 3)):
        cb.cask_score_stats(ctx, batch, prm, qs, s, ws, ws_bytes)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        cb.cask_score_stats(ctx, batch, prm, qs, s, ws, ws_bytes)
    ev1.record(stream)
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    peaks = _peaks()
    byts = hb.k.nbytes + 4 * sum_T * (2 if offsets else 1)
    gbs = byts / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "kv_tokens_scored_per_s", "value": sum_T / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "dtype": "bf16" if w.dtype == wl.DTYPE_BF16 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "scorer": "query statistics (horizon kernel, mean score)" + (", caller offsets" if offsets else ""), "units": hb.n_units,
                   "rows_per_unit": int(hb.T.max()), "n_delta": n_delta,
                   "l2": "inputs larger than L2: %.2f GB of K read per step" % (hb.k.nbytes / 1e9)},
        "roofline": {"kernel": "score_stats_kernel", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                     # bytes per cache row from the ncu capture of this kernel on a 16-unit slice x the rows of this
                     # launch; the kernel for caller offsets has no capture
                     "traffic": None if offsets else 268.5 * sum_T, "peak_source": peaks["source"],
                     "traffic_source": None if offsets else "profiles/score_stats_reasoning32k_16units.txt"},
        "gpu_launches": 2 * args.steps}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="reasoning32k_b512", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--score-path", type=int, default=0, help="0: tensor-core scoring when the shape allows, 1: SIMT")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--scorer", default="attention", choices=["attention", "stats", "stats_offsets"],
                    help="attention: the whole event with the windowed attention-mass score (default); "
                         "stats: time the query-statistics scorer of App. B alone")
    ap.add_argument("--similarity", default="cosine", choices=["cosine", "channel", "band"],
                    help="merge similarity: cosine, channel-weighted inner product, or per-band distance (Sec. 2.5)")
    ap.add_argument("--cpu-units", type=int, default=0,
                    help="units in the oracle's bounded sample (default: about three million cache rows, 10 s of CPU work)")
    ap.add_argument("--max-units", type=int, default=0, help="debug: cut the workload to this many units")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layer-slice", type=int, default=0,
                    help="layers per pass for multi-sequence workloads (default 6)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.scorer in ("stats", "stats_offsets"):
        run_stats_scorer(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
