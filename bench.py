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
    "score_norm": (269.4, "profiles/score_tc_reasoning32k_16units.txt"),
    "score_mass": (272.8, "profiles/score_tc_reasoning32k_16units.txt"),
    "assign": (264.4, "profiles/assign_tc_reasoning32k_16units.txt"),
}


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
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
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


def sm_count(device) -> int:
    import torch
    return int(torch.cuda.get_device_properties(device).multi_processor_count)


def ex2_peak(sms: int, clocks: dict) -> tuple:
    """Roof of the exponential pipe in T exp/s: 16 results per clock per SM (special-function unit) x SMs x the
    maximum SM clock nvidia-smi reports (1.965 GHz when it could not be read)."""
    mhz = clocks.get("sm_max_mhz") or 1965.0
    return sms * 16 * mhz * 1e6 / 1e12, "%d SMs x 16 ex2/clk x %.3f GHz" % (sms, mhz / 1e3)


class Event:
    """One workload resident on the device with everything a compression event needs."""

    def __init__(self, w, units, args, device, local, similarity="cosine", shared=None, pinned=None):
        import torch
        from paper_2604_10900_b200 import binding as cb
        self.cb, self.torch, self.w, self.device = cb, torch, w, device
        t_gen = time.time()
        if shared is not None:       # same rows as an earlier workload, other budget
            hb0 = shared.hb
            n = hb0.n_units
            self.hb = hb = wl.Batch(wl=w, k=hb0.k, v=hb0.v, q=hb0.q, T=hb0.T, P=hb0.P, B=np.full(n, w.budget, np.int32),
                                    reserve=np.full(n, w.reserve, np.int32), tok_off=hb0.tok_off, unit_ids=hb0.unit_ids,
                                    mass_in=hb0.mass_in)
            self.dev = shared.dev
        else:
            self.hb = hb = wl.make_batch(w, units, threads=min(16, os.cpu_count() or 8), pinned_alloc=pinned)
            self.dev = cb.to_device(hb, device)
        self.t_gen = time.time() - t_gen
        self.sum_T = int(hb.tok_off[-1])
        d, rows = w.head_dim, w.group * w.window
        self.d, self.rows = d, rows
        self.mass_dev = None if hb.mass_in is None else torch.from_numpy(hb.mass_in).to(device)
        chan_host, band_host = similarity_weights(similarity, d)
        self.sim_host = dict(chan_w=chan_host, band_w=band_host)
        self.sim_dev = dict(chan_w=None if chan_host is None else torch.from_numpy(chan_host).to(device),
                            band_w=None if band_host is None else torch.from_numpy(band_host).to(device))
        self.batch, self._keep = cb.make_batch(self.dev["k"], self.dev["v"], self.dev["q"], hb.T, hb.P, hb.B, hb.reserve,
                                               hb.tok_off, d, w.group, w.window, w.dtype, mass_in=self.mass_dev,
                                               **self.sim_dev)
        self.prm = cb.params(score_path=args.score_path)
        self.stream = torch.cuda.current_stream(device)
        self.ctx = cb.Context(local, self.stream.cuda_stream)
        self.ws, self.ws_bytes = cb.alloc_workspace(self.batch, self.prm, device)
        self.Bmax = int(hb.B.max())
        self.out = cb.alloc_outputs(hb.n_units, self.sum_T, self.Bmax, d, rows, w.dtype, device, optional=False)
        self.out["lse"] = torch.zeros((hb.n_units, rows), dtype=torch.float32, device=device)   # normalisers used
        self.out_struct = cb.make_outputs(self.out, self.Bmax)

    def step(self, batch=None):
        self.cb.cask_compress_event(self.ctx, batch if batch is not None else self.batch, self.prm, self.out_struct,
                                    self.ws, self.ws_bytes)

    def time_steps(self, steps, barrier, batch=None):
        """Times `steps` events back to back on the stream.  Returns (total ms over all steps, per-step ms list):
        one CUDA event before the first step and one after every step, all on the launching stream, so the total
        is the bracketed time of exactly `steps` steps and the list gives the median and the best."""
        torch = self.torch
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        evs[0].record(self.stream)
        for i in range(steps):
            self.step(batch)
            evs[i + 1].record(self.stream)
        barrier()
        return evs[0].elapsed_time(evs[-1]), [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]

    def kernel_split(self, steps):
        """Per-kernel times from a loop of its own, with an event pair around every launch."""
        self.ctx.profile_enable(True)
        self.ctx.profile_read()
        for _ in range(steps):
            self.step()
        self.torch.cuda.synchronize()
        prof = self.ctx.profile_read()
        self.ctx.profile_enable(False)
        tot = max(sum(x["ms"] for x in prof.values()), 1e-9)
        return {k: dict(ms_per_launch=v["ms"] / v["launches"], launches_per_step=v["launches"] / steps,
                        share=v["ms"] / tot) for k, v in prof.items()}

    def results(self):
        return (self.out["n_out"].cpu().numpy(), self.out["kind"].cpu().numpy(), self.out["unit_status"].cpu().numpy())


def event_roofline(hb, n_out, kind, ms_step, peaks, n_pass=2):
    """The whole event against the HBM roof (algorithmic bytes of the event over its time) and against the composite
    floor max(bytes / bandwidth, scoring flops / tensor peak)."""
    w = hb.wl
    rows, d, sum_T = w.group * w.window, w.head_dim, float(hb.T.sum())
    ev_bytes = algorithmic_bytes(hb, n_out, kind)
    flops_pass = 2.0 * rows * sum_T * d
    t_hbm = ev_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tensor = n_pass * flops_pass / (peaks["bf16_tflops_sustained"] * 1e12)
    gbs = ev_bytes / (ms_step * 1e-3) / 1e9
    return dict(algorithmic_bytes=ev_bytes, gbs=gbs, hbm_frac_measured_peak=gbs / peaks["hbm_gbs"],
                hbm_frac_nominal_8tbs=gbs / 8000.0, composite_floor_ms=max(t_hbm, t_tensor) * 1e3,
                composite_frac=max(t_hbm, t_tensor) * 1e3 / ms_step)


# The other configurations of the benchmark family, timed after the headline on one GPU: the 8k reasoning shape at
# both budgets, the 32k shape at the other two budgets (same rows as the headline), the prompt-heavy two-stage shape
# and its variant at the exhaustion boundary, one layer of the 64-sequence serving sweep, and the sweep's steady state.
OTHER_WORKLOADS = ("reasoning32k_b384", "reasoning32k_b1024", "reasoning8k_b384", "reasoning8k_b512", "prompt_heavy",
                   "prompt_heavy_boundary", "batched_serving", "serving_steady_b512")


def other_workloads(args, device, local, peaks, headline: "Event"):
    import torch
    out = {}
    steps = max(20, args.steps)

    def barrier():
        torch.cuda.synchronize()

    for name in OTHER_WORKLOADS:
        w = wl.WORKLOADS[name]
        n_layers = w.layers
        if name == "batched_serving":
            n_layers = 1                      # one layer of every sequence: 512 ragged units
        elif name == "serving_steady_b512":
            n_layers = 12                     # a third of the layers of every sequence: 6,144 caches of 640 rows
        units = wl.unit_list(w, layers=range(n_layers)) if w.n_seqs > 1 else None
        shared = headline if (w.cfg_id == headline.w.cfg_id and w.n_seqs == 1 and w.prefix == headline.w.prefix
                              and w.decode == headline.w.decode and not args.max_units) else None
        ev = Event(w, units, args, device, local, shared=shared)
        for _ in range(3):
            ev.step()
        barrier()
        total, per = ev.time_steps(steps, barrier)
        n_out, kind, status = ev.results()
        kern = ev.kernel_split(5)
        top = max(kern, key=lambda k: kern[k]["ms_per_launch"] * kern[k]["launches_per_step"])
        med, best = float(np.median(per)), float(min(per))
        hb = ev.hb
        tokens = float(ev.sum_T)
        rec = dict(units=hb.n_units, rows_per_unit=[int(hb.T.min()), int(hb.T.max())], budget=int(hb.B.max()),
                   steps=steps, ms_per_step=total / steps, ms_per_step_median=med, ms_per_step_best=best,
                   value=tokens / (total / steps * 1e-3), unit=UNIT, tokens_per_step=tokens,
                   event_roofline=event_roofline(hb, n_out, kind, med, peaks), dominant_kernel=top,
                   dominant_kernel_ms=kern[top]["ms_per_launch"] * kern[top]["launches_per_step"],
                   kernels={k: round(v["ms_per_launch"] * v["launches_per_step"], 5) for k, v in kern.items()},
                   score_path="tcgen05" if ev.ctx.used_tensor_path else "simt",
                   score_pass_sm_mhz=list(ev.ctx.score_clock_mhz()),
                   status_bits_seen=int(np.bitwise_or.reduce(status)),
                   l2="inputs larger than L2: %.2f GB of K/V read per step" % ((hb.k.nbytes + hb.v.nbytes) / 1e9))
        if w.n_seqs > 1:
            rec.update(sequences=w.n_seqs, layers_in_this_pass=n_layers, layers=w.layers,
                       events_per_s=w.n_seqs * n_layers / w.layers / (med * 1e-3),
                       events_per_s_note="one event = all layers of one sequence; this pass held layers_in_this_pass of them")
        out[name] = rec
        del ev
        torch.cuda.empty_cache()
    return out


def trigger_loop(args, device, local, peaks, n_events=12, n_layers=12):
    """The serving sweep's trigger loop on real previous outputs: every cache of 640 rows is compressed to 512, the
    512 compacted rows (representatives carrying the group mass the event gave them) plus 128 newly appended decode
    rows are the next event's cache, n_events times over.  The appended rows stand in for 128 decode steps: half of
    them near-duplicates of kept decode rows, half fresh; building them is device-side plumbing between the events
    and is timed with the loop, not with the events."""
    import torch
    w = wl.WORKLOADS["serving_steady_b512"]
    ev = Event(w, wl.unit_list(w, layers=range(n_layers)), args, device, local)
    hb, d, cb = ev.hb, ev.d, ev.cb
    n, T, B, P = hb.n_units, int(hb.T.max()), w.budget, w.prefix
    assert int(hb.T.min()) == T and T == B + 128
    k3, v3 = ev.dev["k"].view(n, T, d), ev.dev["v"].view(n, T, d)
    mass = ev.mass_dev.view(n, T)
    scale = torch.from_numpy(np.stack([wl.channel_scale(w, s_, l_) for (s_, l_, _) in hb.unit_ids])).to(device)   # [n, d]
    gen = torch.Generator(device=device)
    gen.manual_seed(2604)
    for _ in range(3):
        ev.step()
    torch.cuda.synchronize()
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_events)]
    t_all0, t_all1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    merged_rows = []
    t_all0.record(ev.stream)
    for it in range(n_events):
        pairs[it][0].record(ev.stream)
        ev.step()
        pairs[it][1].record(ev.stream)
        # the next cache: compacted rows, then 128 appended rows; representatives keep their group mass
        out = ev.out
        k3[:, :B] = out["k_out"]
        v3[:, :B] = out["v_out"]
        src = torch.randint(P, B, (n, 64), device=device, generator=gen)
        near = torch.gather(out["k_out"], 1, src[:, :, None].expand(n, 64, d)).float()
        near = near + 0.05 * scale[:, None, :] * torch.randn((n, 64, d), device=device, generator=gen)
        k3[:, B:B + 64] = near.to(k3.dtype)
        k3[:, B + 64:] = (torch.randn((n, 64, d), device=device, generator=gen) * scale[:, None, :]).to(k3.dtype)
        v3[:, B:] = torch.randn((n, 128, d), device=device, generator=gen).to(v3.dtype)
        mass[:, :B] = torch.where(out["slot_kind"] == 4, out["slot_mass"], torch.zeros_like(out["slot_mass"]))
        mass[:, B:] = 0
        merged_rows.append(out["kind"].eq(5).sum())
    t_all1.record(ev.stream)
    torch.cuda.synchronize()
    per = [a.elapsed_time(b) for a, b in pairs]
    status = ev.out["unit_status"].cpu().numpy()
    assert (ev.out["n_out"].cpu().numpy() == B).all() and ev.ctx.device_flags() == 0
    med = float(np.median(per))
    return dict(units=n, rows_per_unit=T, budget=B, events_timed=n_events, ms_per_event_median=med,
                ms_per_event_best=float(min(per)), ms_per_event_first=per[0], ms_per_event_last=per[-1],
                ms_per_iteration_with_cache_rebuild=t_all0.elapsed_time(t_all1) / n_events,
                value=float(ev.sum_T) / (med * 1e-3), unit=UNIT, sequences=w.n_seqs, layers_in_this_pass=n_layers,
                layers=w.layers, events_per_s=w.n_seqs * n_layers / w.layers / (med * 1e-3),
                merged_rows_per_event=[int(x.item()) for x in merged_rows],
                status_bits_seen=int(np.bitwise_or.reduce(status)),
                note="every event after the first runs on the previous event's own output plus 128 appended rows")


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

    ev = Event(w, units, args, device, local, similarity=args.similarity, pinned=pinned)
    hb, ctx, stream = ev.hb, ev.ctx, ev.stream
    sum_T, d, rows, Bmax = ev.sum_T, ev.d, ev.rows, ev.Bmax
    t_gen = ev.t_gen

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    warm = max(args.warmup, 3)
    ev.step()
    barrier()
    n_out, kind, status = ev.results()
    assert (n_out == np.minimum(hb.B, hb.T)).all() or (n_out <= hb.B).all()

    # ---- the timed region: exactly `steps` events, no per-kernel events inside ----------------------------------
    # The clock sampler needs a moment to start; the warm-up steps come after that pause and straight before the timed
    # ones, so the timed region does not begin on a GPU that has just sat idle.
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    for _ in range(warm):
        ev.step()
    l0 = ctx.launches
    t0 = time.time()
    ms_total, per_step = ev.time_steps(args.steps, barrier)
    t1 = time.time()
    launches = ctx.launches - l0
    clocks = sampler.stop(t0, t1)
    # The same event under sustained load: the passes draw enough power for the board's limit to pull the SM clock down
    # after some tens of milliseconds (the first ten events or so run at the burst clock); a long loop shows the level
    # it settles at.  Reported beside the headline, which stays the bracketed time of exactly `steps` steps.
    sustained = None
    if world == 1 and args.sustained_steps > 0:
        _tot, per_s = ev.time_steps(args.sustained_steps, barrier)
        tail_n = max(1, args.sustained_steps // 4)
        sustained = dict(steps=args.sustained_steps, ms_per_step_mean=_tot / args.sustained_steps,
                         ms_per_step_first8_median=float(np.median(per_s[:8])),
                         ms_per_step_last_quarter_median=float(np.median(per_s[-tail_n:])),
                         score_pass_sm_mhz_last=list(ctx.score_clock_mhz()))
        time.sleep(1.0)
    # per-kernel split: a second loop with an event pair around every launch
    per_kernel = ev.kernel_split(min(args.steps, 10))
    score_mhz = ctx.score_clock_mhz()      # SM clock the two scoring passes of the last event ran at

    # The same event when the caller hands over the window queries' softmax normalisers (a decode attention
    # kernel has them): the normaliser pass is skipped.  Reported beside the headline, never instead of it.
    batch_l, keep_l = cb.make_batch(ev.dev["k"], ev.dev["v"], ev.dev["q"], hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, d,
                                    w.group, w.window, w.dtype, lse_in=ev.out["lse"].clone(), mass_in=ev.mass_dev,
                                    **ev.sim_dev)
    ev.step(batch_l)
    ms_lse_total, _ = ev.time_steps(args.steps, barrier, batch_l)
    ms_lse = ms_lse_total / args.steps
    assert (ev.out["n_out"].cpu().numpy() == n_out).all()

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

    ctx_tensor_path = ctx.used_tensor_path      # of the last event (the self-test below is a call of its own)
    # what the special-function unit sustains on this GPU, measured by the library's own loop
    ex2_rate = cb.cask_selftest_exp_rate(ctx, 4096, ev.ws, ev.ws_bytes) if ev.ws_bytes >= 16384 else None
    peaks = _peaks()
    others = None
    if world == 1 and not args.no_other_workloads and args.workload == "reasoning32k_b512" and \
            args.similarity == "cosine" and not args.max_units:
        others = other_workloads(args, device, local, peaks, ev)
        others["serving_trigger_loop"] = trigger_loop(args, device, local, peaks)

    # ---- end to end through the host-buffer entry point ---------------------------------------
    prm = ev.prm
    hbatch, hkeep = cb.make_batch(hb.k, hb.v, hb.q, hb.T, hb.P, hb.B, hb.reserve, hb.tok_off, d, w.group, w.window,
                                  w.dtype, mass_in=hb.mass_in, **ev.sim_host)
    dev_bytes = cb.cask_host_event_device_bytes(hbatch, prm, Bmax)
    ev.dev = ev.out = ev.out_struct = ev.ws = ev.batch = None
    del batch_l, keep_l
    torch.cuda.empty_cache()
    dev_buf = torch.empty(dev_bytes, dtype=torch.uint8, device=device)
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
    e2e_steps = max(1, args.e2e_steps)
    cb.cask_compress_event_host(ctx, hbatch, prm, ho_struct, dev_buf, dev_bytes)   # warm-up
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
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
    top = max(per_kernel, key=lambda k: per_kernel[k]["ms_per_launch"] * per_kernel[k]["launches_per_step"])
    top_ms = per_kernel[top]["ms_per_launch"]
    flops_pass = 2.0 * rows * float(sum_T) * d        # one Q_w K^T contraction over every unit
    tensor_roof = None
    if top in ("score_norm", "score_mass"):
        # One exponential per (query row, key): the pass is bound by the ex2 pipe, not by the contraction that
        # feeds it (profiles/score_tc_*: ex2 pipe the busiest unit, tensor pipe about 40 %, DRAM under 20 %).
        exps = float(rows) * float(sum_T)
        achieved = exps / (top_ms * 1e-3) / 1e12
        peak, peak_src = ex2_peak(sm_count(device), clocks)
        roof = dict(kernel=top, bound="alu", achieved=achieved, peak=peak, unit="Texp/s", frac=achieved / peak,
                    traffic=None, peak_source=peak_src, ms_per_launch=top_ms, exps_per_launch=exps,
                    sm_mhz_in_kernel=score_mhz[0 if top == "score_norm" else 1] or None,
                    frac_at_kernel_clock=(achieved / (peak * score_mhz[0 if top == "score_norm" else 1] /
                                                      (clocks.get("sm_max_mhz") or 1965.0))
                                          if score_mhz[0 if top == "score_norm" else 1] else None),
                    kernel_clock_note="one CTA's SM cycles over its wall time (cask_last_score_clock_khz): the pass runs "
                                      "under the board's power limit, below the maximum clock",
                    ex2_per_clk_per_sm_measured=ex2_rate,
                    ex2_measured_note="cask_selftest_exp_rate: FFMA + ex2 + FADD + FMUL loop, 16 warps per SM, median over SMs")
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
    event = event_roofline(hb, n_out, kind, ms_step, peaks)

    # ---- the oracle on this machine's host cores, bounded sample ------------------------------------
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w, args.cpu_units, args.similarity)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms_step, "ms_per_step_median": float(np.median(per_step)), "ms_per_step_best": float(min(per_step)),
        "ms_each_step": [round(x, 4) for x in per_step], "sustained": sustained,
        "higher_is_better": True,
        "scaling": "weak" if w.n_seqs == 1 else "strong", "vs_baseline": None, "dtype": "bf16" if w.dtype == wl.DTYPE_BF16 else "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "units_per_gpu": hb.n_units, "rows_per_unit": int(hb.T.max()), "head_dim": d,
                   "query_rows": rows, "budget": int(hb.B.max()), "tokens_per_step": total_tokens,
                   "l2": "inputs larger than L2: %.2f GB of K/V read per step" % ((hb.k.nbytes + hb.v.nbytes) / 1e9),
                   "score_path": "tcgen05" if ctx_tensor_path else "simt", "gen_seconds": round(t_gen, 1),
                   "reduced": bool(args.max_units),
                   "timing": "CUDA events on the launching stream: one bracket around all steps (value, ms_per_step), "
                             "one event after every step (median, best, this rank); per-kernel event pairs only in a "
                             "separate loop (kernels)",
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
        "other_workloads": others,
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
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="reasoning32k_b512", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--score-path", type=int, default=0, help="0: tensor-core scoring when the shape allows, 1: SIMT")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--sustained-steps", type=int, default=200,
                    help="events of the long loop that shows the level under the power limit (0: skip; N = 1 only)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the block of the other benchmark configurations timed after the headline (N = 1 only)")
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
