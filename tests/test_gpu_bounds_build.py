"""The self-checking build of the library (libcask_bounds.so, -DCASK_BOUNDS).

compute-sanitizer is not available where these tests run, so the library carries its own index checks as a build
variant: every index a kernel takes from an array that it or an earlier kernel wrote (seed rows, member rows, slots,
seed numbers) is compared with its range before it addresses memory; a bad one raises CASK_ST_BOUNDS and is replaced by
0 instead of trapping.  Here a spread of small and awkward shapes, both cache layouts, both scoring paths and a short-unit
batch run through that build: no check may fire, and every output must be the ordinary build's, byte for byte.
"""
import gc

import numpy as np
import pytest

from paper_2604_10900_b200 import build as cbuild
from paper_2604_10900_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _cases():
    tiny = wl.WORKLOADS["tiny"]
    r8k = wl.WORKLOADS["reasoning8k_b384"]
    yield "tiny", tiny, {}
    yield "tiny_noncausal", tiny, dict(causal=0)
    yield "tiny_merge_everything", tiny, dict(tau=-1.0)
    yield "tiny_evict_only", tiny, dict(tau=2.0)
    rng = np.random.default_rng(5)
    for i in range(6):                                   # small odd shapes around every branch of the budget split
        T = int(rng.integers(20, 90))
        P = int(rng.integers(0, T // 2))
        B = int(rng.integers(4, T + 4))
        W = int(rng.integers(1, min(9, T - P) + 1))
        yield f"odd{i}", tiny.with_(prefix=P, decode=T - P, budget=B, reserve=int(rng.integers(0, B + 1)), window=W,
                                    layers=2), {}
    yield "bf16_tensor_path", r8k.with_(layers=1, kv_heads=2, decode=1024 + 19), {}
    yield "bf16_paged", r8k.with_(layers=1, kv_heads=2, decode=900), dict(page_size=16)
    yield "bf16_many_seeds", wl.WORKLOADS["reasoning32k_b1024"].with_(layers=1, kv_heads=1, decode=3000), {}
    yield "short_units", wl.WORKLOADS["serving_steady_b512"].with_(layers=1, kv_heads=2, n_seqs=3), {}


def _event(hb, kw):
    import torch
    import gpu_harness as gh
    run = gh.GpuRun(hb, **kw)
    g = run.event()
    flags = run.ctx.device_flags()
    bits = {k: (t.view(torch.uint16) if t.dtype == torch.bfloat16 else t).cpu().numpy() for k, t in run.out.items()}
    run.ctx.close()
    del run
    gc.collect()
    return g, bits, flags


def test_every_index_check_stays_silent_and_the_results_are_the_ordinary_builds():
    from paper_2604_10900_b200 import binding as cb
    cbuild.build_lib()
    cbuild.build_lib(bounds=True)
    ran = 0
    try:
        for name, w, kw in _cases():
            hb = wl.make_batch(w)
            cb.use_library(None)
            g0, b0, f0 = _event(hb, kw)
            cb.use_library(cbuild.LIB_BOUNDS)
            g1, b1, f1 = _event(hb, kw)
            assert f0 == 0 and f1 == 0, (name, f0, f1)
            assert not (g1["unit_status"] & (cb.ST_BOUNDS | cb.ST_TIMEOUT)).any(), name
            for k in b0:
                assert np.array_equal(b0[k], b1[k]), (name, k)
            ran += 1
    finally:
        cb.use_library(None)
    assert ran >= 14
