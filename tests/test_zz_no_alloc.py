"""cask_score_noalloc against cask_score, through the C-ABI.

The no-allocation entry point exists for callers that cannot obtain device memory at call time
(for example code running inside an engine that owns the whole device through its own pool): it
keeps its scratch in a fixed array inside the library.  This test calls it twice in a row on the
same inputs and checks both results against the ordinary entry point, which takes its scratch from
a caller-allocated workspace.  The file sorts last on purpose, so a run that stops at the first
failure has already run every other test.
"""
import numpy as np
import pytest

from paper_2604_10900_b200 import workloads as wl

pytestmark = pytest.mark.gpu

SCORE_RTOL = 1e-5        # the tolerance the parity tests put on scores


def _scores(w, n_calls=2):
    import torch
    import gpu_harness as gh
    hb = wl.make_batch(w)
    run = gh.GpuRun(hb, score_path=1)
    cb = run.cb
    ref = torch.zeros(run.sum_T, dtype=torch.float32, device="cuda:0")
    lse_ref = torch.zeros((hb.n_units, w.group * w.window), dtype=torch.float32, device="cuda:0")
    cb.cask_score(run.ctx, run.batch, run.prm, ref, lse_ref, run.ws, run.ws_bytes)
    stream = torch.cuda.current_stream("cuda:0").cuda_stream
    s = torch.full((run.sum_T,), -1.0, dtype=torch.float32, device="cuda:0")
    lse = torch.zeros_like(lse_ref)
    # one call first: it loads the kernels and resolves the address of the fixed array, which the driver may
    # back with memory of its own; from then on a call must leave the device's free memory where it found it
    cb.cask_score_noalloc(0, stream, run.batch, run.prm, s, lse)
    torch.cuda.synchronize()
    outs = []
    for _ in range(n_calls):
        s.fill_(-1.0)
        lse.zero_()
        torch.cuda.synchronize()
        # cudaMemGetInfo sees every allocation on the device, the library's own included (torch's counters see
        # only torch's allocator); nothing else allocates between the two readings
        free_before, _total = torch.cuda.mem_get_info(0)
        torch_before = torch.cuda.memory_allocated("cuda:0")
        cb.cask_score_noalloc(0, stream, run.batch, run.prm, s, lse)
        torch.cuda.synchronize()
        free_after, _total = torch.cuda.mem_get_info(0)
        assert free_after == free_before, (free_before, free_after)
        assert torch.cuda.memory_allocated("cuda:0") == torch_before
        outs.append((s.cpu().numpy(), lse.cpu().numpy()))
    torch.cuda.synchronize()
    return hb, run, ref.cpu().numpy(), lse_ref.cpu().numpy(), outs


@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("reasoning8k_b384", dict(layers=1, kv_heads=3, decode=4096 + 51)),
])
def test_noalloc_scores_match_the_workspace_entry_point_on_two_calls(name, kw):
    import gpu_harness as gh
    w = wl.WORKLOADS[name].with_(**kw)
    hb, run, ref, lse_ref, outs = _scores(w)
    so = gh.run_oracle(hb)["s"]
    for s, lse in outs:
        # the same kernels with their scratch elsewhere: the same bytes as cask_score with score_path = 1
        assert np.array_equal(s, ref)
        assert np.array_equal(lse, lse_ref)
        # and the oracle's scores within the tolerance of the parity tests
        big = so > 1e-12
        assert (np.abs(s[big] - so[big]) <= SCORE_RTOL * so[big]).all()
        assert np.abs(s[~big] - so[~big]).max(initial=0.0) <= 1e-12
    assert np.array_equal(outs[0][0], outs[1][0])        # the second call sees the first call's leftovers


def test_noalloc_refuses_a_stream_that_is_being_captured_and_keeps_the_current_device():
    import torch
    import gpu_harness as gh
    w = wl.WORKLOADS["tiny"]
    run = gh.GpuRun(wl.make_batch(w), score_path=1)
    cb = run.cb
    s = torch.zeros(run.sum_T, dtype=torch.float32, device="cuda:0")
    side = torch.cuda.Stream("cuda:0")
    torch.cuda.synchronize()
    # a call outside capture first (address look-up), checked against the ordinary entry point below
    cb.cask_score_noalloc(0, side.cuda_stream, run.batch, run.prm, s, None)
    torch.cuda.synchronize()
    assert torch.cuda.current_device() == 0
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side, capture_error_mode="relaxed"):
        rc = cb.cask_score_noalloc(0, side.cuda_stream, run.batch, run.prm, s, None, check=False)
    assert rc == cb.ERR_UNSUPPORTED                      # refused on the host: nothing was recorded or launched
    torch.cuda.synchronize()
    ref = torch.zeros_like(s)
    cb.cask_score(run.ctx, run.batch, run.prm, ref, None, run.ws, run.ws_bytes)
    torch.cuda.synchronize()
    assert np.array_equal(s.cpu().numpy(), ref.cpu().numpy())


def test_noalloc_also_agrees_with_the_tensor_core_path():
    import torch
    import gpu_harness as gh
    w = wl.WORKLOADS["reasoning8k_b384"].with_(layers=1, kv_heads=2, decode=2048 + 5)
    hb = wl.make_batch(w)
    run = gh.GpuRun(hb)                                   # default path: tensor cores for this shape
    cb = run.cb
    ref = torch.zeros(run.sum_T, dtype=torch.float32, device="cuda:0")
    cb.cask_score(run.ctx, run.batch, run.prm, ref, None, run.ws, run.ws_bytes)
    assert run.ctx.used_tensor_path
    s = torch.zeros_like(ref)
    for _ in range(2):
        cb.cask_score_noalloc(0, torch.cuda.current_stream("cuda:0").cuda_stream, run.batch, run.prm, s, None)
    torch.cuda.synchronize()
    r, g = ref.cpu().numpy(), s.cpu().numpy()
    big = r > 1e-12
    assert (np.abs(g[big] - r[big]) <= SCORE_RTOL * r[big]).all()


def test_noalloc_rejects_batches_beyond_its_fixed_capacity():
    import torch
    import gpu_harness as gh
    from paper_2604_10900_b200 import binding as cb
    # more units than the descriptor table holds
    w = wl.WORKLOADS["tiny"].with_(layers=cb.NOALLOC_MAX_UNITS // 2 + 1, decode=40, prefix=8, budget=16, reserve=8,
                                   window=4)
    run = gh.GpuRun(wl.make_batch(w))
    s = torch.zeros(run.sum_T, dtype=torch.float32, device="cuda:0")
    rc = cb.cask_score_noalloc(0, None, run.batch, run.prm, s, None, check=False)
    assert rc == cb.ERR_TOO_LARGE
    # units within the table, but partials larger than the array: 60 units x 17 chunks x 512 rows x 8 B > 4 MiB
    T = np.full(60, 33280, np.int32)
    tok = np.concatenate([[0], np.cumsum(T)]).astype(np.int64)
    b, keep = cb.make_batch(0x1000, 0x2000, 0x3000, T, np.full(60, 512, np.int32), np.full(60, 512, np.int32),
                            np.full(60, 256, np.int32), tok, 128, 4, 128, cb.DTYPE_BF16)
    assert cb.cask_score_noalloc(0, None, b, cb.params(), 0x4000, None, check=False) == cb.ERR_TOO_LARGE
    with pytest.raises(cb.CaskError, match="fixed capacity"):
        cb.cask_score_noalloc(0, None, b, cb.params(), 0x4000, None)
