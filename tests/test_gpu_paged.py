"""GPU parity for the paged cache layout: the same rows scattered over shuffled pages must give the
results of the contiguous layout (and of the oracle, which only knows the logical cache)."""
import numpy as np
import pytest

from paper_2604_10900_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ST_BOUNDS = 64


def _event(hb, **kw):
    import gpu_harness as gh
    run = gh.GpuRun(hb, **kw)
    return run, run.event()


@pytest.mark.parametrize("page_size", [16, 64, 128, 256, 48])
def test_paged_bf16_matches_contiguous_and_oracle(page_size):
    """Config-3 shape with a prefix that is not a multiple of any page size: page pieces of 16 and 64 rows,
    whole 128-row tiles inside larger pages, and a page size (48) only the SIMT kernels can serve."""
    import gpu_harness as gh
    w = wl.WORKLOADS["reasoning32k_b512"].with_(layers=1, kv_heads=2, prefix=500, decode=2048 + 77)
    hb = wl.make_batch(w)
    run_p, g = _event(hb, page_size=page_size)
    tensor = page_size != 48
    assert run_p.ctx.used_tensor_path == tensor
    assert run_p.ctx.device_flags() == 0
    o = gh.run_oracle(hb)
    st = gh.compare_event(hb, g, o)
    assert st["cascaded"] <= 1 and st["merged_elems"] > 0
    assert (g["n_out"] == 512).all()
    # same kernels, same arithmetic order: the contiguous layout gives the same bits
    run_c, c = _event(hb, score_path=0 if tensor else 1)
    for name in ("s", "kind", "seed_of", "assign", "weight", "slot_src", "slot_kind", "slot_mass", "k_out", "v_out",
                 "n_out", "unit_status", "lost_mass"):
        assert np.array_equal(g[name], c[name]), name
    assert not np.any(g["k_out"] == 768.0) and not np.any(g["v_out"] == 768.0)


def test_paged_fp32_tiny():
    """Config 1 (fp32, d=64) on pages of 16 rows: the SIMT kernels through the block table."""
    import gpu_harness as gh
    hb = wl.make_batch(wl.WORKLOADS["tiny"])
    run, g = _event(hb, page_size=16)
    assert not run.ctx.used_tensor_path
    st = gh.compare_event(hb, g, gh.run_oracle(hb))
    assert st["cascaded"] == 0 and (g["n_out"] == 128).all()


@pytest.mark.parametrize("page_size", [16, 48])
def test_page_id_outside_the_pool_is_flagged_not_followed(page_size):
    """A block-table entry beyond the pool raises CASK_ST_BOUNDS (the kernels read page 0 instead)."""
    w = wl.WORKLOADS["reasoning32k_b512"].with_(layers=1, kv_heads=2, prefix=512, decode=1024)
    hb = wl.make_batch(w)
    run, g = _event(hb, page_size=page_size, bad_page=5)
    assert run.ctx.device_flags() & ST_BOUNDS
    assert (g["unit_status"] & ST_BOUNDS).all()
    assert (g["n_out"] == 512).all()


@pytest.mark.parametrize("page_size", [16, 48])
def test_writeback_puts_the_compacted_rows_into_the_units_own_pages(page_size):
    """After cask_writeback_paged, logical row t of a unit (read through its block table) is slot t of the
    compacted cache, bit for bit; rows beyond n_out and the pool's spare pages are untouched."""
    import torch
    w = wl.WORKLOADS["reasoning32k_b512"].with_(layers=1, kv_heads=2, prefix=500, decode=1024 + 5)
    hb = wl.make_batch(w)
    run, g = _event(hb, page_size=page_size)
    cb = run.cb
    before = {n: run.dev[n].clone() for n in ("k", "v")}
    cb.cask_writeback_paged(run.ctx, run.batch, run.prm, run.out_struct, run.dev["k"], run.dev["v"], run.ws, run.ws_bytes)
    torch.cuda.synchronize()
    assert run.ctx.device_flags() == 0
    table = run.block_table.cpu().numpy().astype(np.int64)
    ps = page_size
    touched = np.zeros(run.dev["k"].shape[0], bool)
    off = 0
    for u in range(hb.n_units):
        n = int(g["n_out"][u])
        t = np.arange(n)
        rows = table[off + t // ps] * ps + t % ps
        touched[rows] = True
        for name in ("k", "v"):
            got = run.dev[name][torch.from_numpy(rows).to(run.device)].view(torch.uint16).cpu().numpy()
            want = run.out[name + "_out"][u, :n].view(torch.uint16).cpu().numpy()
            assert np.array_equal(got, want), (u, name)
        off += (int(hb.T[u]) + ps - 1) // ps
    keep = torch.from_numpy(~touched).to(run.device)
    for name in ("k", "v"):
        assert torch.equal(run.dev[name][keep].view(torch.uint16), before[name][keep].view(torch.uint16))
    # a contiguous batch is refused
    run_c, _ = _event(hb)
    assert cb.cask_writeback_paged(run_c.ctx, run_c.batch, run_c.prm, run_c.out_struct, run_c.dev["k"], run_c.dev["v"],
                                   run_c.ws, run_c.ws_bytes, check=False) == cb.ERR_SHAPE
