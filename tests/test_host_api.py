"""Host-side checks of the C-ABI library that need no GPU: exports, budget split, workspace sizing."""
import ctypes as C
import json
import os
import re

import numpy as np
import pytest

from oracle import cask_oracle as orc
from paper_2604_10900_b200 import binding as cb
from paper_2604_10900_b200 import build as cbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    cbuild.build_lib()


def _batch(T, P, B, reserve, W=4, d=64, g=2, dtype=1, k=0x1000, **kw):
    T = np.atleast_1d(np.array(T, np.int32))
    tok = np.concatenate([[0], np.cumsum(T)]).astype(np.int64)
    return cb.make_batch(kw.pop("k", k), kw.pop("v", 0x2000), kw.pop("q", 0x3000), T, np.atleast_1d(P),
                         np.atleast_1d(B), np.atleast_1d(reserve), tok, d, g, W, dtype, **kw)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "cask.h")).read()
    declared = set(re.findall(r"\b(cask_[a-z_]+)\s*\(", header))
    assert declared == set(cb.EXPORTS), declared ^ set(cb.EXPORTS)
    lib = C.CDLL(cb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_plan_host_matches_hand_worked_table_and_oracle_rule():
    tab = json.load(open(os.path.join(ROOT, "tests", "golden", "budget_split_table.json")))
    for T, P, B, res, W, Bp, Pk, Bd, r, c, m, exh, nout in tab["rows"]:
        b, keep = _batch(T, P, B, res, W=W)
        pl = cb.cask_plan_host(b, cb.params())[0]
        assert list(pl[:6]) == [Bp, Pk, Bd, r, c, m]
        assert bool(pl[6] & cb.ST_PREFIX_BUDGET_EXHAUSTED) == bool(exh) and pl[7] == nout
    for gamma in (0.0, 0.25, 0.5, 1.0):
        for T in range(1, 14):
            for P in range(0, T + 1):
                for B in range(1, 15):
                    for res in range(0, B + 1):
                        for W in (1, 3):
                            if W > T:
                                continue
                            b, keep = _batch(T, P, B, res, W=W)
                            pl = cb.cask_plan_host(b, cb.params(gamma=gamma))[0]
                            assert np.array_equal(pl, orc.plan(T, P, B, res, W, gamma)), (T, P, B, res, W, gamma)


def test_workspace_bytes_and_rejections():
    b, keep = _batch([1000, 300], [100, 0], [128, 64], [64, 32])
    n = cb.cask_workspace_bytes(b, cb.params())
    assert n > 1300 * 4 * 4 and n % 256 == 0
    bad, keep2 = _batch([1000], [100], [128], [200])          # reserve > B
    assert cb.cask_workspace_bytes(bad, cb.params()) == 0
    bad, keep2 = _batch([1000], [100], [128], [64], k=0x1004)  # misaligned base
    assert cb.cask_workspace_bytes(bad, cb.params()) == 0
    bad, keep2 = _batch([1000], [100], [128], [64], page_size=16)
    assert cb.cask_workspace_bytes(bad, cb.params()) == 0
    assert cb.cask_workspace_bytes(b, cb.params(gamma=-0.1)) == 0
    assert b"NULL" in cb.lib().cask_strerror(cb.ERR_NULL)
    empty = cb.CaskBatch()                                    # n_units = 0: nothing to plan, no error
    assert cb.cask_plan_host(empty, cb.params()).shape == (0, 8)
    with pytest.raises(cb.CaskError):
        oops, keep3 = _batch([10], [100], [4], [1])           # P > T
        cb.cask_plan_host(oops, cb.params())


def test_null_context_is_refused():
    b, keep = _batch([1000], [100], [128], [64])
    rc = cb.lib().cask_score(None, C.byref(b), C.byref(cb.params()), 0x100, None, 0x100, 1 << 30)
    assert rc == cb.ERR_NULL


def test_host_event_device_bytes_of_one_slice_and_of_many():
    """The host-buffer entry point cuts a batch with more than 16 MB of keys into slices of units, each with its own
    staging area and workspace inside the caller's buffer: the size it asks for holds the keys and values of every
    unit once, grows with the batch, and is the plain single-batch size below the cut."""
    prm = cb.params()
    d, W, g, Bmax = 128, 16, 2, 256
    kv = lambda T: 2 * int(np.sum(T)) * d * 4          # fp32 keys + values (the dtype _batch builds)
    small_T = [3000] * 4                                # 6 MB of keys: one slice
    b1, keep1 = _batch(small_T, [100] * 4, [Bmax] * 4, [64] * 4, W=W, d=d, g=g)
    n1 = cb.cask_host_event_device_bytes(b1, prm, Bmax)
    assert n1 % 256 == 0 and n1 > kv(small_T) + cb.cask_workspace_bytes(b1, prm)
    big_T = [9000 + 37 * (i % 5) for i in range(60)]    # 277 MB of keys: about ten slices of ragged units
    b2, keep2 = _batch(big_T, [100] * 60, [Bmax] * 60, [64] * 60, W=W, d=d, g=g)
    n2 = cb.cask_host_event_device_bytes(b2, prm, Bmax)
    assert n2 % 256 == 0 and n2 > kv(big_T)
    # per-slice workspaces together stay close to the workspace of the whole batch (a fixed part per slice)
    whole = kv(big_T) + cb.cask_workspace_bytes(b2, prm)
    assert whole < n2 < 1.6 * whole
    assert cb.cask_host_event_device_bytes(b2, prm, 0) == 0          # no output rows
    bad, keep3 = _batch(big_T, [100] * 60, [Bmax] * 60, [300] * 60, W=W, d=d, g=g)   # reserve > B
    assert cb.cask_host_event_device_bytes(bad, prm, Bmax) == 0
