"""The bounds-checked build of the library (-DSH_DEBUG_BOUNDS), the stand-in for a memory checker on machines
where none can be run: every index a kernel derives from workspace state is range-checked, and a violation is
reported through the device error word (sh_state -> SH_EDEVICE) instead of being dereferenced.  The parity cases
below run that build in lockstep with the oracle - no check may fire on healthy state - and one case corrupts a
per-unit row count in the workspace and expects the report, with nothing written out of range."""
import ctypes as C

import numpy as np
import pytest
import torch

from lockstep import SortedView, run_lockstep, run_lockstep_chunked, run_lockstep_recompute
from paper_2305_17118_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3, "int4": 2e-3}


@pytest.fixture()
def shb(monkeypatch):
    """The binding with the bounds-checked library in place of the normal one."""
    import gc
    from paper_2305_17118_b200 import binding, build
    gc.collect()                                             # handles of earlier tests go while their library is current
    dbg = binding.declare(C.CDLL(build.build(debug_bounds=True)))
    monkeypatch.setattr(binding, "lib", dbg)
    yield binding
    gc.collect()


def _healthy(sh, h):
    assert sh.lib.sh_state(h._h, None, None, None, None, None, None) == sh.SH_OK


@pytest.mark.parametrize("dtype,d,kernel,U", [("f32", 64, None, 5), ("f16", 128, None, 5), ("bf16", 128, 2, 5), ("int4", 128, None, 5),
                                               ("f16", 64, 1, 601), ("int4", 128, None, 601), ("bf16", 128, None, 301)])
@pytest.mark.parametrize("stable", [False, True])
def test_no_check_fires_on_healthy_state_decode_and_compress(shb, dtype, d, kernel, U, stable):
    B, r, w, m, T = 150, 9, 37, 41, 330
    q, k, v = wl.random_stream(U, d, T, seed=131 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = shb.Handle(B, r, w, m, U, d, dtype, auto_compress=False, kernel=kernel, unordered=not stable)
    units = torch.arange(U) if U <= 8 else torch.tensor([0, 1, 148, U - 1])
    res, _ = run_lockstep(h, dtype, lambda t: (q[t - 1], k[t - 1], v[t - 1]), T, units, TOL[dtype])
    assert res.compressions >= 4
    _healthy(shb, h)
    del h


@pytest.mark.parametrize("dtype,d", [("f16", 128), ("int4", 128), ("f32", 64), ("bf16", 64)])
def test_no_check_fires_on_healthy_state_chunks_and_recount(shb, dtype, d):
    U, B, r, w, m, T = 6, 150, 9, 37, 41, 300
    q, k, v = wl.random_stream(U, d, T + 40, seed=137, dtype=dtype, peaked=3.0, device="cuda")
    h = shb.Handle(B, r, w, m, U, d, dtype, auto_compress=False, recompute_record=True)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype], recompute=True, chunk_sizes=[64, 7, 33])
    run_lockstep_recompute(h, dtype, lambda t: (q[t - 1], k[t - 1], v[t - 1]), 40, torch.arange(U), TOL[dtype], orc=orc)
    _healthy(shb, h)
    del h


@pytest.mark.parametrize("kernel", [1, 2])
def test_corrupt_row_count_is_reported_not_dereferenced(shb, kernel):
    """A ragged handle keeps per-unit row counts in the workspace.  One of them is overwritten with a value beyond
    the budget (a workspace image restored from foreign data could hold that); the bounds-checked kernels skip
    the unit and set the error word, the other units are served as usual, memory next to the unit's rows is
    untouched."""
    dtype, d, lengths, ups, B, r, w, m = "f16", 128, [3, 9], 2, 16, 2, 8, 6
    U = len(lengths) * ups
    q, k, v = wl.random_stream(U, d, 12, seed=139, dtype=dtype, device="cuda")
    good = shb.Handle(B, r, w, m, U, d, dtype, kernel=kernel, auto_compress=False)
    bad = shb.Handle(B, r, w, m, U, d, dtype, kernel=kernel, auto_compress=False)
    for h in (good, bad):
        h.prefill_ragged(q[:9].contiguous(), k[:9].contiguous(), v[:9].contiguous(), lengths)
    # find the per-unit row counts in the workspace: the only place that holds [3, 3, 9, 9] as consecutive int32
    words = bad.slab[bad._slab_off:bad._slab_off + bad.workspace_bytes].view(torch.int32)
    pattern = torch.tensor([3, 3, 9, 9], dtype=torch.int32, device="cuda")
    hits = (words.unfold(0, 4, 1) == pattern).all(dim=1).nonzero().flatten().tolist()
    assert len(hits) == 2                       # row counts, then tokens streamed (the same numbers so far)
    before = bad.slab.clone()
    words[hits[0] + 1] = B + 7                  # unit 1 claims more rows than its budget
    out_g = good.decode_step(q[9], k[9], v[9])
    out_b = bad.decode_step(q[9], k[9], v[9])
    assert shb.lib.sh_state(good._h, None, None, None, None, None, None) == shb.SH_OK
    assert shb.lib.sh_state(bad._h, None, None, None, None, None, None) == shb.SH_EDEVICE
    keep = [0, 2, 3]
    assert torch.equal(out_g[keep], out_b[keep])            # the healthy units are served as usual
    # unit 1's key and value rows are exactly as they were (nothing appended, nothing beyond them touched)
    rowb = d * 2
    K1 = slice(bad._slab_off + 1 * B * rowb, bad._slab_off + 2 * B * rowb)
    assert torch.equal(bad.slab[K1], before[K1])
    del good, bad
