"""A seeded sweep over randomly drawn shapes, storage types, kernels, compaction modes and entry points,
each in lockstep with the oracle: decode steps, chunked prompts and the recompute mode on shapes nobody
picked by hand (budgets and windows that are not multiples of anything, r and m at their extremes,
1 to 700 units)."""
import random

import pytest
import torch

from lockstep import SortedView, run_lockstep, run_lockstep_chunked, run_lockstep_recompute
from paper_2305_17118_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3, "int4": 2e-3}


def _draw(rng):
    dtype = rng.choice(["f32", "f16", "bf16", "int4"])
    d = rng.choice([64, 128])
    U = rng.choice([1, 2, 3, 7, 130, 300, 600, 700])
    B = rng.choice([2, 5, 33, 64, 97, 150, 257, 410, 600])
    r = rng.randint(0, B - 1)
    m = rng.randint(1, B - r)
    w = rng.choice([1, 2, 7, 31, 32, 33, 64, 100, 200])
    unordered = rng.random() < 0.5
    kernel = rng.choice([None, None, 1, 2])
    mode = rng.choice(["decode", "decode", "chunk", "recompute"])
    if mode in ("chunk", "recompute") and w < 2:
        mode = "decode"
    return dtype, d, U, B, r, w, m, unordered, kernel, mode


@pytest.mark.parametrize("seed", [101, 102, 103, 104])
def test_random_shapes_in_lockstep(seed):
    from paper_2305_17118_b200 import binding as sh
    rng = random.Random(seed)
    for _ in range(12):
        dtype, d, U, B, r, w, m, unordered, kernel, mode = _draw(rng)
        T = min(B + 3 * m + 7, B + 220)
        q, k, v = wl.random_stream(U, d, T, seed=rng.randint(0, 10 ** 6), dtype=dtype, peaked=rng.choice([1.0, 3.0]),
                                   device="cuda")
        units = torch.arange(U) if U <= 8 else torch.unique(torch.tensor(sorted(rng.sample(range(U), 6) + [0, U - 1])))
        kw = dict(auto_compress=False, kernel=kernel, unordered=unordered)
        what = f"seed {seed}: {dtype} d={d} U={U} B={B} r={r} w={w} m={m} unordered={unordered} kernel={kernel} {mode}"
        try:
            if mode == "recompute":
                h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, recompute_record=True, **kw), units=units.numpy())
                run_lockstep_recompute(h, dtype, lambda t: (q[t - 1], k[t - 1], v[t - 1]), T, units, TOL[dtype])
            elif mode == "chunk":
                h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, **kw), units=units.numpy())
                sizes = [rng.randint(1, 64) for _ in range(4)]
                blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
                run_lockstep_chunked(h, dtype, blk, T, units, TOL[dtype], chunk_sizes=sizes)
            else:
                h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, **kw), units=units.numpy())
                run_lockstep(h, dtype, lambda t: (q[t - 1], k[t - 1], v[t - 1]), T, units, TOL[dtype])
        except AssertionError as e:
            raise AssertionError(f"{what}: {e}") from e
