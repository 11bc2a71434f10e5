"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from lockstep import (SortedView, assert_same_state, run_lockstep, run_lockstep_chunked, run_lockstep_recompute,
                      to_oracle)
from paper_2305_17118_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3, "int4": 2e-3}


@pytest.fixture(scope="module")
def sh():
    from paper_2305_17118_b200 import binding
    return binding


def _stream_fn(q, k, v):
    return lambda t: (q[t - 1], k[t - 1], v[t - 1])


# ---- small shapes, every unit, every dtype, several splits and ragged sizes --------------
@pytest.mark.parametrize("dtype,d", [("f32", 64), ("f32", 128), ("f16", 128), ("f16", 64), ("bf16", 128),
                                      ("bf16", 64), ("int4", 128), ("int4", 64)])
@pytest.mark.parametrize("split", [1, 2, 4, 8])
@pytest.mark.parametrize("stable", [False, True])
def test_lockstep_small(sh, dtype, d, split, stable):
    """Every storage type and head size, every cluster split, both compaction modes (the default, which
    fills holes from the tail, and the stable one)."""
    U, B, r, w, m, T = 5, 150, 9, 37, 41, 420      # ragged: B, w not multiples of 32; several tiles
    q, k, v = wl.random_stream(U, d, T, seed=7 + split, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, split=split, auto_compress=False, unordered=not stable)
    res, _ = run_lockstep(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 6
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("B,r,w,m", [(33, 0, 1, 33), (64, 63, 5, 1), (32, 4, 100, 7), (1000, 10, 400, 500),
                                     (2, 1, 3, 1), (97, 5, 64, 92), (3000, 10, 400, 1500)])
@pytest.mark.parametrize("stable", [False, True])
def test_lockstep_edge_parameters(sh, B, r, w, m, stable):
    U, d, dtype = 3, 64, "f16"
    T = min(3 * B + 50, 1300) if B <= 1000 else B + 100
    q, k, v = wl.random_stream(U, d, T, seed=B, dtype=dtype, peaked=2.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=not stable)
    res, _ = run_lockstep(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 1


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("f32", 128), ("f16", 64), ("bf16", 64), ("f16", 128), ("bf16", 128),
                                      ("int4", 128), ("int4", 64)])
def test_lockstep_direct_kernel_many_units(sh, dtype, d):
    """The direct-load decode kernel in the CTA shape it takes from 592 units on (4 warps, more rows per
    thread), every storage type and head size, i.e. every instance the launcher can pick; a sample of
    units in lockstep."""
    U, B, r, w, m, T = 601, 77, 6, 21, 30, 150
    q, k, v = wl.random_stream(U, d, T, seed=13, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, kernel=1, auto_compress=False)
    units = torch.tensor([0, 1, 17, 148, 299, 300, 592, 600])
    res, _ = run_lockstep(h, dtype, _stream_fn(q, k, v), T, units, TOL[dtype])
    assert res.compressions >= 3
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("dtype,d", [("f16", 128), ("bf16", 128), ("f32", 128), ("f32", 64)])
@pytest.mark.parametrize("U,B,r,w,m", [(5, 150, 9, 37, 41), (301, 130, 16, 33, 50), (3, 700, 5, 64, 300), (2, 40, 3, 9, 20),
                                       (200, 150, 9, 37, 41), (296, 90, 4, 20, 35)])
def test_lockstep_pipelined_kernel(sh, dtype, d, U, B, r, w, m):
    """The persistent bulk-copy variant of the decode kernel, forced on shapes that
    cover fewer units than CTAs, more units than SMs, ragged last tiles and tiny caches,
    for every row size it serves (256 and 512 bytes); between one and two units per SM (the last two
    cases) the 16-bit stores run two CTAs per SM with tiles of 64 rows."""
    T = 2 * B + 2 * m + 7
    q, k, v = wl.random_stream(U, d, T, seed=11 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, split=1, kernel=2, auto_compress=False)
    res, _ = run_lockstep(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 3
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("U,B,r,w,m,sizes", [(5, 150, 9, 37, 41, [64, 7, 33, 1, 50]), (3, 410, 64, 128, 64, [64]),
                                             (2, 700, 5, 64, 300, [32, 17]), (4, 40, 3, 9, 20, [5, 9, 2]),
                                             (130, 96, 8, 70, 30, [64, 31])])
@pytest.mark.parametrize("chunk_kernel", [1, 2, 3])
def test_lockstep_chunked_prompt_kernel(sh, dtype, U, B, r, w, m, sizes, chunk_kernel):
    """sh_prefill_chunk against the oracle replaying the same steps one by one: outputs of
    every step, its record bits, positions, counters and kept sets."""
    d, T = 128, 2 * B + 2 * m + 11
    q, k, v = wl.random_stream(U, d, T, seed=17 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, prefill_chunk=chunk_kernel)   # 1: tcgen05, persistent CTAs and TMA; 2: warp-level MMA; 3: tcgen05, one CTA per unit
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype], chunk_sizes=sizes)
    assert res.steps == T and res.compressions >= 3
    assert res.adoptions <= 1e-4 * res.slot_steps + 2
    # and the decode step carries on from the state the chunks left
    q2, k2, v2 = wl.random_stream(U, d, 40, seed=99, dtype=dtype, peaked=3.0, device="cuda")
    run_lockstep(h, dtype, lambda t: (q2[t - T - 1], k2[t - T - 1], v2[t - T - 1]), 40, torch.arange(U), TOL[dtype], orc=orc)


@pytest.mark.parametrize("U,B,r,w,m,sizes", [(5, 150, 9, 37, 41, [37, 7, 33, 1]), (3, 410, 64, 128, 64, [64]),
                                             (150, 96, 8, 70, 30, [64, 31]), (2, 1300, 10, 64, 650, [64, 13])])
def test_lockstep_chunked_int4_store(sh, U, B, r, w, m, sizes):
    """The chunk kernel of the int4-g64 store (codes as tensor-core operands, scales applied in fp32):
    outputs, record bits, positions, counters and kept sets against the oracle's quantised cache; then
    decode steps from the state the chunks left; and the quantised rows equal the oracle's bit for bit."""
    dtype, d, T = "int4", 128, min(2 * B + 2 * m + 11, B + 2 * m + 60)
    q, k, v = wl.random_stream(U, d, T, seed=37 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False))
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype], chunk_sizes=sizes)
    assert res.steps == T and res.compressions >= 2
    assert res.adoptions <= 1e-4 * res.slot_steps + 2
    n = h.n
    for u in (0, U - 1):
        K, V = h.export_unit(u)
        oK, oV = orc.cache(u)
        assert (K[:n].astype(np.float64) == oK).all() and (V[:n].astype(np.float64) == oV).all()
    q2, k2, v2 = wl.random_stream(U, d, 30, seed=97, dtype=dtype, peaked=3.0, device="cuda")
    run_lockstep(h, dtype, lambda t: (q2[t - T - 1], k2[t - T - 1], v2[t - T - 1]), 30, torch.arange(U), TOL[dtype], orc=orc)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("U,B,r,w,m,sizes", [(2, 2100, 10, 400, 1050, [64, 64, 13]), (150, 33, 2, 70, 11, [64, 3]),
                                             (1, 129, 1, 64, 64, [64]), (3, 1000, 10, 5, 500, [5, 2])])
def test_lockstep_chunked_tcgen05_kernel_shapes(sh, dtype, U, B, r, w, m, sizes):
    """The tcgen05 chunk kernel on shapes the warp-level one cannot take (budgets beyond ~700), with more
    units than CTA slots, a single key tile, a tile boundary at n0 + 1, and a window shorter than a chunk."""
    d, T = 128, min(2 * B + 2 * m + 11, B + m + 150)
    q, k, v = wl.random_stream(U, d, T, seed=27 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype], chunk_sizes=sizes)
    assert res.steps == T and res.compressions >= 1
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("U,B,r,w,m,sizes", [(700, 150, 9, 64, 41, [64, 7, 33]), (1000, 70, 5, 64, 30, [64]),
                                             (297, 200, 9, 64, 90, [13, 64])])
def test_lockstep_chunked_persistent_ctas(sh, dtype, U, B, r, w, m, sizes):
    """The persistent tcgen05 chunk kernel with more units than CTAs (two per SM): every CTA walks over several
    units, unevenly many, so its tile rings, the query buffer and the output accumulator are reused across
    units; chunk lengths that leave stale cache rows in the last value tile, a first tile that already holds
    rows of the chunk (n0 < 64), and a last unit that is the only second unit of its CTA (U = 297)."""
    d, T = 128, B + 2 * m + 40
    q, k, v = wl.random_stream(U, d, T, seed=41 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    units = torch.cat([torch.arange(0, 6), torch.arange(290, min(U, 310)), torch.arange(U - 5, U)]).unique()
    res, _ = run_lockstep_chunked(h, dtype, blk, T, units, TOL[dtype], chunk_sizes=sizes)
    assert res.steps == T and res.compressions >= 2
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


def _poison_rows(h):
    """Every byte of the handle's K and V regions becomes 0xFF: NaN in each floating-point storage type."""
    row_bytes = {0: 4 * h.D, 1: 2 * h.D, 2: 2 * h.D}[h.dtype]
    kv = 2 * ((h.U * h.B * row_bytes + 255) // 256 * 256)
    h.slab[h._slab_off:h._slab_off + kv] = 0xFF


@pytest.mark.parametrize("dtype,d,chunk_kernel,recompute", [("f16", 128, 1, False), ("bf16", 128, 1, True), ("f16", 128, 3, True),
                                                            ("f16", 128, 2, False), ("f32", 128, 1, False), ("f16", 64, 1, True),
                                                            ("f32", 64, 1, False)])
def test_rows_that_hold_no_token_are_never_used(sh, dtype, d, chunk_kernel, recompute):
    """A cache whose unused rows hold NaN (a caller's workspace is not cleared by the library): chunks whose last
    tile reaches past the live rows, the recount, the decode steps and the compressions must neither read such a
    row into a result nor let it through a masked product (0 x NaN)."""
    U, B, r, w, m, T = 7, 150, 9, 64, 41, 300
    q, k, v = wl.random_stream(U, d, T + 40, seed=61, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, prefill_chunk=chunk_kernel, recompute_record=recompute)
    _poison_rows(h)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    outs = []
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype], chunk_sizes=[64, 7, 33], recompute=recompute,
                                    outs=outs)
    assert res.steps == T and res.compressions >= 2
    assert all(torch.isfinite(o).all() for o in outs)
    if not recompute:
        run_lockstep(h, dtype, lambda t: (q[t - 1], k[t - 1], v[t - 1]), 40, torch.arange(U), TOL[dtype], orc=orc)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("U,B,r,w,m,sizes", [(600, 600, 10, 400, 300, [128, 77, 100, 65]), (900, 300, 9, 128, 150, [128, 90]),
                                             (592, 200, 3, 128, 128, [128]), (749, 130, 2, 200, 100, [65, 128, 1]),
                                             (5, 600, 10, 400, 300, [128, 77, 100, 65]), (330, 300, 9, 128, 150, [128, 90])])
def test_lockstep_chunked_wide_kernel(sh, dtype, U, B, r, w, m, sizes):
    """Chunks of 65 to 128 tokens.  From four units per SM on: the wide shape of the persistent tcgen05 kernel (one
    query per MMA row, 16 softmax warps, one CTA per SM), with several units per CTA and mixed with chunks of the
    narrow shape; with fewer units (the last two cases) the same chunks go as two launches of the narrow shape."""
    d, T = 128, B + 2 * m + 40
    q, k, v = wl.random_stream(U, d, T + 30, seed=51 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    assert h.prefill_chunk_max == 128
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    units = torch.arange(U) if U <= 8 else torch.cat([torch.arange(0, 3), torch.arange(147, 150), torch.arange(U - 3, U)]).unique()
    res, orc = run_lockstep_chunked(h, dtype, blk, T, units, TOL[dtype], chunk_sizes=sizes)
    assert res.steps == T and res.compressions >= 2
    assert res.adoptions <= 1e-4 * res.slot_steps + 2
    run_lockstep(h, dtype, lambda t: (q[t - 1], k[t - 1], v[t - 1]), 30, units, TOL[dtype], orc=orc)


@pytest.mark.parametrize("dtype,U", [("f16", 5), ("bf16", 640)])
def test_chunked_prompt_without_outputs_leaves_the_same_state(sh, dtype, U):
    """sh_prefill with no output buffer (the second contraction is skipped altogether) leaves state bit-identical
    to a twin that asked for the outputs: rows, positions, record, counters."""
    B, r, w, m, d, T = 150, 9, 64, 41, 128, 400
    q, k, v = wl.random_stream(U, d, T, seed=5, dtype=dtype, peaked=3.0, device="cuda")
    a = sh.Handle(B, r, w, m, U, d, dtype)
    b = sh.Handle(B, r, w, m, U, d, dtype)
    out = torch.empty(T, U, d, device="cuda")
    a.prefill(q, k, v, out)
    b.prefill(q, k, v, None)
    assert a.state()[1] == T
    assert_same_state(a, b)
    assert torch.isfinite(out).all()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("U,B,r,w,m,chunk_kernel", [(5, 150, 9, 37, 41, 1), (3, 410, 64, 128, 64, 1), (140, 96, 8, 70, 30, 1),
                                                    (2, 40, 3, 9, 20, 1), (2, 1300, 10, 200, 650, 1), (5, 150, 9, 37, 41, 2),
                                                    (3, 410, 64, 128, 64, 2), (140, 96, 8, 70, 30, 2),
                                                    (5, 150, 9, 37, 41, 3), (3, 410, 64, 128, 64, 3), (2, 1300, 10, 200, 650, 3),
                                                    (700, 100, 9, 140, 41, 1), (3, 300, 5, 300, 120, 1)])
def test_lockstep_record_recomputed_at_compression(sh, dtype, U, B, r, w, m, chunk_kernel):
    """SH_OPT_RECORD_MODE = 1: Algorithm 2 as stated, the record rebuilt at each compression from
    the stored queries of the last w steps against the present cache."""
    d, T = 128, min(2 * B + 3 * m + 5, B + 2 * m + 30)
    q, k, v = wl.random_stream(U, d, T, seed=23 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, recompute_record=True, prefill_chunk=chunk_kernel)
    res, orc = run_lockstep_recompute(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 3
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("U,B,r,w,m", [(5, 150, 9, 37, 41), (3, 410, 64, 128, 64), (140, 96, 8, 70, 30)])
@pytest.mark.parametrize("unordered", [False, True])
def test_lockstep_record_recomputed_int4_store(sh, U, B, r, w, m, unordered):
    """SH_OPT_RECORD_MODE = 1 on the int4 store: the decode kernel keeps the ring of queries, the int4 chunk
    kernel recounts against the quantised cache (w beyond 64: two CTAs per unit)."""
    dtype, d, T = "int4", 128, min(2 * B + 3 * m + 5, B + 2 * m + 30)
    q, k, v = wl.random_stream(U, d, T, seed=43 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, recompute_record=True, unordered=unordered)
    h = SortedView(h) if unordered else h
    res, orc = run_lockstep_recompute(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 3
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


def test_recompute_mode_through_prefill_and_automatic_compression(sh):
    """Same mode driven the way an application would: chunked sh_prefill, then decode steps with
    automatic compression.  The library decides on its own here, so its per-step bits cannot be handed
    to the oracle; instead a twin handle is driven through the same launches by hand (chunks, then
    steps, explicit recount and compression) in lockstep with the oracle, and the free-running handle
    must end bit-identical to the twin, outputs included."""
    U, d, B, r, w, m, P, T, dtype = 12, 128, 120, 8, 50, 40, 300, 420, "f16"
    q, k, v = wl.random_stream(U, d, T, seed=31, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, recompute_record=True)
    outs = torch.empty(T, U, d, device="cuda")
    h.prefill(q[:P].contiguous(), k[:P].contiguous(), v[:P].contiguous(), outs[:P])
    for t in range(P, T):
        h.decode_step(q[t], k[t], v[t], outs[t])
    twin = sh.Handle(B, r, w, m, U, d, dtype, recompute_record=True, auto_compress=False)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    t_outs = []
    res, orc = run_lockstep_chunked(twin, dtype, blk, P, torch.arange(U), TOL[dtype], recompute=True, outs=t_outs,
                                    single_via_step=True)
    res2, _ = run_lockstep_recompute(twin, dtype, _stream_fn(q, k, v), T - P, torch.arange(U), TOL[dtype], orc=orc)
    assert res.compressions + res2.compressions >= 7
    assert torch.equal(outs[:P], torch.cat(t_outs))
    assert_same_state(h, twin)


def test_paper_hyperparameters_chunked_prompt_then_decode(sh):
    """The values the paper uses in all its experiments (Section 4.1: r = 10, w = 400, m = 0.5 B): chunks of 128
    tokens on the wide shape of the persistent kernel."""
    U, d, B, r, w, m, dtype = 3, 128, 600, 10, 400, 300, "bf16"
    T = B + 2 * m + 40
    q, k, v = wl.random_stream(U, d, T + 60, seed=61, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    assert h.prefill_chunk_max == 128
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype])
    assert res.compressions == 3
    run_lockstep(h, dtype, _stream_fn(q, k, v), 60, torch.arange(U), TOL[dtype], orc=orc)


@pytest.mark.parametrize("name,units,prompt,compressions", [("opt6b", 24, 700, 5), ("opt13b", 640, 900, 4)])
def test_prefill_uses_chunks_and_matches_oracle(sh, name, units, prompt, compressions):
    """sh_prefill with its automatic chunking and compression on the OPT-6.7B-shaped stream (chunks of 64 tokens) and
    on a layer of the OPT-13B-shaped one with enough units for the wide shape (chunks of 128).  A twin handle
    is driven through the same sequence of launches by hand, in lockstep with the oracle (every output,
    record bit, counter and kept set, with adoption inside the 1e-6 window); the handle that went
    through sh_prefill must be bit-identical to the twin.  Then decode steps in lockstep."""
    cfg = wl.CONFIGS[name].scaled(units=units, prompt=prompt)
    st = wl.Stream(cfg, device="cuda")
    h = sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False)
    q, k, v = st.block(1, cfg.prompt + 1)
    out = torch.empty(cfg.prompt, cfg.units, cfg.head_dim, device="cuda")
    before = h.launch_count
    h.prefill(q, k, v, out)
    assert h.launch_count - before < cfg.prompt // 8        # chunks, not one launch per token
    twin = sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False)
    sample = torch.arange(cfg.units) if cfg.units <= 32 else torch.tensor([0, 1, 147, 148, 295, 296, cfg.units - 2, cfg.units - 1])
    t_outs = []
    res, orc = run_lockstep_chunked(twin, cfg.dtype, lambda t0, t1: (q[t0 - 1:t1 - 1], k[t0 - 1:t1 - 1], v[t0 - 1:t1 - 1]),
                                    cfg.prompt, sample, TOL[cfg.dtype], outs=t_outs, single_via_step=True)
    assert res.compressions == compressions
    assert torch.equal(out, torch.cat(t_outs))
    assert_same_state(h, twin)
    run_lockstep(h, cfg.dtype, st.step, 70, sample, TOL[cfg.dtype], orc=orc)


# ---- the benchmark's own configurations ----------------------------------------------------
def test_config_tiny_every_step(sh):
    cfg = wl.CONFIGS["tiny"]
    st = wl.Stream(cfg, device="cuda")
    h = sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False)
    res, orc = run_lockstep(h, cfg.dtype, st.step, cfg.total_steps, torch.arange(cfg.units), TOL[cfg.dtype])
    assert res.compressions == 13
    # the four boosted keys are what the record is meant to keep
    for p in wl.PIVOT_POSITIONS:
        assert (orc.positions() == p).any(axis=1).all()


@pytest.mark.parametrize("name", ["opt6b", "opt6b_int4"])
@pytest.mark.parametrize("stable", [False, True])
def test_config_opt6b_shapes(sh, name, stable):
    cfg = wl.CONFIGS[name]
    st = wl.Stream(cfg, device="cuda")
    units = wl.sample_units(cfg, 48)
    h = sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False, unordered=not stable)
    res, _ = run_lockstep(h, cfg.dtype, st.step, cfg.total_steps, units, TOL[cfg.dtype], state_every=16)
    assert res.compressions == 26
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("unordered", [True, False])
def test_config_opt66b_full_size_sampled_units(sh, unordered):
    """The workload the benchmark times, in its launch configuration (unordered compaction; the
    library's default stable compaction as well), checked on a sample of units all the way through
    prompt and decode."""
    cfg = wl.CONFIGS["opt66b"]
    st = wl.Stream(cfg, device="cuda")
    units = wl.sample_units(cfg, 24)
    h = SortedView(sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False,
                             unordered=unordered), units=units)
    res, _ = run_lockstep(h, cfg.dtype, st.step, cfg.total_steps, units, TOL[cfg.dtype], state_every=64)
    assert res.compressions == 30
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


def test_config_opt66b_full_size_chunked_prompt_sampled_units(sh):
    """The prompt phase of the benchmark's workload at full size (9216 units per launch of the tcgen05
    chunk kernel, unordered compaction as the benchmark runs it), a sample of units in lockstep with
    the oracle through several compressions, then decode steps from the state the chunks left."""
    cfg = wl.CONFIGS["opt66b"]
    st = wl.Stream(cfg, device="cuda")
    units = wl.sample_units(cfg, 24)
    h = SortedView(sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False,
                             unordered=True), units=units)
    T = cfg.B + 5 * cfg.m + 20
    blk = lambda t0, t1: st.block(t0, t1)
    res, orc = run_lockstep_chunked(h, cfg.dtype, blk, T, units, TOL[cfg.dtype], chunk_sizes=[64])
    assert res.steps == T and res.compressions == 6
    assert res.adoptions <= 1e-4 * res.slot_steps + 2
    run_lockstep(h, cfg.dtype, st.step, 30, units, TOL[cfg.dtype], orc=orc)


@pytest.mark.parametrize("layer", [0, 13, 26, 39])
def test_config_opt13b_layer_sampled_units(sh, layer):
    """One layer's handle of the 40-layer workload at full size (1280 units per launch, the launch the
    benchmark times), 16 sampled units in lockstep through prompt and decode.  Layers differ only in the
    seed of their input stream and each has a handle of its own, so four of them sample the forty."""
    cfg = wl.CONFIGS["opt13b"]
    st = wl.Stream(cfg, device="cuda", layer=layer)
    units = wl.sample_units(cfg, 16)
    h = sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False)
    res, _ = run_lockstep(h, cfg.dtype, st.step, cfg.total_steps, units, TOL[cfg.dtype], state_every=64)
    assert res.compressions == 13


# ---- pieces -----------------------------------------------------------------------------------
def _select_cases(rng, n):
    yield "uniform", rng.integers(0, 129, size=n)
    yield "all_equal", np.full(n, 7)
    yield "two_valued", rng.integers(0, 2, size=n) * 50
    yield "ascending", np.sort(rng.integers(0, 400, size=n))
    yield "descending", np.sort(rng.integers(0, 400, size=n))[::-1].copy()
    yield "zeros", np.zeros(n, dtype=np.int64)
    yield "large", rng.integers(16000, 16385, size=n)


@pytest.mark.parametrize("n,r,m", [(410, 64, 64), (410, 0, 1), (410, 0, 410), (512, 128, 384), (37, 5, 11),
                                   (1, 0, 1), (1000, 999, 1), (4097, 100, 2000)])
def test_select_kernel_bit_exact_on_oracle_records(sh, n, r, m):
    rng = np.random.default_rng(n * 31 + m)
    names, rows = zip(*_select_cases(rng, n))
    I = np.stack(rows).astype(np.int32)
    # "exactly m above the cut": m large values, the rest tied below
    extra = np.zeros(n, dtype=np.int32)
    if n - r >= m:
        extra[rng.choice(n - r, size=m, replace=False)] = 9
    I = np.concatenate([I, extra[None]], axis=0)
    got = sh.select(torch.from_numpy(I).cuda(), r, m).cpu().numpy()
    for i in range(I.shape[0]):
        want = oracle.select(I[i], r, m)
        assert (got[i] == want).all(), f"case {i}"


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16", "int4"])
@pytest.mark.parametrize("stable", [False, True])
def test_compaction_moves_rows_bit_identically(sh, dtype, stable):
    """Stored key and value rows after several compressions equal the oracle's bit for bit, on a handle in
    lockstep with the oracle; and a second handle that compresses by itself (SH_OPT_AUTO_COMPRESS, the
    default) ends bit-identical to the first, outputs included."""
    U, d, B, r, w, m, T = 4, 128, 96, 8, 20, 40, 200
    q, k, v = wl.random_stream(U, d, T, seed=3, dtype=dtype, peaked=3.0, device="cuda")
    auto = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=True, unordered=not stable)
    outs = torch.stack([auto.decode_step(q[t], k[t], v[t]) for t in range(T)])
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=not stable)
    twin_outs = []
    res, orc = run_lockstep(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype], outs=twin_outs)
    assert res.compressions >= 3
    n, by_pos = h.n, SortedView(h)
    for u in range(U):
        K, V = by_pos.export_unit(u)
        oK, oV = orc.cache(u)
        assert (K[:n].astype(np.float64) == oK).all() and (V[:n].astype(np.float64) == oV).all()
    assert torch.equal(outs, torch.stack(twin_outs))
    assert_same_state(auto, h)


# ---- SH_OPT_COMPACTION = 1: holes filled from the tail, slots in no particular order -------------
@pytest.mark.parametrize("dtype,d,kernel", [("f32", 64, None), ("f16", 128, None), ("bf16", 128, 2), ("int4", 128, None),
                                             ("f16", 64, 1)])
@pytest.mark.parametrize("U,B,r,w,m", [(5, 150, 9, 37, 41), (3, 700, 5, 64, 300), (4, 96, 0, 20, 1), (2, 64, 63, 5, 1),
                                       (3, 33, 0, 1, 33), (2, 1100, 10, 400, 550), (2, 2400, 10, 1, 1200),
                                       (2, 3000, 10, 400, 1500), (3, 130, 7, 40, 1)])
def test_lockstep_unordered_compaction(sh, dtype, d, kernel, U, B, r, w, m):
    """Same protocol as the ordered mode; the library's slots are read back in position order.
    The shape with w = 1 (counters of 0 or 1) has tie classes beyond the shared-memory list of the
    selection kernel; the last one is too large for the fused single-launch compression and takes the
    selection + hole-filling pair; the others run fused."""
    T = min(2 * B + 4 * m + 9, 2 * B + 300) if B < 2000 else B + m + 20
    q, k, v = wl.random_stream(U, d, T, seed=71 + B, dtype=dtype, peaked=3.0, device="cuda")
    h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, kernel=kernel, unordered=True))
    res, _ = run_lockstep(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 2
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("U,B,r,w,m,sizes", [(5, 150, 9, 37, 41, [64, 7, 33, 1, 50]), (3, 410, 64, 128, 64, [64]),
                                             (130, 96, 8, 70, 30, [64, 31])])
def test_lockstep_unordered_chunked_prompt(sh, U, B, r, w, m, sizes):
    dtype, d, T = "f16", 128, 2 * B + 2 * m + 11
    q, k, v = wl.random_stream(U, d, T, seed=19 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=True))
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype], chunk_sizes=sizes)
    assert res.steps == T and res.compressions >= 3
    q2, k2, v2 = wl.random_stream(U, d, 40, seed=98, dtype=dtype, peaked=3.0, device="cuda")
    run_lockstep(h, dtype, lambda t: (q2[t - T - 1], k2[t - T - 1], v2[t - T - 1]), 40, torch.arange(U), TOL[dtype], orc=orc)


@pytest.mark.parametrize("U,B,r,w,m", [(5, 150, 9, 37, 41), (3, 410, 64, 128, 64), (140, 96, 8, 70, 30)])
def test_lockstep_unordered_record_recomputed(sh, U, B, r, w, m):
    dtype, d, T = "bf16", 128, 2 * B + 3 * m + 5
    q, k, v = wl.random_stream(U, d, T, seed=29 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, recompute_record=True, unordered=True))
    res, orc = run_lockstep_recompute(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 4


def test_unordered_compaction_moves_at_most_m_rows_and_keeps_them_bit_identical(sh):
    """Rows that stay are not touched: a slot below n - m that survives a compression holds the same
    token before and after; and every kept token's key and value rows equal the oracle's."""
    U, d, B, r, w, m, T, dtype = 4, 128, 96, 8, 20, 40, 200, "f16"
    q, k, v = wl.random_stream(U, d, T, seed=3, dtype=dtype, peaked=3.0, device="cuda")
    raw = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=True)
    h = SortedView(raw)
    orc = oracle.Oracle(U, B, r, w, m, d)
    idx = torch.arange(U, device="cuda")
    for t in range(T):
        h.decode_step(q[t], k[t], v[t])
        out, alpha, low, amb = orc.attend(to_oracle(q[t], idx), to_oracle(k[t], idx), to_oracle(v[t], idx))
        glow = h.state()[4]
        orc.record(glow if not ((glow != low) & ~amb).any() else low)
        if orc.full:
            before = raw.state(counters=False, low=False)[2].copy()
            orc.compress()
            assert raw.compress() == m
            n2, _, after, _, _ = raw.state(counters=False, low=False)
            assert n2 == B - m
            for u in range(U):
                head = before[u, : B - m]
                kept = np.isin(head, orc.positions()[u])
                assert (after[u][kept] == head[kept]).all()          # survivors in the head did not move
            assert (np.sort(after, axis=1) == orc.positions()).all()
    n = h.n
    for u in range(U):
        K, V = h.export_unit(u)
        oK, oV = orc.cache(u)
        assert (K[:n].astype(np.float64) == oK).all() and (V[:n].astype(np.float64) == oV).all()


def test_prefill_equals_token_by_token_steps(sh):
    U, d, B, r, w, m, T, dtype = 6, 128, 80, 8, 24, 30, 260, "f16"
    q, k, v = wl.random_stream(U, d, T, seed=5, dtype=dtype, peaked=3.0, device="cuda")
    a = sh.Handle(B, r, w, m, U, d, dtype, prefill_chunk=False)    # one decode step per prompt token
    b = sh.Handle(B, r, w, m, U, d, dtype)
    out_a = torch.empty(T, U, d, device="cuda")
    a.prefill(q, k, v, out_a)
    out_b = torch.stack([b.decode_step(q[t], k[t], v[t]) for t in range(T)])
    assert torch.equal(out_a, out_b)
    sa, sb = a.state(), b.state()
    assert sa[0] == sb[0] and sa[1] == sb[1] == T
    for x, y in zip(sa[2:], sb[2:]):
        assert (x == y).all()
    assert torch.equal(a.slab[a._slab_off:a._slab_off + 2 * U * B * d * 2], b.slab[b._slab_off:b._slab_off + 2 * U * B * d * 2])


@pytest.mark.parametrize("pinned,U", [(True, 7), (False, 7), (True, 2400)])
def test_host_buffer_step_matches_device_step(sh, pinned, U):
    """sh_decode_step_host against sh_decode_step, bit for bit; 2400 units run the many-units shape of the
    decode kernel on host-resident inputs."""
    d, B, r, w, m, T, dtype = 128, 64, 4, 16, 20, 100, "bf16"
    q, k, v = wl.random_stream(U, d, T, seed=6, dtype=dtype, peaked=2.0, device="cuda")
    a = sh.Handle(B, r, w, m, U, d, dtype)
    b = sh.Handle(B, r, w, m, U, d, dtype)
    pin = (lambda x: x.pin_memory()) if pinned else (lambda x: x)
    qh, kh, vh = (pin(x.cpu()) for x in (q, k, v))
    oh = pin(torch.empty(U, d))
    for t in range(T):
        oa = a.decode_step(q[t], k[t], v[t])
        b.decode_step_host(qh[t], kh[t], vh[t], oh)
        assert torch.equal(oa.cpu(), oh)
    for x, y in zip(a.state()[2:], b.state()[2:]):
        assert (x == y).all()


def test_snapshot_restore_replays_identically(sh):
    U, d, B, r, w, m, dtype = 4, 64, 48, 4, 12, 16, "f32"
    q, k, v = wl.random_stream(U, d, 150, seed=8, dtype=dtype, peaked=2.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype)
    for t in range(70):
        h.decode_step(q[t], k[t], v[t])
    snap = h.snapshot()
    first = [h.decode_step(q[t], k[t], v[t]).clone() for t in range(70, 150)]
    s1 = h.state()
    h.restore(snap)
    second = [h.decode_step(q[t], k[t], v[t]).clone() for t in range(70, 150)]
    s2 = h.state()
    assert all(torch.equal(x, y) for x, y in zip(first, second))
    assert s1[0] == s2[0] and s1[1] == s2[1] and all((x == y).all() for x, y in zip(s1[2:], s2[2:]))


def _ragged_lockstep(sh, dtype, d, lengths, ups, B, r, w, m, T_dec, kernel, unordered, split, seed):
    """Sequences of different prompt lengths in one handle (sh_prefill_ragged), then decode steps in
    lockstep: one oracle per sequence, each with its own n, t and compression schedule.  Returns the
    number of steps at which some sequence compressed."""
    nseq = len(lengths)
    U, p_max = nseq * ups, max(lengths)
    q, k, v = wl.random_stream(U, d, p_max + T_dec, seed=seed, dtype=dtype, peaked=3.0, device="cuda")
    kw = dict(auto_compress=False, kernel=kernel, unordered=unordered, split=split)
    raw = sh.Handle(B, r, w, m, U, d, dtype, **kw)
    h = SortedView(raw)
    out_p = torch.zeros(p_max, U, d, device="cuda")
    h.prefill_ragged(q[:p_max].contiguous(), k[:p_max].contiguous(), v[:p_max].contiguous(), lengths, out_p)
    # The prompt of each sequence once more, on a handle of its own that is driven through the same launches
    # by hand in lockstep with an oracle (adoption inside the 1e-6 window); the ragged handle's units of that
    # sequence must then hold bit-identical state, which ties every one of them to the oracle.
    orcs = []
    pos_r, cnt_r, low_r = raw.state_full()
    quant = dtype == "int4"
    for sq in range(nseq):
        sl = slice(sq * ups, (sq + 1) * ups)
        twin_raw = sh.Handle(B, r, w, m, ups, d, dtype, **kw)
        twin = SortedView(twin_raw)
        qs, ks, vs = (x[:, sl].contiguous() for x in (q, k, v))
        t_outs = []
        if lengths[sq] == 0:
            o = oracle.Oracle(ups, B, r, w, m, d, quant=quant)
        elif twin_raw.prefill_chunk_max >= 2:
            blk = lambda t0, t1: (qs[t0 - 1:t1 - 1].contiguous(), ks[t0 - 1:t1 - 1].contiguous(), vs[t0 - 1:t1 - 1].contiguous())
            _, o = run_lockstep_chunked(twin, dtype, blk, lengths[sq], torch.arange(ups), TOL[dtype], outs=t_outs,
                                        single_via_step=True)
        else:
            _, o = run_lockstep(twin, dtype, _stream_fn(qs, ks, vs), lengths[sq], torch.arange(ups), TOL[dtype], outs=t_outs)
            t_outs = [x[None] for x in t_outs]
        if lengths[sq]:
            assert torch.equal(out_p[: lengths[sq], sl], torch.cat(t_outs))
        pos_t, cnt_t, low_t = twin_raw.state_full()
        assert (pos_r[sl] == pos_t).all() and (cnt_r[sl] == cnt_t).all() and (low_r[sl] == low_t).all()
        for j in sorted(set(range(0, ups, 37)) | {ups - 1}):
            Kr, Vr = raw.export_unit(sq * ups + j)
            Kt, Vt = twin_raw.export_unit(j)
            assert (Kr[: o.n] == Kt[: o.n]).all() and (Vr[: o.n] == Vt[: o.n]).all()
        orcs.append(o)
    n_seq, t_seq = h.sequence_state()
    assert n_seq.tolist() == [o.n for o in orcs] and t_seq.tolist() == list(lengths)
    pos, cnt, _ = h.state_full()
    for sq, o in enumerate(orcs):
        sl = slice(sq * ups, (sq + 1) * ups)
        assert (pos[sl, : o.n] == o.positions()).all() and (cnt[sl, : o.n].astype(np.int32) == o.counters()).all()
        assert (pos[sl, o.n:] == 0).all()
    compressions = 0
    for step in range(T_dec):
        ti = p_max + step
        out = h.decode_step(q[ti], k[ti], v[ti])
        pos, cnt, low = h.state_full()
        for sq, o in enumerate(orcs):
            idx = torch.arange(sq * ups, (sq + 1) * ups, device="cuda")
            sl = slice(sq * ups, (sq + 1) * ups)
            oo, alpha, o_low, amb = o.attend(to_oracle(q[ti], idx), to_oracle(k[ti], idx), to_oracle(v[ti], idx))
            assert np.abs(out[idx].double().cpu().numpy() - oo).max() <= TOL[dtype]
            g_low = low[sl, : o.n]
            assert not low[sl, o.n:].any()
            diff = g_low != o_low
            assert not (diff & ~amb).any(), f"sequence {sq}, step {step}: record bits differ outside the 1e-6 window"
            o.record(g_low)
            assert (pos[sl, : o.n] == o.positions()).all() and (cnt[sl, : o.n].astype(np.int32) == o.counters()).all()
        n_seq, t_seq = h.sequence_state()
        due = [sq for sq in range(nseq) if n_seq[sq] == B]
        assert h.compress() == (m if due else 0)
        if due:
            compressions += 1
            pos, cnt, _ = h.state_full()
            for sq in due:
                o = orcs[sq]
                assert o.full
                o.compress()
                sl = slice(sq * ups, (sq + 1) * ups)
                assert (pos[sl, : o.n] == o.positions()).all() and (pos[sl, o.n:] == 0).all()
                assert (cnt[sl, : o.n].astype(np.int32) == o.counters()).all()
        n_seq, t_seq = h.sequence_state()
        assert all(n_seq[sq] == orcs[sq].n for sq in range(nseq))
        assert t_seq.tolist() == [lengths[sq] + step + 1 for sq in range(nseq)]
    return compressions


@pytest.mark.parametrize("dtype,kernel,unordered", [("f16", None, False), ("bf16", 2, False), ("f16", 1, False),
                                                    ("f32", None, False), ("f16", None, True), ("bf16", 2, True)])
def test_ragged_sequences_lockstep(sh, dtype, kernel, unordered):
    d = 128 if dtype != "f32" else 64
    lengths = [0, 37, 150, 96, 211, 95]            # empty, short, several compressions, exactly full, long, one short of full
    compressions = _ragged_lockstep(sh, dtype, d, lengths, ups=3, B=96, r=8, w=40, m=30, T_dec=170, kernel=kernel,
                                    unordered=unordered, split=2, seed=51)
    assert compressions >= 12                    # the sequences fill at different steps


@pytest.mark.parametrize("dtype", ["f16", "int4"])
def test_ragged_sequences_many_units(sh, dtype):
    """Ragged sequences on the many-units shape of the direct decode kernel (600 units: per-unit row counts
    read and advanced on the device by 4-warp CTAs), every unit in lockstep."""
    compressions = _ragged_lockstep(sh, dtype, 128, [3, 41], ups=300, B=48, r=4, w=12, m=16, T_dec=40, kernel=1,
                                    unordered=False, split=None, seed=57)
    assert compressions >= 3


def test_persistence_diagnostics_match_oracle_scores(sh):
    """Persistence ratio and pivotal-set size (Section 3.2) from the library's record bits, against
    the same quantities from the oracle's fp64 scores on a full (never compressed) cache."""
    from paper_2305_17118_b200 import diagnostics
    l, U, d, dtype = 96, 6, 128, "f16"
    q, k, v = wl.random_stream(U, d, l, seed=41, dtype=dtype, peaked=3.0, device="cuda")
    got = diagnostics.persistence(q, k, v, dtype)
    orc = oracle.Oracle(U, l + 1, 0, l, 1, d)
    idx = torch.arange(U, device="cuda")
    piv = np.zeros((U, l, l), dtype=bool)
    amb_any = np.zeros(U, dtype=bool)
    for s in range(l):
        _o, alpha, low, amb = orc.attend(to_oracle(q[s], idx), to_oracle(k[s], idx), to_oracle(v[s], idx))
        orc.record(low)
        piv[:, s, : s + 1] = ~low
        if s > 0:                                      # at the first step alpha = 1 = 1/t exactly, on both sides
            amb_any |= amb.any(axis=1)
    t = l // 2
    assert got.t == t and got.l == l
    for u in range(U):
        if amb_any[u]:
            continue                                   # a score within 1e-6 of 1/t may legitimately flip
        first, later = piv[u, :t, :t].any(axis=0), piv[u, t:, :t].any(axis=0)
        want = (first & later).sum() / later.sum() if later.any() else np.nan
        assert (np.isnan(want) and np.isnan(got.ratio[u])) or abs(got.ratio[u] - want) < 1e-12
        assert abs(got.pivotal_frac[u] - first.sum() / t) < 1e-12
    assert (~amb_any).sum() >= U - 1
    assert np.nanmin(got.ratio) >= 0 and np.nanmax(got.ratio) <= 1


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("f16", 128), ("bf16", 64), ("int4", 128)])
@pytest.mark.parametrize("unordered", [False, True])
def test_scores_entry_point_matches_oracle_scores(sh, dtype, d, unordered):
    """sh_scores against the oracle's fp64 alpha of the same step, on caches that have been through
    several compressions, at several fill levels (n not a multiple of anything)."""
    U, B, r, w, m, T = 5, 150, 9, 37, 41, 330
    q, k, v = wl.random_stream(U, d, T + 1, seed=83, dtype=dtype, peaked=3.0, device="cuda")
    h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=unordered))
    _, orc = run_lockstep(h, dtype, _stream_fn(q, k, v), T - 3, torch.arange(U), TOL[dtype])
    idx = torch.arange(U, device="cuda")
    for t in range(T - 3, T):
        h.decode_step(q[t], k[t], v[t])
        got = h.scores(q[t]).cpu().numpy().astype(np.float64)
        n, _, pos, _, low = h.state(counters=False)
        _o, alpha, o_low, amb = orc.attend(to_oracle(q[t], idx), to_oracle(k[t], idx), to_oracle(v[t], idx))
        assert not ((low != o_low) & ~amb).any()
        orc.record(low)
        assert n == orc.n and (pos == orc.positions()).all()
        raw_pos = h._h.state(counters=False, low=False)[2]
        by_pos = np.take_along_axis(got[:, :n], np.argsort(raw_pos, axis=1), axis=1)      # slot order -> position order
        assert np.abs(by_pos - alpha).max() <= 2e-5 * alpha.max() + 1e-9
        assert (np.abs(by_pos - alpha) <= 1e-4 * alpha + 1e-9).all()
        assert (got[:, n:] == 0).all() and abs(got.sum(axis=1) - 1).max() < 1e-5
        assert not orc.full


def test_scores_on_ragged_sequences_and_after_restore(sh):
    """sh_scores reads each unit's own row count (ragged handle), and a snapshot of an unordered handle
    replays identically after sh_restore."""
    dtype, d = "f16", 128
    lengths = [5, 40, 17]
    ups, B, r, w, m = 2, 48, 4, 12, 16
    U, p_max = len(lengths) * ups, max(lengths)
    q, k, v = wl.random_stream(U, d, p_max + 1, seed=91, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, unordered=True)
    h.prefill_ragged(q[:p_max].contiguous(), k[:p_max].contiguous(), v[:p_max].contiguous(), lengths)
    n_seq, _ = h.sequence_state()
    got = h.scores(q[p_max]).cpu().numpy().astype(np.float64)
    for sq, L in enumerate(lengths):
        o = oracle.Oracle(ups, B, r, w, m, d)
        idx = torch.arange(sq * ups, (sq + 1) * ups, device="cuda")
        for t in range(L):
            o.step(to_oracle(q[t], idx), to_oracle(k[t], idx), to_oracle(v[t], idx))
        assert n_seq[sq] == o.n
        qf = to_oracle(q[p_max], idx)
        for j, u in enumerate(range(sq * ups, (sq + 1) * ups)):
            K, _ = o.cache(j)
            z = K @ qf[j] / math.sqrt(d)
            e = np.exp(z - z.max())
            want = np.sort(e / e.sum())
            assert np.abs(np.sort(got[u, : o.n]) - want).max() <= 1e-4 * want.max() + 1e-9     # same multiset of scores
            assert (got[u, o.n:] == 0).all()
    # snapshot / restore on a uniform unordered handle
    U2 = 4
    q2, k2, v2 = wl.random_stream(U2, d, 150, seed=92, dtype=dtype, peaked=2.0, device="cuda")
    g = sh.Handle(B, r, w, m, U2, d, dtype, unordered=True)
    for t in range(70):
        g.decode_step(q2[t], k2[t], v2[t])
    snap = g.snapshot()
    first = [g.decode_step(q2[t], k2[t], v2[t]).clone() for t in range(70, 150)]
    s1 = g.state()
    g.restore(snap)
    second = [g.decode_step(q2[t], k2[t], v2[t]).clone() for t in range(70, 150)]
    s2 = g.state()
    assert all(torch.equal(x, y) for x, y in zip(first, second))
    assert s1[0] == s2[0] and s1[1] == s2[1] and all((x == y).all() for x, y in zip(s1[2:], s2[2:]))


def test_score_change_ratio_diagnostic(sh):
    """(alpha_s - alpha_o) / alpha_o of the last step's query, budgeted cache against full cache, from
    the library; the same from two oracles' caches with the softmax written out here.  The budgeted
    oracle is brought along in lockstep with a twin handle fed through the same launches as the
    diagnostic's own (adoption inside the 1e-6 window), so every unit is compared."""
    from paper_2305_17118_b200 import diagnostics
    U, d, B, r, w, m, t, dtype = 8, 128, 64, 6, 24, 20, 173, "f16"
    q, k, v = wl.random_stream(U, d, t, seed=87, dtype=dtype, peaked=3.0, device="cuda")
    got = diagnostics.score_change_ratio(q, k, v, dtype, B, r, w, m)
    twin = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    _, o_s = run_lockstep_chunked(twin, dtype, blk, t, torch.arange(U), TOL[dtype], single_via_step=True)
    o_o = oracle.Oracle(U, t + 1, 0, 1, 1, d)
    idx = torch.arange(U, device="cuda")
    for s in range(t):
        o_o.step(to_oracle(q[s], idx), to_oracle(k[s], idx), to_oracle(v[s], idx))
    qf = to_oracle(q[t - 1], idx)
    for u in range(U):
        def scores(o):
            K, _ = o.cache(u)
            z = K @ qf[u] / math.sqrt(d)
            e = np.exp(z - z.max())
            return e / e.sum()
        pos_s = o_s.positions()[u]
        assert got.kept[u].sum() == len(pos_s) and got.kept[u][pos_s - 1].all()
        want = np.full(t, -1.0)
        a_o = scores(o_o)
        want[pos_s - 1] = (scores(o_s) - a_o[pos_s - 1]) / a_o[pos_s - 1]
        assert np.abs(got.ratio[u] - want).max() <= 2e-4
        assert (got.ratio[u][~got.kept[u]] == -1).all() and (got.ratio[u][got.kept[u]] >= -1e-4).all()


@pytest.mark.parametrize("B,w,m", [(8192, 48, 4096), (2048, 16384, 1024)])
def test_large_budget_lockstep(sh, B, w, m):
    """B = 8192: every kernel's large-size path (many key tiles, 256 record words per bit-plane row,
    selection from global memory); w = 16384: the longest history window the library takes.  Both in
    lockstep with the oracle through two compressions."""
    U, d, r, dtype = 1, 64, 10, "f16"
    T = B + m + 12
    q, k, v = wl.random_stream(U, d, T, seed=101, dtype=dtype, peaked=2.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    res, _ = run_lockstep(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype], state_every=2048)
    assert res.compressions == 2


@pytest.mark.parametrize("unordered", [False, True])
def test_maximum_budget_properties(sh, unordered):
    """The largest budget the library takes (B = 32768) with the longest window that fits the test
    (w = 2048): the prompt goes through the chunk kernel, the cache fills, one compression drops
    m = 16384 tokens.  The oracle would need minutes here, so the check is by properties that hold at
    any size, plus one step's attention output and scores against the plain definition (softmax of
    q.K / sqrt(d), then times V) evaluated in fp64 on the rows the library exports."""
    U, d, B, r, w, m, dtype = 1, 128, 32768, 100, 2048, 16384, "f16"
    T = B - 1
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=unordered)
    blk = 4096
    for t0 in range(0, T, blk):
        n_tok = min(blk, T - t0)
        x = (torch.randn(3, n_tok, U, d, generator=g, device="cuda") * 0.7).to(torch.float16)
        h.prefill(x[0], x[1], x[2])
    assert h.n == B - 1
    x = (torch.randn(3, U, d, generator=g, device="cuda") * 0.7).to(torch.float16)
    out = h.decode_step(x[0], x[1], x[2])
    n, t, pos, cnt, low = h.state()
    assert n == B and t == B and (pos[0] == np.arange(1, B + 1)).all()
    assert cnt.max() <= w and (cnt[0, -1] <= 1)
    K, V = h.export_unit(0)
    z = K.astype(np.float64) @ x[0][0].double().cpu().numpy() / math.sqrt(d)
    e = np.exp(z - z.max())
    alpha = e / e.sum()
    assert np.abs(out[0].double().cpu().numpy() - alpha @ V.astype(np.float64)).max() <= TOL[dtype]
    got_alpha = h.scores(x[0]).cpu().numpy().astype(np.float64)[0]
    assert np.abs(got_alpha - alpha).max() <= 1e-4 * alpha.max() + 1e-9
    amb = np.abs(alpha - 1.0 / t) <= 1e-6
    assert ((low[0] == (alpha < 1.0 / t)) | amb).all()          # this step's record bits
    # compression: m tokens go, none of the r newest, the survivors keep position, counter and rows
    assert h.compress() == m
    n2, _, pos2, cnt2, _ = h.state(low=False)
    assert n2 == B - m and len(set(pos2[0].tolist())) == n2
    assert set(range(B - r + 1, B + 1)) <= set(pos2[0].tolist())
    if not unordered:
        assert (np.diff(pos2[0]) > 0).all()
    assert (cnt2[0] == cnt[0][pos2[0] - 1]).all()
    dropped = np.setdiff1d(np.arange(1, B + 1), pos2[0])
    cand = np.arange(1, B - r + 1)
    kept_cand = np.setdiff1d(cand, dropped)
    assert cnt[0][dropped - 1].min() >= cnt[0][kept_cand - 1].max()      # the m largest counters went
    tie = cnt[0][dropped - 1].min()
    tie_kept = kept_cand[cnt[0][kept_cand - 1] == tie]
    tie_dropped = dropped[cnt[0][dropped - 1] == tie]
    assert len(tie_kept) == 0 or tie_dropped.max() < tie_kept.min()      # oldest first among equals
    K2, V2 = h.export_unit(0)
    assert (K2[:n2] == K[pos2[0] - 1]).all() and (V2[:n2] == V[pos2[0] - 1]).all()


def test_error_codes(sh):
    import ctypes as C
    lib = sh.lib
    h = C.c_void_p()
    assert lib.sh_create(8, 4, 2, 5, 1, 64, sh.SH_F16, C.byref(h)) == sh.SH_EINVAL      # m > B - r
    assert lib.sh_create(8, 1, 2, 2, 1, 96, sh.SH_F16, C.byref(h)) == sh.SH_EINVAL      # head_dim
    assert lib.sh_create(8, 1, 2, 2, 1, 64, 9, C.byref(h)) == sh.SH_EINVAL              # dtype
    assert lib.sh_create(8, 1, 2, 2, 1, 64, sh.SH_F16, C.byref(h)) == sh.SH_OK
    buf = torch.zeros(64, dtype=torch.float16, device="cuda")
    out = torch.zeros(64, device="cuda")
    assert lib.sh_decode_step(h, buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), out.data_ptr(), None) == sh.SH_ESTATE
    lib.sh_destroy(h)
    hd = sh.Handle(4, 1, 2, 2, 1, 64, "f16", auto_compress=False)
    for _ in range(4):
        hd.decode_step(buf.view(1, 64), buf.view(1, 64), buf.view(1, 64))
    with pytest.raises(sh.ShError) as ei:
        hd.decode_step(buf.view(1, 64), buf.view(1, 64), buf.view(1, 64))
    assert ei.value.status == sh.SH_EFULL
    assert hd.compress() == 2 and hd.n == 2
    assert hd.compress() == 0
    with pytest.raises(sh.ShError):
        hd.set_option(sh.SH_OPT_SPLIT, 2)    # options are frozen after the first step
    assert lib.sh_decode_step(hd._h, None, buf.data_ptr(), buf.data_ptr(), out.data_ptr(), None) == sh.SH_EINVAL
    assert lib.sh_decode_step(hd._h, buf.data_ptr() + 2, buf.data_ptr(), buf.data_ptr(), out.data_ptr(), None) == sh.SH_EINVAL


def test_bounded_wait_gives_up_and_reports_device_error(sh):
    """The give-up path of the kernels' bounded waits, made to happen without faulting anything: with
    SH_OPT_SELFTEST_SKIP_TILE the first CTA of the pipelined decode kernel never requests one of its tiles
    (no copy is in flight for it), so the wait for that tile runs out after about a second.  The kernel
    must end by itself, sh_state must say SH_EDEVICE from then on, later calls on the handle must return
    normally, and a fresh handle on the same device must work."""
    import ctypes as C
    import time
    U, d, B, r, w, m, dtype = 5, 128, 300, 4, 16, 100, "f16"
    q, k, v = wl.random_stream(U, d, 200, seed=77, dtype=dtype, peaked=2.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, kernel=2, auto_compress=False)
    h.set_option(sh.SH_OPT_SELFTEST_SKIP_TILE, 1)      # the second tile CTA 0 would stream in a launch
    for t in range(129):                               # up to 128 cached rows a unit is a single tile: nothing is skipped
        h.decode_step(q[t], k[t], v[t])
    assert sh.lib.sh_state(h._h, None, None, None, None, None, None) == sh.SH_OK
    t0 = time.time()
    h.decode_step(q[129], k[129], v[129])              # 129 cached rows: two tiles, the second never arrives
    rc = sh.lib.sh_state(h._h, None, None, None, None, None, None)
    took = time.time() - t0
    assert rc == sh.SH_EDEVICE and took < 20.0
    assert b"bounded wait" in sh.lib.sh_strerror(rc)
    n, t = C.c_int(0), C.c_longlong(0)
    assert sh.lib.sh_state(h._h, None, C.byref(n), C.byref(t), None, None, None) == sh.SH_EDEVICE     # sticky
    assert n.value == 130 and t.value == 130
    out = torch.empty(U, d, device="cuda")
    assert sh.lib.sh_decode_step(h._h, q[130].data_ptr(), k[130].data_ptr(), v[130].data_ptr(), out.data_ptr(), None) == sh.SH_OK
    assert sh.lib.sh_state(h._h, None, None, None, None, None, None) == sh.SH_EDEVICE
    torch.cuda.synchronize()
    # the device and the library are fine: a fresh handle runs in lockstep with the oracle
    g = sh.Handle(B, r, w, m, U, d, dtype, kernel=2, auto_compress=False)
    res, _ = run_lockstep(g, dtype, _stream_fn(q, k, v), 200, torch.arange(U), TOL[dtype])
    assert res.steps == 200


@pytest.mark.parametrize("skip", [0, 1])
def test_bounded_wait_gives_up_in_the_chunk_kernel(sh, skip):
    """The same self-test on the persistent tcgen05 chunk kernel: its first CTA never requests one key tile (tile 0:
    the first sweep's, so the softmax warps leave before the barriers that end the first sweep and have to
    release one another there; tile 1: the second sweep's).  The MMA-issuing thread, the copy threads and the
    softmax warps must all give up by themselves within seconds, tensor memory must be released (a fresh handle's
    chunk kernel allocates it again), and sh_state must report SH_EDEVICE."""
    import time
    U, d, B, r, w, m, dtype = 5, 128, 300, 4, 64, 100, "f16"
    q, k, v = wl.random_stream(U, d, 330, seed=79, dtype=dtype, peaked=2.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    h.set_option(sh.SH_OPT_SELFTEST_SKIP_TILE, skip)
    out = torch.empty(64, U, d, device="cuda")
    t0 = time.time()
    h.prefill_chunk(q[:64].contiguous(), k[:64].contiguous(), v[:64].contiguous(), out)     # one key tile, two sweeps
    rc = sh.lib.sh_state(h._h, None, None, None, None, None, None)
    took = time.time() - t0
    assert rc == sh.SH_EDEVICE and took < 30.0
    assert b"bounded wait" in sh.lib.sh_strerror(rc)
    torch.cuda.synchronize()
    g = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, _ = run_lockstep_chunked(g, dtype, blk, 330, torch.arange(U), TOL[dtype], chunk_sizes=[64, 20])
    assert res.steps == 330 and res.compressions >= 1


def test_restore_boundaries_and_output_alignment(sh):
    import ctypes as C
    U, d, B, r, w, m, dtype = 4, 64, 16, 2, 8, 6, "f16"
    q, k, v = wl.random_stream(U, d, 40, seed=78, dtype=dtype, device="cuda")
    # a snapshot taken at a full cache (manual compression) can be resumed: the next call is sh_compress
    a = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    b = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False)
    for t in range(B):
        a.decode_step(q[t], k[t], v[t])
        b.decode_step(q[t], k[t], v[t])
    snap = a.snapshot()
    assert snap[1] == B
    for t in range(B, 30):
        for h in (a, b):
            h.compress()
            h.decode_step(q[t], k[t], v[t])
    a.restore(snap)
    out = torch.empty(U, d, device="cuda")
    with pytest.raises(sh.ShError) as ei:
        a.decode_step(q[B], k[B], v[B], out)
    assert ei.value.status == sh.SH_EFULL
    for t in range(B, 30):
        a.compress()
        a.decode_step(q[t], k[t], v[t])
    assert_same_state(a, b)
    assert sh.lib.sh_restore(a._h, B + 1, 100) == sh.SH_EINVAL
    assert sh.lib.sh_restore(a._h, 5, 4) == sh.SH_EINVAL
    # once sequences differ in length one (n, t) pair cannot describe the handle
    rg = sh.Handle(B, r, w, m, U, d, dtype)
    rg.prefill_ragged(q[:9].contiguous(), k[:9].contiguous(), v[:9].contiguous(), [3, 9])
    assert sh.lib.sh_restore(rg._h, 3, 3) == sh.SH_ESTATE
    n_seq, t_seq = rg.sequence_state()
    assert n_seq.tolist() == [3, 9] and t_seq.tolist() == [3, 9]          # untouched
    rg.decode_step(q[9], k[9], v[9])
    assert rg.sequence_state()[0].tolist() == [4, 10]
    # the output pointer is checked like the inputs
    buf = torch.empty(U * d + 4, device="cuda")
    assert sh.lib.sh_decode_step(b._h, q[30].data_ptr(), k[30].data_ptr(), v[30].data_ptr(), buf.data_ptr() + 2, None) == sh.SH_EINVAL
    assert sh.lib.sh_decode_step(b._h, q[30].data_ptr(), k[30].data_ptr(), v[30].data_ptr(), buf.data_ptr() + 4, None) == sh.SH_OK


def test_select_at_its_size_limit(sh):
    n, r, m = sh.SH_SELECT_MAX_N, 1000, 300
    rng = np.random.default_rng(5)
    I = rng.integers(0, 16385, size=(2, n)).astype(np.int32)
    I[1] = rng.integers(0, 3, size=n)
    got = sh.select(torch.from_numpy(I).cuda(), r, m).cpu().numpy()
    for i in range(2):
        assert (got[i] == oracle.select(I[i], r, m)).all()
    big = torch.zeros(1, n + 1, dtype=torch.int16, device="cuda")
    out = torch.empty(1, m, dtype=torch.int32, device="cuda")
    assert sh.lib.sh_select(big.data_ptr(), 1, n + 1, r, m, out.data_ptr(), None) == sh.SH_EINVAL


def test_record_mode_overlap_diagnostic(sh):
    """Kept sets with the record kept online against the record recomputed at compression: both handles keep the
    recent window, so the overlap is at least r/n; each side's kept set is checked against an oracle running the
    same variant in lockstep with a twin handle, which makes the reported overlap the oracle's as well."""
    from paper_2305_17118_b200 import diagnostics
    U, d, B, r, w, m, t, dtype = 6, 128, 64, 6, 24, 20, 173, "f16"
    q, k, v = wl.random_stream(U, d, t, seed=88, dtype=dtype, peaked=3.0, device="cuda")
    got = diagnostics.record_mode_overlap(q, k, v, dtype, B, r, w, m)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    _, o_a = run_lockstep_chunked(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False), dtype, blk, t, torch.arange(U),
                                  TOL[dtype], single_via_step=True)
    _, o_b = run_lockstep_chunked(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, recompute_record=True), dtype, blk,
                                  t, torch.arange(U), TOL[dtype], single_via_step=True, recompute=True)
    pa, pb = o_a.positions(), o_b.positions()
    want = np.array([len(np.intersect1d(pa[u], pb[u])) for u in range(U)]) / o_a.n
    assert got.n == o_a.n == o_b.n and np.abs(got.overlap - want).max() < 1e-12
    assert (got.overlap >= r / got.n - 1e-12).all() and (got.overlap <= 1).all()


_BULK_STORES = [("f16", 128, False), ("bf16", 128, True), ("int4", 128, False), ("f32", 64, False)]
_BULK_SHAPES = [(300, 96, 8, 40, 30), (150, 150, 9, 37, 41), (90, 120, 4, 16, 20)]


# (the last shape drops one token per round, 570 rounds: one storage type is enough for it)
@pytest.mark.parametrize("dtype,d,stable,p,B,r,w,m", [st + sh_ for sh_ in _BULK_SHAPES for st in _BULK_STORES] +
                         [("f16", 128, False, 700, 130, 10, 200, 1)])
def test_bulk_prompt_reading_lockstep(sh, dtype, d, stable, p, B, r, w, m):
    """The prompting stage read as a bulk operation (sh_import_compressed / sh_prefill_bulk): the prompt is
    attended in full on a handle that never compresses, in lockstep with an oracle of the same budget;
    both sides then bring that cache under the real budget by rounds of Algorithm 2 on the record as it
    stands, and must hold the same tokens, records and rows; generation continues in lockstep.  The
    one-call form must end bit-identical to the composed one."""
    U, T_dec = 4, 80
    q, k, v = wl.random_stream(U, d, p + T_dec, seed=111 + p, dtype=dtype, peaked=3.0, device="cuda")
    kw = dict(auto_compress=False, unordered=not stable)
    src = sh.Handle(p + 1, 0, w, 1, U, d, dtype, **kw)
    o_src = oracle.Oracle(U, p + 1, 0, w, 1, d, quant=(dtype == "int4"))
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    outs = []
    if src.prefill_chunk_max >= 2:
        run_lockstep_chunked(src, dtype, blk, p, torch.arange(U), TOL[dtype], orc=o_src, outs=outs, single_via_step=True)
    else:
        run_lockstep(src, dtype, _stream_fn(q, k, v), p, torch.arange(U), TOL[dtype], orc=o_src, outs=outs)
        outs = [x[None] for x in outs]
    dst = sh.Handle(B, r, w, m, U, d, dtype, **kw)
    dst.import_compressed(src)
    o_dst = oracle.Oracle(U, B, r, w, m, d, quant=(dtype == "int4"))
    rounds = o_dst.import_compressed(o_src)
    assert rounds == (0 if p < B else (p - B) // m + 1)
    view = SortedView(dst)
    n, t, pos, cnt, _ = view.state(low=False)
    assert n == o_dst.n == p - rounds * m and t == o_dst.t == p
    assert (pos == o_dst.positions()).all() and (cnt.astype(np.int32) == o_dst.counters()).all()
    for u in range(U):
        K, V = view.export_unit(u)
        oK, oV = o_dst.cache(u)
        assert (K[:n].astype(np.float64) == oK).all() and (V[:n].astype(np.float64) == oV).all()
    one = sh.Handle(B, r, w, m, U, d, dtype, **kw)
    out1 = torch.empty(p, U, d, device="cuda")
    one.prefill_bulk(q[:p].contiguous(), k[:p].contiguous(), v[:p].contiguous(), out1)
    assert torch.equal(out1, torch.cat(outs))
    sa, sb = one.state(), dst.state()
    assert sa[0] == sb[0] and sa[1] == sb[1] and all((x == y).all() for x, y in zip(sa[2:], sb[2:]))
    res, _ = run_lockstep(dst, dtype, lambda tt: (q[tt - 1], k[tt - 1], v[tt - 1]), T_dec, torch.arange(U), TOL[dtype], orc=o_dst)
    assert res.steps == T_dec
    with pytest.raises(sh.ShError):
        dst.import_compressed(src)                     # the target must be fresh


_SIMT_SHAPES = [("f32", 64, None), ("f32", 128, None), ("f16", 64, None), ("bf16", 64, None), ("int4", 64, None),
                ("f16", 128, 4), ("bf16", 128, 4), ("int4", 128, 4)]


@pytest.mark.parametrize("dtype,d,mode", _SIMT_SHAPES)
@pytest.mark.parametrize("U,B,r,w,m,sizes", [(5, 150, 9, 37, 41, [64, 7, 33, 1, 50]), (3, 410, 64, 128, 64, [64]),
                                             (130, 96, 8, 70, 30, [64, 31]), (2, 1300, 10, 64, 650, [64, 13]),
                                             (4, 40, 3, 9, 20, [5, 9, 2])])
def test_lockstep_chunked_cuda_core_kernel(sh, dtype, d, mode, U, B, r, w, m, sizes):
    """The CUDA-core chunk kernel: the storage types and head sizes the tensor-core kernels do not take
    (fp32 rows, head_dim 64), and the others when forced (SH_OPT_PREFILL_CHUNK = 4).  Every step's output,
    record bits, positions, counters and kept sets against the oracle; int4 rows bit-identical; then
    decode steps from the state the chunks left."""
    T = min(2 * B + 2 * m + 11, B + 2 * m + 60)
    q, k, v = wl.random_stream(U, d, T + 30, seed=47 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = SortedView(sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, prefill_chunk=mode))
    assert h.prefill_chunk_max == min(64, w)
    blk = lambda t0, t1: (q[t0 - 1:t1 - 1].contiguous(), k[t0 - 1:t1 - 1].contiguous(), v[t0 - 1:t1 - 1].contiguous())
    res, orc = run_lockstep_chunked(h, dtype, blk, T, torch.arange(U), TOL[dtype], chunk_sizes=sizes)
    assert res.steps == T and res.compressions >= 2
    assert res.adoptions <= 1e-4 * res.slot_steps + 2
    if dtype == "int4":
        n = h.n
        for u in (0, U - 1):
            K, V = h.export_unit(u)
            oK, oV = orc.cache(u)
            assert (K[:n].astype(np.float64) == oK).all() and (V[:n].astype(np.float64) == oV).all()
    run_lockstep(h, dtype, _stream_fn(q, k, v), 30, torch.arange(U), TOL[dtype], orc=orc)


@pytest.mark.parametrize("dtype,d,mode", _SIMT_SHAPES)
@pytest.mark.parametrize("U,B,r,w,m", [(5, 150, 9, 37, 41), (3, 410, 64, 128, 64), (140, 96, 8, 70, 30), (2, 300, 10, 200, 150)])
@pytest.mark.parametrize("stable", [False, True])
def test_lockstep_record_recomputed_cuda_core_kernel(sh, dtype, d, mode, U, B, r, w, m, stable):
    """SH_OPT_RECORD_MODE = 1 (Algorithm 2 as stated) on every storage type and head size: the recount runs
    on the CUDA-core kernel (w beyond 64: several CTAs per unit), visibility by position in both compaction modes."""
    T = min(2 * B + 3 * m + 5, B + 2 * m + 30)
    q, k, v = wl.random_stream(U, d, T, seed=53 + U, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, recompute_record=True, prefill_chunk=mode, unordered=not stable)
    res, orc = run_lockstep_recompute(h, dtype, _stream_fn(q, k, v), T, torch.arange(U), TOL[dtype])
    assert res.compressions >= 2
    assert res.adoptions <= 1e-4 * res.slot_steps + 2


@pytest.mark.parametrize("recompute", [False, True])
def test_config_tiny_chunked_prompt_and_both_record_modes(sh, recompute):
    """The fp32, head_dim 64 workload with its prompt through the chunk kernel, and Algorithm 2 as stated."""
    cfg = wl.CONFIGS["tiny"]
    st = wl.Stream(cfg, device="cuda")
    h = sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, auto_compress=False, recompute_record=recompute)
    res, orc = run_lockstep_chunked(h, cfg.dtype, st.block, cfg.prompt, torch.arange(cfg.units), TOL[cfg.dtype],
                                    recompute=recompute, single_via_step=True)
    assert res.steps == cfg.prompt
    run = run_lockstep_recompute if recompute else run_lockstep
    res2, _ = run(h, cfg.dtype, st.step, cfg.decode, torch.arange(cfg.units), TOL[cfg.dtype], orc=orc)
    assert res2.compressions == 13


@pytest.mark.parametrize("U,B,r,w,m", [(601, 77, 6, 21, 30), (600, 410, 64, 128, 64), (592, 33, 0, 1, 33), (700, 150, 9, 37, 1)])
@pytest.mark.parametrize("recompute", [False, True])
def test_lockstep_int4_tensor_core_decode_kernel(sh, U, B, r, w, m, recompute):
    """The decode kernel the library picks for the int4 store from 592 units on (codes unpacked to fp16, dot
    products as warp-level MMAs): sampled units in lockstep, ragged row counts (n not a multiple of 8 or 16),
    the step's own token quantised bit-identically, and the query ring kept for the recompute mode."""
    dtype, d = "int4", 128
    T = min(B + 2 * m + 40, B + 150)
    q, k, v = wl.random_stream(U, d, T, seed=59 + B, dtype=dtype, peaked=3.0, device="cuda")
    h = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, recompute_record=recompute)
    units = torch.tensor([0, 1, 17, 148, 299, 300, 591, U - 1])
    run = run_lockstep_recompute if recompute else run_lockstep
    res, orc = run(h, dtype, _stream_fn(q, k, v), T, units, TOL[dtype])
    assert res.compressions >= 2
    assert res.adoptions <= 1e-4 * res.slot_steps + 2
    view = SortedView(h, units=units.numpy())
    n = h.n
    for i, u in enumerate(units.tolist()):
        K, V = view.export_unit(u)
        oK, oV = orc.cache(i)
        assert (K[:n].astype(np.float64) == oK).all() and (V[:n].astype(np.float64) == oV).all()


def test_ragged_sequences_int4_tensor_core_kernel(sh):
    compressions = _ragged_lockstep(sh, "int4", 128, [3, 41], ups=300, B=48, r=4, w=12, m=16, T_dec=40, kernel=None,
                                    unordered=None, split=None, seed=58)
    assert compressions >= 3
