"""Lockstep parity harness: drives the CUDA library and the CPU oracle through
the same stream, step by step.

The library decides ``alpha_j < 1/t`` in fp32, the oracle in fp64; they can
differ only where alpha_j is within rounding of the threshold.  Because the
record feeds back into which tokens survive, one such flip would make every
later kept set incomparable, so at each step the oracle takes over the
library's bit wherever its own alpha_j lies within 1e-6 of 1/t (an "adoption",
counted and reported) and any other disagreement is a failure.  With that,
positions, counters and kept sets must agree bit for bit at every step, and
attention outputs within the stated tolerance.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

import oracle as oracle_mod


@dataclasses.dataclass
class LockstepResult:
    steps: int = 0
    compressions: int = 0
    adoptions: int = 0
    slot_steps: int = 0
    max_abs_err: float = 0.0


class SortedView:
    """A handle whose slots are read back in position order.

    With SH_OPT_COMPACTION = 1 the library keeps the surviving tokens in no particular slot order,
    while the oracle keeps them oldest first.  What each side holds per token (position, record,
    this step's bit, key and value row) is unique, so the comparison sorts the library's slots by
    position and stays element by element.  For an ordered handle the permutation is the identity.
    ``units``: sort only these units' rows (the others come back as stored), for large handles of
    which a test checks a sample."""

    def __init__(self, handle, units=None):
        self._h = handle
        self._units = None if units is None else np.asarray(units, dtype=np.int64)

    def _argsort(self, key):
        if self._units is None:
            return np.argsort(key, axis=1, kind="stable")
        perm = np.broadcast_to(np.arange(key.shape[1]), key.shape).copy()
        perm[self._units] = np.argsort(key[self._units], axis=1, kind="stable")
        return perm

    def __getattr__(self, name):
        return getattr(self._h, name)

    def _perm(self):
        n, _, pos, _, _ = self._h.state(pos=True, counters=False, low=False)
        perm = self._argsort(pos)
        rows = slice(None) if self._units is None else self._units
        assert (np.diff(np.take_along_axis(pos, perm, axis=1)[rows], axis=1) > 0).all(), "duplicate positions in a unit"
        return n, perm

    def state(self, pos=True, counters=True, low=True, stream=None):
        n, t, p, c, l = self._h.state(pos=True, counters=counters, low=low, stream=stream)
        perm = self._argsort(p)
        srt = lambda a: np.take_along_axis(a, perm, axis=1) if a is not None else None
        return n, t, (srt(p) if pos else None), srt(c), srt(l)

    def state_full(self, stream=None):
        p, c, l = self._h.state_full(stream)
        key = np.where(p > 0, p, np.iinfo(np.int32).max)          # free slots (position 0) go last
        perm = self._argsort(key)
        return tuple(np.take_along_axis(a, perm, axis=1) for a in (p, c, l))

    def export_record(self, unit, stream=None):
        n, perm = self._perm()
        planes = self._h.export_record(unit, stream)
        out = planes.copy()
        out[:, :n] = planes[:, perm[unit]]
        return out

    def export_unit(self, unit, stream=None):
        n, perm = self._perm()
        K, V = self._h.export_unit(unit, stream)
        K[:n], V[:n] = K[perm[unit]], V[perm[unit]]
        return K, V


def to_oracle(x: torch.Tensor, units) -> np.ndarray:
    """Rows ``units`` of a [U, d] storage-dtype tensor as exact fp64."""
    return x[units].to(torch.float64).cpu().numpy()


def run_lockstep(handle, cfg_dtype: str, inputs, steps: int, units, tol: float, state_every: int = 1,
                 res: LockstepResult = None, orc=None, outs=None):
    """``inputs(t)`` -> (q, k, v) CUDA tensors [U, d] for 1-based step t.
    ``units``: LongTensor of unit indices checked against the oracle.
    The handle must have been created with auto_compress=False.  ``outs``: a list that receives every
    step's output tensor [U, d].  Returns (LockstepResult, oracle)."""
    units = torch.as_tensor(units, dtype=torch.long)
    un = units.numpy()
    if not isinstance(handle, SortedView):          # slots are compared in position order, whatever the compaction mode
        handle = SortedView(handle, units=un)
    if orc is None:
        orc = oracle_mod.Oracle(len(un), handle.B, handle.r, handle.w, handle.m, handle.D,
                                quant=(cfg_dtype == "int4"))
    res = res or LockstepResult()
    dev_units = units.to(handle.device)
    for _ in range(steps):
        t = orc.t + 1
        q, k, v = inputs(t)
        out = handle.decode_step(q, k, v)
        if outs is not None:
            outs.append(out)
        want_state = (t % state_every == 0) or (orc.n + 1 == handle.B)
        n, tt, pos, cnt, low = handle.state(pos=want_state, counters=want_state, low=True)
        o_out, alpha, o_low, amb = orc.attend(to_oracle(q, dev_units), to_oracle(k, dev_units),
                                              to_oracle(v, dev_units))
        assert n == orc.n and tt == orc.t == t
        err = float(np.abs(out[dev_units].double().cpu().numpy() - o_out).max())
        res.max_abs_err = max(res.max_abs_err, err)
        assert err <= tol, f"step {t}: attention output off by {err:.3e} > {tol}"
        g_low = low[un]
        diff = g_low != o_low
        bad = diff & ~amb
        assert not bad.any(), (f"step {t}: {int(bad.sum())} record bits differ where the oracle's score is not "
                               f"within 1e-6 of 1/t; first at (unit, slot) {np.argwhere(bad)[0].tolist()}")
        res.adoptions += int(diff.sum())
        res.slot_steps += g_low.size
        orc.record(g_low)
        if want_state:
            assert (pos[un] == orc.positions()).all(), f"step {t}: positions differ"
            assert (cnt[un].astype(np.int32) == orc.counters()).all(), f"step {t}: importance records differ"
        if orc.full:
            dropped = orc.compress()
            got = handle.compress()
            assert dropped is not None and got == handle.m
            n2, _, pos2, cnt2, _ = handle.state(low=False)
            assert n2 == orc.n == handle.B - handle.m
            o_pos = orc.positions()
            assert (pos2[un] == o_pos).all(), f"step {t}: kept sets differ after compression"
            assert (cnt2[un].astype(np.int32) == orc.counters()).all(), f"step {t}: records differ after compaction"
            res.compressions += 1
        res.steps += 1
    return res, orc


def run_lockstep_chunked(handle, cfg_dtype: str, inputs_block, steps: int, units, tol: float, chunk_sizes=None,
                         res: LockstepResult = None, orc=None, recompute: bool = False, outs=None,
                         single_via_step: bool = False):
    """Same protocol as run_lockstep, driving the library through sh_prefill_chunk.

    ``inputs_block(t0, t1)`` -> (q, k, v) CUDA tensors [t1-t0, U, d] for stream positions t0 .. t1-1
    (1-based).  The library evaluates a whole chunk in one launch; the oracle then replays the chunk
    step by step, and each step's record bits are read back from the unit's bit-planes (no
    compression happens inside a chunk, so nothing has moved them).  ``chunk_sizes`` cycles through
    requested chunk lengths (clipped to what the library and the remaining budget allow).  With
    ``single_via_step`` a chunk of one token goes through sh_decode_step, as sh_prefill does it: with the
    default sizes the sequence of launches is then exactly sh_prefill's, so a second handle fed through
    sh_prefill must end bit-identical to this one.
    ``recompute``: the handle runs SH_OPT_RECORD_MODE = 1; at each compression the library's recomputed
    bit-planes are compared with the oracle's recount (adoption inside the window) before both compress.
    ``outs``: a list that receives each chunk's output tensor [cnt, U, d]."""
    units = torch.as_tensor(units, dtype=torch.long)
    un = units.numpy()
    if not isinstance(handle, SortedView):          # slots are compared in position order, whatever the compaction mode
        handle = SortedView(handle, units=un)
    if orc is None:
        orc = oracle_mod.Oracle(len(un), handle.B, handle.r, handle.w, handle.m, handle.D,
                                quant=(cfg_dtype == "int4"))
    res = res or LockstepResult()
    dev_units = units.to(handle.device)
    cap = handle.prefill_chunk_max
    assert cap >= 2, "the chunk kernel does not serve this handle"
    sizes = list(chunk_sizes or [cap])
    done, k_i = 0, 0
    while done < steps:
        cnt = min(sizes[k_i % len(sizes)], cap, steps - done, handle.B - orc.n)
        k_i += 1
        t0 = orc.t + 1
        q, k, v = inputs_block(t0, t0 + cnt)
        out = torch.empty(cnt, handle.U, handle.D, device=handle.device)
        if cnt == 1 and single_via_step:
            handle.decode_step(q[0], k[0], v[0], out[0])
        else:
            handle.prefill_chunk(q, k, v, out)
        if outs is not None:
            outs.append(out)
        n, tt, pos, cnt_rec, _ = handle.state(low=False)
        planes = [handle.export_record(int(u)) for u in un]      # [w, B] bool per sampled unit
        for i in range(cnt):
            t = t0 + i
            o_out, alpha, o_low, amb = orc.attend(to_oracle(q[i], dev_units), to_oracle(k[i], dev_units),
                                                  to_oracle(v[i], dev_units))
            err = float(np.abs(out[i][dev_units].double().cpu().numpy() - o_out).max())
            res.max_abs_err = max(res.max_abs_err, err)
            assert err <= tol, f"step {t}: attention output off by {err:.3e} > {tol}"
            nn = orc.n
            g_low = np.stack([pl[t % handle.w, :nn] for pl in planes])
            beyond = np.stack([pl[t % handle.w, nn:] for pl in planes])
            assert not beyond.any(), f"step {t}: record bits set beyond the slots live at that step"
            diff = g_low != o_low
            bad = diff & ~amb
            assert not bad.any(), (f"step {t}: {int(bad.sum())} record bits differ outside the 1e-6 window; "
                                   f"first at (unit, slot) {np.argwhere(bad)[0].tolist()}")
            res.adoptions += int(diff.sum())
            res.slot_steps += g_low.size
            orc.record(g_low)
            res.steps += 1
        assert n == orc.n and tt == orc.t
        assert (pos[un] == orc.positions()).all(), f"after step {orc.t}: positions differ"
        assert (cnt_rec[un].astype(np.int32) == orc.counters()).all(), f"after step {orc.t}: records differ"
        if orc.full:
            if recompute:
                _adopt_recount(handle, orc, un, res)
            orc.compress()
            assert handle.compress() == handle.m
            n2, _, pos2, cnt2, _ = handle.state(low=False)
            assert n2 == orc.n
            assert (pos2[un] == orc.positions()).all(), f"after step {orc.t}: kept sets differ"
            assert (cnt2[un].astype(np.int32) == orc.counters()).all()
            res.compressions += 1
        done += cnt
    return res, orc


def _adopt_recount(handle, orc, un, res):
    """SH_OPT_RECORD_MODE = 1 at a full cache: the library recomputes its bit-planes, the oracle recounts
    from its own stored queries; bits may differ only inside the 1e-6 window, where the oracle takes the
    library's; the counters must then be identical."""
    t = orc.t
    handle.recompute_record()
    nn = orc.n
    g = np.stack([handle.export_record(int(u))[:, :nn] for u in un])          # [units, w, n]
    _a, o_low, amb, steps_in = orc.recount()
    live_rows = steps_in > 0
    assert not g[:, ~live_rows].any(), "bits in rows of steps outside the window"
    diff = g != o_low
    bad = diff & ~amb
    assert not bad.any(), (f"step {t}: {int(bad.sum())} recomputed bits differ outside the 1e-6 window; "
                           f"first at (unit, row, slot) {np.argwhere(bad)[0].tolist()}")
    res.adoptions += int(diff.sum())
    res.slot_steps += int(live_rows.sum()) * nn * len(un)
    orc.set_record(g, steps_in)
    _n1, _, _pos1, cnt1, _ = handle.state(low=False)
    assert (cnt1[un].astype(np.int32) == orc.counters()).all(), f"step {t}: recomputed records differ"


def run_lockstep_recompute(handle, cfg_dtype: str, inputs, steps: int, units, tol: float, res: LockstepResult = None,
                           orc=None):
    """Lockstep for SH_OPT_RECORD_MODE = 1 (the record recomputed at compression time).
    Every step: outputs compared.  When the cache fills: the library recomputes its
    bit-planes, the oracle recounts from its own stored queries; bits may differ only
    inside the 1e-6 window (the oracle then adopts the library's), after which counters,
    positions and kept sets must be identical."""
    units = torch.as_tensor(units, dtype=torch.long)
    un = units.numpy()
    if not isinstance(handle, SortedView):          # slots are compared in position order, whatever the compaction mode
        handle = SortedView(handle, units=un)
    if orc is None:
        orc = oracle_mod.Oracle(len(un), handle.B, handle.r, handle.w, handle.m, handle.D, quant=(cfg_dtype == "int4"))
    res = res or LockstepResult()
    dev_units = units.to(handle.device)
    w = handle.w
    for _ in range(steps):
        t = orc.t + 1
        q, k, v = inputs(t)
        out = handle.decode_step(q, k, v)
        o_out, _alpha, _low, _amb = orc.attend(to_oracle(q, dev_units), to_oracle(k, dev_units),
                                               to_oracle(v, dev_units))
        err = float(np.abs(out[dev_units].double().cpu().numpy() - o_out).max())
        res.max_abs_err = max(res.max_abs_err, err)
        assert err <= tol, f"step {t}: attention output off by {err:.3e} > {tol}"
        if orc.full:
            _adopt_recount(handle, orc, un, res)
            orc.compress()
            assert handle.compress() == handle.m
            n2, _, pos2, cnt2, _ = handle.state(low=False)
            assert n2 == orc.n
            assert (pos2[un] == orc.positions()).all(), f"step {t}: kept sets differ"
            res.compressions += 1
        res.steps += 1
    return res, orc




def assert_same_state(a, b, rows: bool = True):
    """Two handles of the library hold bit-identical state: counters, positions, record, this step's
    bits and (``rows``) every byte of the workspace's K and V regions."""
    sa, sb = a.state(), b.state()
    assert sa[0] == sb[0] and sa[1] == sb[1], "n or t differ"
    for name, x, y in zip(("positions", "counters", "last bits"), sa[2:], sb[2:]):
        assert (x == y).all(), f"{name} differ"
    if rows:
        row_bytes = {0: 4 * a.D, 1: 2 * a.D, 2: 2 * a.D, 3: a.D // 2}[a.dtype]
        kv = 2 * ((a.U * a.B * row_bytes + 255) // 256 * 256)            # the K region, then the V region
        assert torch.equal(a.slab[a._slab_off:a._slab_off + kv], b.slab[b._slab_off:b._slab_off + kv]), "K/V rows differ"
