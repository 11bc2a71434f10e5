"""Persistence-of-importance diagnostics on synthetic streams (Section 3.2).

A token is *pivotal* for position t when the query at t gives it a score above
1/t; S_{a->b} is the union of the pivotal sets of positions a..b.  For a
sentence of length l the paper measures, with t = l/2,

    persistence ratio = |S_{t+1->l} n S_{1->t}| / |{x in S_{t+1->l} : x among x_1..x_t}|

and the relative size |S_{1->t}| / t.  Both come straight out of the library's
importance record: a handle whose budget holds the whole sentence never
compresses, and with a history window of l steps its bit-planes keep, for every
step, which cached tokens scored below 1/t.  The attention itself runs in the
CUDA kernels; only the set algebra on the exported bits is done here.

The paper measures these on trained OPT models over text; here the inputs are
the synthetic streams of ``workloads`` (there are no weights or corpora in this
repository), so the numbers characterise those streams, not a language model.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from . import binding as sh


@dataclasses.dataclass
class Persistence:
    ratio: np.ndarray        # [units] persistence ratio (nan where the later half has no pivotal token in the first half)
    pivotal_frac: np.ndarray # [units] |S_{1->t}| / t
    t: int
    l: int


def pivotal_table(handle: "sh.Handle", unit: int, l: int) -> np.ndarray:
    """[l, l] bool: entry (s-1, j) = token j+1 was pivotal for position s (score not below 1/s).
    Needs a handle that has streamed exactly l tokens with B > l and w >= l (no compression, every
    step's bit-plane row still present)."""
    planes = handle.export_record(unit)              # [w, B]: row s mod w, slot j; bit set = "low"
    rows = np.arange(1, l + 1) % handle.w
    low = planes[rows][:, :l]
    seen = np.tril(np.ones((l, l), dtype=bool))      # position s only sees tokens 1..s
    return seen & ~low


def persistence(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, dtype: str, device="cuda:0") -> Persistence:
    """q, k, v: [l, units, head_dim] CUDA tensors in the storage dtype.  Runs full-cache attention
    over the stream (budget l + 1, window l) and evaluates the two measures per unit."""
    l, U, d = q.shape
    h = sh.Handle(l + 1, 0, l, 1, U, d, dtype, device=device, auto_compress=False, prefill_chunk=False)
    h.prefill(q, k, v)
    t = l // 2
    ratio = np.full(U, np.nan)
    frac = np.zeros(U)
    for u in range(U):
        piv = pivotal_table(h, u, l)
        first = piv[:t, :t].any(axis=0)              # S_{1->t}
        later = piv[t:, :t].any(axis=0)              # S_{t+1->l} restricted to x_1..x_t
        if later.any():
            ratio[u] = (first & later).sum() / later.sum()
        frac[u] = first.sum() / t
    return Persistence(ratio, frac, t, l)


@dataclasses.dataclass
class ScoreChange:
    ratio: np.ndarray        # [units, t] (alpha_s - alpha_o) / alpha_o per stream position 1..t; -1 where the token was dropped
    kept: np.ndarray         # [units, t] bool: the token is still in the budgeted cache
    alpha_s: np.ndarray      # [units, t] score over the budgeted cache (0 where dropped)
    alpha_o: np.ndarray      # [units, t] score over the full cache
    t: int


def score_change_ratio(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, dtype: str, B: int, r: int, w: int, m: int,
                       device="cuda:0", unordered=None) -> ScoreChange:
    """Change ratio of the attention scores (the paper's ablation on attention score error):
    the t tokens of ``q, k, v`` ([t, units, head_dim], storage dtype, CUDA) are streamed through a
    handle with budget ``B`` (compressing as it goes) and through one that keeps everything; the
    last step's query is then scored over both caches (``sh_scores``) and compared token by token,
    a dropped token counting as a score of 0 (ratio -1).  Scores come from the CUDA kernels; only
    the scatter by position and the division are done here."""
    t, U, d = q.shape
    hs = sh.Handle(B, r, w, m, U, d, dtype, device=device, unordered=unordered)
    ho = sh.Handle(t + 1, 0, 1, 1, U, d, dtype, device=device)          # never fills: the original cache
    hs.prefill(q, k, v)
    ho.prefill(q, k, v)
    a_s = hs.scores(q[t - 1].contiguous()).cpu().numpy().astype(np.float64)
    a_o = ho.scores(q[t - 1].contiguous()).cpu().numpy().astype(np.float64)[:, :t]
    n, _, pos, _, _ = hs.state(counters=False, low=False)
    alpha_s = np.zeros((U, t))
    kept = np.zeros((U, t), dtype=bool)
    rows = np.arange(U)[:, None]
    alpha_s[rows, pos - 1] = a_s[:, :n]
    kept[rows, pos - 1] = True
    return ScoreChange((alpha_s - a_o) / a_o, kept, alpha_s, a_o, t)


@dataclasses.dataclass
class RecordModeOverlap:
    overlap: np.ndarray      # [units] |kept_online n kept_recomputed| / n
    overlap_old: np.ndarray  # [units] the same over the tokens outside the recent window only (those the record decided)
    n: int                   # tokens kept per unit
    t: int


def record_mode_overlap(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, dtype: str, B: int, r: int, w: int, m: int,
                        device="cuda:0") -> RecordModeOverlap:
    """Kept sets under the two ways of obtaining the importance record (Section 4.1, "Overhead Tradeoff"):
    kept online during generation (one comparison per cached token per step, against the cache as it was
    at that step) or recomputed at each compression from the last w queries against the cache as it is
    then (Algorithm 2 as stated).  The same ``q, k, v`` ([t, units, head_dim], storage dtype, CUDA) are
    streamed through one handle of each kind; returned is, per unit, the fraction of kept tokens the two
    have in common.  Everything but the set intersection runs in the CUDA kernels."""
    t, U, d = q.shape
    a = sh.Handle(B, r, w, m, U, d, dtype, device=device)
    b = sh.Handle(B, r, w, m, U, d, dtype, device=device, recompute_record=True)
    a.prefill(q, k, v)
    b.prefill(q, k, v)
    n, _, pos_a, _, _ = a.state(counters=False, low=False)
    n_b, _, pos_b, _, _ = b.state(counters=False, low=False)
    assert n == n_b
    both = np.array([len(np.intersect1d(pos_a[u], pos_b[u])) for u in range(U)])
    old = t - r
    both_old = np.array([len(np.intersect1d(pos_a[u][pos_a[u] <= old], pos_b[u][pos_b[u] <= old])) for u in range(U)])
    return RecordModeOverlap(both / n, both_old / max(n - min(r, n), 1), n, t)
