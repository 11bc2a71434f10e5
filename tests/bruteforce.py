"""From-the-definition simulation of one unit, for pinning the oracle on tiny
streams.  Deliberately organised differently from the oracle: it never deletes
anything.  It keeps every token ever streamed, a set of live positions, and the
full table ``low[i][p]`` (step i, position p) of threshold comparisons, and at
each compression recomputes the importance record from that table by the
definition in Algorithm 2 and finds the dropped set by exhaustive search over
all subsets of the candidates.  Pure Python/numpy: tiny inputs only.
"""
from __future__ import annotations

import itertools

import numpy as np


def full_attention(q, K, V, scale):
    """softmax(scale * q K^T) V with numpy, fp64 (Section 4.1, first display)."""
    s = scale * (K @ q)
    p = np.exp(s - s.max())
    p = p / p.sum()
    return p @ V, p


class BruteForceUnit:
    """``threshold``, ``window_plus1``, ``tie_newest``, ``trigger_literal``: the alternative readings
    the oracle also offers (1/t of the compression step or 1/n instead of 1/t of the step; w+1 steps;
    newest first among equal counters; compress only when n exceeds B)."""

    def __init__(self, B, r, w, m, d, scale, threshold=0, window_plus1=False, tie_newest=False, trigger_literal=False):
        self.B, self.r, self.w, self.m, self.d, self.scale = B, r, w, m, d, scale
        self.threshold, self.window_plus1, self.tie_newest, self.trigger_literal = threshold, window_plus1, tie_newest, trigger_literal
        self.keys, self.vals = {}, {}      # position -> vector, never deleted
        self.live = set()                  # positions currently cached
        self.score = {}                    # step -> {position: alpha}
        self.n_at = {}                     # step -> number of tokens attended
        self.t = 0
        self.dropped_log = []              # (step, sorted dropped positions)

    def _is_low(self, i, p):
        a = self.score.get(i, {}).get(p)
        if a is None:
            return False                   # not cached at step i: no information, not counted
        thr = {0: 1.0 / i, 1: 1.0 / self.t, 2: 1.0 / self.n_at[i]}[self.threshold]
        return bool(a < thr)

    def counters(self):
        """I_p = #{ i in (t-w, t] : p was cached at step i and alpha_{i,p} < threshold }."""
        t, w = self.t, self.w
        first = max(1, t - w + (0 if self.window_plus1 else 1))
        return {p: sum(1 for i in range(first, t + 1) if self._is_low(i, p)) for p in self.live}

    def step(self, q, k, v):
        self.t += 1
        t = self.t
        self.keys[t], self.vals[t] = np.asarray(k, float), np.asarray(v, float)
        self.live.add(t)
        order = sorted(self.live)
        K = np.stack([self.keys[p] for p in order])
        V = np.stack([self.vals[p] for p in order])
        out, alpha = full_attention(np.asarray(q, float), K, V, self.scale)
        self.score[t] = dict(zip(order, alpha))
        self.n_at[t] = len(order)
        dropped = None
        if len(self.live) == self.B + (1 if self.trigger_literal else 0):
            dropped = self._compress()
        return out, dict(zip(order, alpha)), dropped

    def _key(self, order, I):
        n = len(order)
        rank = {p: i for i, p in enumerate(order)}       # 0 = oldest
        # Unique composite key: larger counter first, then older first (or newer first).
        return {p: I[p] * (n + 1) + ((rank[p] + 1) if self.tie_newest else (n - rank[p])) for p in order[: n - self.r]}

    def _compress(self):
        I = self.counters()
        order = sorted(self.live)
        key = self._key(order, I)                        # the r newest are never candidates
        best, best_sum = None, None
        for sub in itertools.combinations(list(key), self.m):
            s = sum(key[p] for p in sub)
            if best_sum is None or s > best_sum:
                best, best_sum = sub, s
        for p in best:
            self.live.remove(p)
        d = sorted(best)
        self.dropped_log.append((self.t, d))
        return d

    def shrink_below(self, B, m, r):
        """The bulk reading of the prompting stage: with the record as it stands, drop m tokens at a
        time until fewer than B remain (no more than B with the literal trigger).  The key of a token does
        not change between rounds and the r newest stay the same, so k rounds drop the k*m candidates
        with the largest keys: done here as one sort."""
        I = self.counters()
        order = sorted(self.live)
        self.r = r
        key = self._key(order, I)
        rounds = 0
        n = len(order)
        while n >= B + (1 if self.trigger_literal else 0):
            n -= m
            rounds += 1
        gone = sorted(key, key=lambda p: -key[p])[: rounds * m]
        assert len(gone) == rounds * m
        for p in gone:
            self.live.remove(p)
        return rounds, sorted(gone)
