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
    def __init__(self, B, r, w, m, d, scale):
        self.B, self.r, self.w, self.m, self.d, self.scale = B, r, w, m, d, scale
        self.keys, self.vals = {}, {}      # position -> vector, never deleted
        self.live = set()                  # positions currently cached
        self.low = {}                      # step -> {position: bool}
        self.t = 0
        self.dropped_log = []              # (step, sorted dropped positions)

    def counters(self):
        """I_p = #{ i in (t-w, t] : p was cached at step i and alpha_{i,p} < 1/i }."""
        t, w = self.t, self.w
        I = {}
        for p in self.live:
            I[p] = sum(1 for i in range(max(1, t - w + 1), t + 1) if self.low.get(i, {}).get(p, False))
        return I

    def step(self, q, k, v):
        self.t += 1
        t = self.t
        self.keys[t], self.vals[t] = np.asarray(k, float), np.asarray(v, float)
        self.live.add(t)
        order = sorted(self.live)
        K = np.stack([self.keys[p] for p in order])
        V = np.stack([self.vals[p] for p in order])
        out, alpha = full_attention(np.asarray(q, float), K, V, self.scale)
        self.low[t] = {p: bool(a < 1.0 / t) for p, a in zip(order, alpha)}
        dropped = None
        if len(self.live) == self.B:
            dropped = self._compress()
        return out, dict(zip(order, alpha)), dropped

    def _compress(self):
        I = self.counters()
        order = sorted(self.live)
        n = len(order)
        cand = order[: n - self.r]                       # the r newest are never candidates
        rank = {p: i for i, p in enumerate(order)}       # 0 = oldest
        # Unique composite key: larger counter first, then older first.
        key = {p: I[p] * (n + 1) + (n - rank[p]) for p in cand}
        best, best_sum = None, None
        for sub in itertools.combinations(cand, self.m):
            s = sum(key[p] for p in sub)
            if best_sum is None or s > best_sum:
                best, best_sum = sub, s
        for p in best:
            self.live.remove(p)
        d = sorted(best)
        self.dropped_log.append((self.t, d))
        return d
