"""Brute-force statements used to pin the oracle on tiny inputs (pure Python / numpy).

Nothing here is shared with the oracle or the CUDA path: attention is the textbook
full softmax over the explicitly retained list, hits come from enumerating subsets,
CRF is the closed-form sum over a recorded hit log (Section 5.2), and eviction is an
exhaustive argmin.
"""
from __future__ import annotations

import itertools

import numpy as np
import torch


def f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def naive_attention(q, K, V, scale):
    """q [G,d], K [n,d], V [n,d] float64 -> (prob [G,n], y [G,d])."""
    s = scale * (q @ K.T)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    p = e / e.sum(axis=1, keepdims=True)
    return p, p @ V


def smallest_covering_sets(pbar, p):
    """All subsets of minimum cardinality whose mass reaches p; [(mass, frozenset)]."""
    n = len(pbar)
    for r in range(1, n + 1):
        found = []
        for S in itertools.combinations(range(n), r):
            m = float(sum(pbar[i] for i in S))
            if m >= p:
                found.append((m, frozenset(S)))
        if found:
            return found
    return []


def brute_hits(pbar, p):
    """The hit set by enumeration: minimum cardinality, then maximum mass."""
    found = smallest_covering_sets(pbar, p)
    if not found:  # total mass below p (rounding): everything is needed
        return frozenset(range(len(pbar))), 1
    best = max(m for m, _ in found)
    winners = [S for m, S in found if m == best]
    return winners[0], len(winners)


class BruteUnit:
    """One (sequence, layer, kv-head) cache simulated from definitions."""

    def __init__(self, budget, lam, top_p, scale, evict_every=1, literal_return=False):
        self.B, self.lam, self.p, self.scale = budget, lam, top_p, scale
        self.m = max(1, evict_every)   # eviction waits until the head is m entries over its budget
        self.literal = literal_return  # nothing of Algorithm 1 runs while the head is below its budget
        self.pos, self.K, self.V = [], [], []
        self.hits = []     # per entry: list of hit times
        self.arrival = []  # per entry: arrival time (tau before the first hit)

    def append(self, pos, k, v, arrival):
        self.pos.append(pos); self.K.append(k); self.V.append(v)
        self.hits.append([]); self.arrival.append(arrival)

    def crf(self, i, t):
        """Closed form CRF(e_i) = sum_j lambda^(t - t_j) over the hit log."""
        return sum(self.lam ** (t - tj) for tj in self.hits[i])  # 0 ** 0 == 1

    def last(self, i):
        return self.hits[i][-1] if self.hits[i] else self.arrival[i]

    def _drop(self, gone):
        for name in ("pos", "K", "V", "hits", "arrival"):
            setattr(self, name, [x for j, x in enumerate(getattr(self, name)) if j not in gone])

    def shrink(self, budget, t_last):
        """A budget that shrank (Algorithm 2, or set by hand): the head keeps its `budget` best
        entries at once.  Ranking from the definitions: CRF is the Section 5.2 sum evaluated at
        the time of the last step, then the last hit (or arrival) time, then the position; the
        lowest leave.  Returns the smallest relative distance of the cut from flipping."""
        self.B = budget
        n, gap = len(self.pos), np.inf
        if n > budget:
            keys = sorted((self.crf(i, t_last), self.last(i), self.pos[i], i) for i in range(n))
            kk = n - budget
            a, b = keys[kk - 1][0], keys[kk][0]
            if a != b:
                gap = abs(b - a) / max(abs(a), abs(b))
            self._drop({x[3] for x in keys[:kk]})
        return gap

    def tie_flags(self, q, t, eps):
        """What the tie log should say about a think step at time t with query q, BEFORE the
        step is taken: (nucleus, evict).  nucleus: the inclusive or the exclusive mass at the
        last hit lies within eps (relative to p) of p, or the last hit's score is within eps
        (relative to itself) of the first miss's.  evict: the k-th and (k+1)-th lowest CRF
        differ by less than eps relative to the larger, without being equal."""
        K = np.stack(self.K)
        prob, _ = naive_attention(q, K, np.stack(self.V), self.scale)
        pbar = prob.mean(axis=0)
        S, _ = brute_hits(list(pbar), self.p)
        srt = np.sort(pbar)[::-1]
        c = np.cumsum(srt)
        k = len(S)
        nucleus = abs(c[k - 1] - self.p) / self.p < eps or abs((c[k - 2] if k > 1 else 0.0) - self.p) / self.p < eps
        if k < len(srt) and srt[k - 1] > 0:
            nucleus = nucleus or abs(srt[k - 1] - srt[k]) / srt[k - 1] < eps
        evict = False
        n = len(self.pos)
        if n - self.B >= self.m:
            crf = sorted(self.crf(i, t) + (1.0 if i in S else 0.0) for i in range(n))
            a, b = crf[n - self.B - 1], crf[n - self.B]
            evict = a != b and abs(b - a) < eps * max(abs(a), abs(b))
        return bool(nucleus), bool(evict)

    def step(self, q, t, track=True, evict=True):
        """Attention at time t; returns (y, min_gap) where min_gap is the smallest
        relative distance of any decision from flipping (for skipping near-ties)."""
        K, V = np.stack(self.K), np.stack(self.V)
        prob, y = naive_attention(q, K, V, self.scale)
        gap = np.inf
        if track and not (self.literal and len(self.pos) < self.B):
            pbar = prob.mean(axis=0)
            (S, nwin) = brute_hits(list(pbar), self.p)
            srt = np.sort(pbar)[::-1]
            c = np.cumsum(srt)
            k = len(S)
            gap = min(gap, abs(c[k - 1] - self.p), abs((c[k - 2] if k > 1 else 0.0) - self.p))
            if k < len(srt):
                gap = min(gap, abs(srt[k - 1] - srt[k]) / srt[k - 1])
            for i in S:
                self.hits[i].append(t)
            n = len(self.pos)
            if evict and n - self.B >= self.m:
                keys = [(self.crf(i, t), self.last(i), self.pos[i], i) for i in range(n)]
                keys.sort()
                kk = n - self.B
                a, b = keys[kk - 1][0], keys[kk][0]
                if a != b:
                    gap = min(gap, abs(b - a) / max(abs(a), abs(b)))
                self._drop({x[3] for x in keys[:kk]})
        return y, gap
