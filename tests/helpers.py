"""Shared test helpers: draw a unit's inputs, and independent numpy restatements used as pins."""
from __future__ import annotations

import itertools

import numpy as np
import torch

from paper_2503_00979_b200 import synth


def unit_inputs(w: synth.Workload, layer: int, b: int, hkv: int, positions, device="cpu"):
    """q [G,len,d], k [len,d], v [len,d] float64 numpy for one unit at the given positions."""
    st = synth.Stream(w, device)
    k, v = st.kv(positions, [layer], [b], [hkv])
    q = st.q(positions, [layer], [b], [hkv])
    return (q[0, 0].double().cpu().numpy(), k[0, 0, 0].double().cpu().numpy(), v[0, 0, 0].double().cpu().numpy())


def causal_attention(q, k, v):
    """Textbook causal soft-max attention, one head: q,k,v [T,d] -> [T,d] (self-inclusive)."""
    T, d = q.shape
    out = np.zeros_like(v)
    for t in range(T):
        s = k[: t + 1] @ q[t] / np.sqrt(d)
        p = np.exp(s - s.max())
        p /= p.sum()
        out[t] = p @ v[: t + 1]
    return out


def softmax_over(qv, keys):
    """Soft-max weights of one query over a list of key vectors (fp64)."""
    s = np.array([np.dot(qv, kk) for kk in keys]) / np.sqrt(len(qv))
    p = np.exp(s - s.max())
    return p / p.sum()


def best_subset_by_enumeration(F: dict, C: int):
    """The size-C subset of candidates with the largest total fused score, found by
    trying every subset (only for a handful of candidates)."""
    keys = sorted(F)
    best, best_val = None, -np.inf
    for sub in itertools.combinations(keys, C):
        val = sum(F[p] for p in sub)
        if val > best_val:
            best, best_val = set(sub), val
    return best


class ShadowMorphKV:
    """A dictionary-based restatement of the MorphKV bookkeeping used to pin the oracle on tiny inputs.

    It remembers, for every generated token, the attention weights it assigned (a dict position ->
    weight per head), recomputed here from the raw vectors.  At each step it ranks ALL candidates
    by a plain Python sort and also finds the best size-C subset by exhaustive enumeration.
    """

    def __init__(self, G, d, C, R, fusion, evict_interval=1, norm="frozen"):
        self.G, self.d, self.C, self.R, self.fusion = G, d, C, R, fusion
        # "current": a window row's weights are divided by what is left of its mass on the tokens still cached
        self.norm = norm
        # coarse-grained eviction (appendix): the policy runs on generation steps T, 2T, 3T, ... only
        self.T = evict_interval
        self.generated = 0
        self.keys, self.vals = {}, {}
        self.profile = {}  # position -> list over g of {pos: weight}
        self.cached = set()
        self.t = 0
        self.last_F, self.last_ranked, self.last_dropped = None, None, []

    def prefill(self, k, v, qwin):
        P = k.shape[0]
        Rw = min(self.R, P)
        for j in range(P):
            self.keys[j], self.vals[j] = k[j], v[j]
        for i in range(Rw):
            r = P - Rw + i
            self.profile[r] = []
            for g in range(self.G):
                w = softmax_over(qwin[g, i], [k[j] for j in range(r + 1)])
                self.profile[r].append({j: w[j] for j in range(r + 1)})
        self.cached = set(range(P))
        self.t = P
        self._select()

    def _window(self):
        return set(range(max(0, self.t - self.R), self.t))

    def _fused(self, cand):
        win = sorted(self._window())
        F = {}
        left = {(r, g): (sum(wt for p, wt in self.profile[r][g].items() if p in self.cached) if self.norm == "current" else 1.0)
                for r in win for g in range(self.G)}
        for c in cand:
            per_row = [sum(self.profile[r][g][c] / left[(r, g)] for g in range(self.G)) for r in win]
            F[c] = sum(per_row) if self.fusion == "sum" else max(per_row)
        return F

    def _select(self):
        cand = self.cached - self._window()
        self.last_F, self.last_dropped = None, []
        if len(cand) > self.C:
            F = self._fused(cand)
            ranked = sorted(cand, key=lambda p: (-F[p], p))
            self.last_F = F
            self.last_ranked = ranked
            self.last_dropped = sorted(ranked[self.C:])
            self.cached -= set(ranked[self.C:])

    def step(self, q, k_new, v_new):
        t = self.t
        self.keys[t], self.vals[t] = k_new, v_new
        J = sorted(self.cached | {t})
        out = np.zeros((self.G, self.d))
        self.profile[t] = []
        for g in range(self.G):
            w = softmax_over(q[g], [self.keys[j] for j in J])
            self.profile[t].append(dict(zip(J, w)))
            out[g] = sum(wj * self.vals[j] for wj, j in zip(w, J))
        self.cached.add(t)
        self.t = t + 1
        self.generated += 1
        self.last_F, self.last_dropped = None, []
        if self.generated % self.T == 0:
            self._select()
        return out
