"""Pins for the CPU oracle: what the paper and the mathematics fix, not the oracle against itself."""
import os

import numpy as np
import pytest
import torch

from paper_2503_00979_b200 import synth
from tests.helpers import (ShadowMorphKV, best_subset_by_enumeration, causal_attention, unit_inputs)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

TINY = synth.Workload("tiny", 1, 1, 4, 2, 16, "f32", 6, 24, 3, 2, "sum", 1234)


def _run(ora, w, unit=(0, 0, 0), steps=None, recompute=False, T=1, hook=None, C=None, R=None, fusion=None,
         transform=None):
    """Prefill + decode one unit of workload `w`; returns list of outputs and the oracle unit."""
    steps = w.steps if steps is None else steps
    G, d = w.group, w.head_dim
    q, k, v = unit_inputs(w, *unit, positions=np.arange(w.prompt_len + steps))
    if transform:
        q, k, v = transform(q, k, v)
    u = ora.Unit(G, d, C or w.C, R or w.R, fusion or w.fusion, evict_interval=T, recompute=recompute)
    P = w.prompt_len
    Rw = min(u.R, P)
    u.prefill(k[:P], v[:P], q[:, P - Rw:P])
    outs = []
    for s in range(steps):
        t = P + s
        o = u.step(q[:, t], k[t], v[t])
        outs.append(o)
        if hook:
            hook(u, t)
    return np.array(outs), u, (q, k, v)


# ---- P1: with C + R >= sequence length nothing is evicted and Eq. 1 is plain causal attention ----
@pytest.mark.parametrize("fusion", ["sum", "max"])
def test_full_attention_special_case(oracle, fusion):
    w = synth.WORKLOADS["c0"].replace(prompt_len=40, steps=60)
    outs, u, (q, k, v) = _run(oracle, w, C=90, R=16, fusion=fusion)
    assert u.count == 100
    P = w.prompt_len
    for g in range(w.group):
        ref = causal_attention(q[g], k, v)[P:]
        assert np.abs(outs[:, g] - ref).max() < 1e-12
    # library cross-check: torch SDPA in float64 on the CPU
    tq = torch.from_numpy(q)[None]                      # [1,G,T,d]
    tk = torch.from_numpy(k)[None, None].expand(1, w.group, -1, -1)
    tv = torch.from_numpy(v)[None, None].expand(1, w.group, -1, -1)
    sd = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0, :, P:]
    assert np.abs(outs - sd.permute(1, 0, 2).numpy()).max() < 1e-12


def test_full_attention_when_capacity_equals_length_exactly(oracle):
    # boundary: C + R == P + S, the last step fills the last slot and still evicts nothing
    w = TINY.replace(prompt_len=5, steps=7)
    outs, u, (q, k, v) = _run(oracle, w, C=9, R=3)
    assert u.count == 12
    for g in range(w.group):
        assert np.abs(outs[:, g] - causal_attention(q[g], k, v)[5:]).max() < 1e-12


# ---- P2: invariants of Eq. 7 / H1 ----
@pytest.mark.parametrize("fusion", ["sum", "max"])
def test_cache_invariants(oracle, fusion):
    w = synth.WORKLOADS["c0"].replace(steps=200)
    C, R = w.C, w.R
    state = {"prev": None, "gone": set()}

    def hook(u, t):
        pos = u.positions()
        assert len(pos) == len(set(pos.tolist())) == min(t + 1, C + R) == u.count
        assert pos.max() == t and (pos >= 0).all()
        assert set(range(t - R + 1, t + 1)) <= set(pos.tolist())          # H1: last R always kept
        cur = set(pos.tolist())
        assert not (cur & state["gone"])                                    # evicted tokens never return
        if state["prev"] is not None:
            assert cur <= state["prev"] | {t}                               # G' is a subset of G
            ev = (state["prev"] | {t}) - cur
            assert len(ev) == 1 and list(ev) == u.last_evicted().tolist()   # one eviction per step when full
            assert max(ev) <= t - R
            state["gone"] |= ev
        state["prev"] = cur

    _run(oracle, w, hook=hook, fusion=fusion)


def test_prefill_keeps_window_and_top_c(oracle):
    w = synth.WORKLOADS["c0"]
    q, k, v = unit_inputs(w, 0, 0, 1, np.arange(w.prompt_len))
    u = oracle.Unit(w.group, w.head_dim, w.C, w.R, w.fusion)
    u.prefill(k, v, q[:, -w.R:])
    pos = u.positions()
    assert len(pos) == w.C + w.R
    assert set(range(w.prompt_len - w.R, w.prompt_len)) <= set(pos.tolist())


# ---- P3: the paper's worked numbers ----
def test_walkthrough_numbers(oracle):
    rows, expect = [], {}
    for line in open(os.path.join(GOLDEN, "walkthrough_fusion.txt")):
        if line.startswith("#") or not line.strip():
            continue
        tag, *vals = line.split()
        if tag == "row":
            rows.append([float(x) for x in vals])
        else:
            expect[tag] = [float(x) for x in vals]
    S = np.array(rows)
    F, keep = oracle.fuse_select(S, 1, "sum")
    assert np.allclose(F, expect["sum"], atol=1e-15) and keep.tolist() == [bool(x) for x in expect["keep_top1"]]
    F, keep = oracle.fuse_select(S, 1, "max")
    assert np.allclose(F, expect["max"], atol=1e-15) and keep.tolist() == [bool(x) for x in expect["keep_top1"]]


def test_fuse_select_sum_and_max_disagree_where_they_should(oracle):
    # one strong vote vs many weak votes: sum keeps the consistently attended token, max the spike
    S = np.array([[0.30, 0.20], [0.01, 0.20], [0.01, 0.20]])
    F, keep = oracle.fuse_select(S, 1, "sum")
    assert np.allclose(F, [0.32, 0.60]) and keep.tolist() == [False, True]
    F, keep = oracle.fuse_select(S, 1, "max")
    assert np.allclose(F, [0.30, 0.20]) and keep.tolist() == [True, False]


def test_fuse_select_ties_keep_lower_position(oracle):
    S = np.array([[0.2, 0.1, 0.2, 0.2, 0.05]])
    _, keep = oracle.fuse_select(S, 2, "sum")
    assert keep.tolist() == [True, False, True, False, False]


# ---- P4: brute force on tiny inputs ----
@pytest.mark.parametrize("fusion", ["sum", "max"])
@pytest.mark.parametrize("G,C,R,P", [(1, 2, 2, 3), (2, 3, 2, 6), (4, 4, 3, 9), (2, 1, 1, 4), (2, 5, 4, 2), (1, 3, 1, 1)])
def test_against_exhaustive_shadow(oracle, fusion, G, C, R, P):
    w = TINY.replace(n_q_heads=2 * G, prompt_len=P, steps=14, C=C, R=R, fusion=fusion, seed=99 + G + C)
    q, k, v = unit_inputs(w, 0, 0, 1, np.arange(P + w.steps))
    u = oracle.Unit(G, w.head_dim, C, R, fusion)
    sh = ShadowMorphKV(G, w.head_dim, C, R, fusion)
    Rw = min(R, P)
    u.prefill(k[:P], v[:P], q[:, P - Rw:P])
    sh.prefill(k[:P], v[:P], q[:, P - Rw:P])
    assert set(u.positions().tolist()) == sh.cached
    n_sel = 0
    for s in range(w.steps):
        t = P + s
        o = u.step(q[:, t], k[t], v[t])
        o2 = sh.step(q[:, t], k[t], v[t])
        assert np.abs(o - o2).max() < 1e-12
        assert set(u.positions().tolist()) == sh.cached
        assert len(sh.cached) <= C + R
        if sh.last_F is not None:
            n_sel += 1
            pos, F = u.last_scores()
            assert pos.tolist() == sh.last_ranked                      # full ranking of ALL candidates
            assert np.allclose(F, [sh.last_F[p] for p in pos], rtol=1e-12, atol=1e-300)
            # "the C largest": exhaustive search over subsets agrees with the ranking's head
            assert best_subset_by_enumeration(sh.last_F, C) == set(sh.last_ranked[:C])
    assert n_sel > 0


# ---- P5: reductions ----
def test_r1_sum_equals_max(oracle):
    w = synth.WORKLOADS["c0"].replace(steps=80)
    a, ua, _ = _run(oracle, w, R=1, fusion="sum")
    b, ub, _ = _run(oracle, w, R=1, fusion="max")
    assert np.array_equal(a, b) and np.array_equal(ua.positions(), ub.positions())


def test_r1_g1_scores_are_own_attention_weights(oracle):
    w = TINY.replace(n_q_heads=2, n_kv_heads=2, prompt_len=8, steps=10, C=4, R=1)
    q, k, v = unit_inputs(w, 0, 0, 0, np.arange(18))
    u = oracle.Unit(1, w.head_dim, 4, 1, "sum")
    u.prefill(k[:8], v[:8], q[:, 7:8])
    for s in range(10):
        t = 8 + s
        before = u.positions().tolist()
        u.step(q[:, t], k[t], v[t])
        J = before + [t]
        sc = np.array([k[j] @ q[0, t] for j in J]) / np.sqrt(w.head_dim)
        p = np.exp(sc - sc.max())
        p /= p.sum()
        pos, F = u.last_scores()
        for pp, ff in zip(pos, F):
            assert abs(ff - p[J.index(pp)]) < 1e-14


def test_gqa_sums_the_group_before_max(oracle):
    # with G=2 and max fusion, F must be max_r(sum_g) -- not sum_g(max_r) and not max over (r,g)
    w = TINY.replace(n_q_heads=4, n_kv_heads=2, prompt_len=7, steps=6, C=3, R=3, fusion="max")
    q, k, v = unit_inputs(w, 0, 0, 0, np.arange(13))
    sh = ShadowMorphKV(2, w.head_dim, 3, 3, "max")
    u = oracle.Unit(2, w.head_dim, 3, 3, "max")
    u.prefill(k[:7], v[:7], q[:, 4:7]); sh.prefill(k[:7], v[:7], q[:, 4:7])
    differs = False
    for s in range(6):
        t = 7 + s
        u.step(q[:, t], k[t], v[t]); sh.step(q[:, t], k[t], v[t])
        pos, F = u.last_scores()
        win = sorted(sh._window())
        for pp, ff in zip(pos, F):
            right = max(sum(sh.profile[r][g][pp] for g in range(2)) for r in win)
            wrong1 = sum(max(sh.profile[r][g][pp] for r in win) for g in range(2))
            wrong2 = max(sh.profile[r][g][pp] for r in win for g in range(2))
            assert abs(ff - right) < 1e-14
            differs |= abs(right - wrong1) > 1e-6 and abs(right - wrong2) > 1e-6
    assert differs


# ---- P6: stored profile == recompute from the frozen (max, denominator) ----
@pytest.mark.parametrize("fusion", ["sum", "max"])
def test_stored_equals_frozen_recompute(oracle, fusion):
    w = synth.WORKLOADS["c0"].replace(steps=160)
    a, ua, _ = _run(oracle, w, fusion=fusion)
    gaps = []

    def hook(u, t):
        kth, k1 = u.last_boundary()
        gaps.append(abs(kth - k1) / max(abs(kth), abs(k1)))

    b, ub, _ = _run(oracle, w, fusion=fusion, recompute=True, hook=hook)
    assert np.abs(a - b).max() < 1e-12
    assert np.array_equal(ua.positions(), ub.positions())
    pa, fa = ua.last_scores()
    pb, fb = ub.last_scores()
    assert np.array_equal(pa, pb) and np.allclose(fa, fb, rtol=1e-11, atol=0)
    assert min(gaps) > 1e-9          # the agreement above is not an accident of ties


# ---- P7: metamorphic ----
def test_key_shift_invariance(oracle):
    w = synth.WORKLOADS["c0"].replace(steps=60)
    rng = np.random.default_rng(0)
    c = rng.normal(size=w.head_dim)
    a, ua, _ = _run(oracle, w)
    b, ub, _ = _run(oracle, w, transform=lambda q, k, v: (q, k + c, v))
    assert np.abs(a - b).max() < 1e-9
    assert np.array_equal(ua.positions(), ub.positions())


def test_value_scaling(oracle):
    w = synth.WORKLOADS["c0"].replace(steps=40)
    a, ua, _ = _run(oracle, w)
    b, ub, _ = _run(oracle, w, transform=lambda q, k, v: (q, k, -3.0 * v))
    assert np.abs(-3.0 * a - b).max() < 1e-12
    assert np.array_equal(ua.positions(), ub.positions())


def test_units_are_independent_mha(oracle):
    # G = 1 (MHA): each head is its own unit; running head 1 alone equals running it beside head 0
    w = TINY.replace(n_q_heads=2, n_kv_heads=2, steps=12)
    a, ua, _ = _run(oracle, w, unit=(0, 0, 1))
    q, k, v = unit_inputs(w, 0, 0, 1, np.arange(w.prompt_len + 12))
    u = oracle.Unit(1, w.head_dim, w.C, w.R, w.fusion)
    u.prefill(k[:6], v[:6], q[:, 4:6])
    b = np.array([u.step(q[:, 6 + s], k[6 + s], v[6 + s]) for s in range(12)])
    assert np.array_equal(a, b)


# ---- P8: prefill ----
def test_prefill_identity_when_everything_fits(oracle):
    w = TINY.replace(prompt_len=9)
    q, k, v = unit_inputs(w, 0, 0, 0, np.arange(9))
    u = oracle.Unit(w.group, w.head_dim, 7, 2, "sum")    # C == P - R exactly
    u.prefill(k, v, q[:, 7:9])
    assert u.positions().tolist() == list(range(9))
    u = oracle.Unit(w.group, w.head_dim, 6, 2, "sum")    # one too many
    u.prefill(k, v, q[:, 7:9])
    assert len(u.positions()) == 8


def test_prefill_window_stats_are_causal_softmax_stats(oracle):
    w = TINY.replace(prompt_len=10)
    q, k, v = unit_inputs(w, 0, 0, 0, np.arange(10))
    u = oracle.Unit(w.group, w.head_dim, 3, 2, "sum")
    u.prefill(k, v, q[:, 8:10])
    for i, r in enumerate((8, 9)):
        for g in range(w.group):
            s = k[: r + 1] @ q[g, r] / np.sqrt(w.head_dim)
            m, l = u.window_stats(r, g)
            assert abs(m - s.max()) < 1e-14 and abs(l - np.exp(s - s.max()).sum()) < 1e-12


# ---- coarse-grained eviction (appendix): policy every T-th step, cache peaks at C + R + T - 1 ----
def test_coarse_grained_eviction_bounds(oracle):
    w = synth.WORKLOADS["c0"].replace(steps=64)
    T = 8
    sizes = []
    _run(oracle, w, T=T, hook=lambda u, t: sizes.append(u.count))
    assert max(sizes) == w.C + w.R + T - 1
    assert sizes[T - 1::T] == [w.C + w.R] * (64 // T)


@pytest.mark.parametrize("fusion", ["sum", "max"])
@pytest.mark.parametrize("T", [2, 3, 8])
@pytest.mark.parametrize("G,C,R,P", [(1, 3, 2, 4), (2, 4, 3, 9), (4, 5, 2, 12), (2, 2, 4, 3)])
def test_coarse_grained_eviction_against_exhaustive_shadow(oracle, fusion, T, G, C, R, P):
    """Which tokens a T-step policy drops, and on which steps: the dictionary shadow (plain sort over all
    candidates, policy on generation steps T, 2T, ...) against the oracle, after every step."""
    w = TINY.replace(n_q_heads=2 * G, prompt_len=P, steps=4 * T + 3, C=C, R=R, fusion=fusion, seed=500 + 7 * G + T)
    q, k, v = unit_inputs(w, 0, 0, 1, np.arange(P + w.steps))
    u = oracle.Unit(G, w.head_dim, C, R, fusion, evict_interval=T)
    sh = ShadowMorphKV(G, w.head_dim, C, R, fusion, evict_interval=T)
    Rw = min(R, P)
    u.prefill(k[:P], v[:P], q[:, P - Rw:P])
    sh.prefill(k[:P], v[:P], q[:, P - Rw:P])
    assert set(u.positions().tolist()) == sh.cached
    policy_steps, multi = [], 0
    for s in range(w.steps):
        t = P + s
        o = u.step(q[:, t], k[t], v[t])
        o2 = sh.step(q[:, t], k[t], v[t])
        assert np.abs(o - o2).max() < 1e-12
        assert set(u.positions().tolist()) == sh.cached, f"step {s + 1}: retained sets differ"
        assert sorted(u.last_evicted().tolist()) == sh.last_dropped, f"step {s + 1}: different tokens dropped"
        if (s + 1) % T != 0:
            assert len(u.last_evicted()) == 0 and len(u.last_scores()[0]) == 0      # no policy between multiples of T
        if sh.last_F is not None:
            policy_steps.append(s + 1)
            multi += len(sh.last_dropped) > 1
            pos, F = u.last_scores()
            assert pos.tolist() == sh.last_ranked                      # full ranking of ALL candidates
            assert np.allclose(F, [sh.last_F[p] for p in pos], rtol=1e-12, atol=1e-300)
            assert best_subset_by_enumeration(sh.last_F, C) == set(sh.last_ranked[:C])
            assert len(sh.cached) == C + R                             # back to C + R after the policy
        assert len(sh.cached) <= C + R + T - 1
    assert policy_steps and all(p % T == 0 for p in policy_steps)
    assert multi > 0                                                   # several tokens dropped at once was exercised


# ---- the other reading of Eq. 4: window rows renormalised over the tokens still cached ("current") ----
@pytest.mark.parametrize("fusion", ["sum", "max"])
@pytest.mark.parametrize("recompute", [False, True])
@pytest.mark.parametrize("G,C,R,P", [(1, 3, 2, 5), (2, 4, 3, 9), (4, 5, 4, 12)])
def test_current_normalisation_against_exhaustive_shadow(oracle, fusion, recompute, G, C, R, P):
    w = TINY.replace(n_q_heads=2 * G, prompt_len=P, steps=16, C=C, R=R, fusion=fusion, seed=900 + G)
    q, k, v = unit_inputs(w, 0, 0, 1, np.arange(P + w.steps))
    u = oracle.Unit(G, w.head_dim, C, R, fusion, recompute=recompute, norm="current")
    sh = ShadowMorphKV(G, w.head_dim, C, R, fusion, norm="current")
    Rw = min(R, P)
    for x in (u, sh):
        x.prefill(k[:P], v[:P], q[:, P - Rw:P])
    assert set(u.positions().tolist()) == sh.cached
    n_sel, rescaled = 0, False
    for s in range(w.steps):
        t = P + s
        o = u.step(q[:, t], k[t], v[t])
        o2 = sh.step(q[:, t], k[t], v[t])
        assert np.abs(o - o2).max() < 1e-12
        assert set(u.positions().tolist()) == sh.cached
        if sh.last_F is not None:
            n_sel += 1
            pos, F = u.last_scores()
            assert pos.tolist() == sh.last_ranked
            assert np.allclose(F, [sh.last_F[p] for p in pos], rtol=1e-11, atol=1e-300)
            # every window row's weights sum to 1 over what the row can still see, so a fused score under "current"
            # is never below the stored-weights score of the same state, and is above it once mass was evicted
            Ffrozen = ShadowMorphKV._fused(_with_norm(sh, "frozen"), set(pos.tolist()))
            assert all(sh.last_F[p] >= Ffrozen[p] * (1 - 1e-12) for p in pos)
            rescaled |= any(sh.last_F[p] > Ffrozen[p] * (1 + 1e-9) for p in pos)
    assert n_sel > 0 and rescaled


def _with_norm(shadow, norm):
    """A view of a shadow's state that scores under the other normalisation (state before the last selection is not
    needed: only weights of tokens still cached plus the just-dropped ones enter, which `profile` still holds)."""
    import copy
    other = copy.copy(shadow)
    other.norm = norm
    # scores are taken before the selection drops anything: restore the candidates of that moment
    other.cached = set(shadow.cached) | set(shadow.last_dropped)
    return other


@pytest.mark.parametrize("fusion", ["sum", "max"])
def test_current_equals_frozen_for_a_window_of_one(oracle, fusion):
    # R = 1: the only window row was generated on this very step, nothing it saw has been evicted since
    w = synth.WORKLOADS["c0"].replace(steps=60)
    a, ua, _ = _run(oracle, w, R=1, fusion=fusion)
    q, k, v = unit_inputs(w, 0, 0, 0, np.arange(w.prompt_len + 60))
    u = oracle.Unit(w.group, w.head_dim, w.C, 1, fusion, norm="current")
    u.prefill(k[:w.prompt_len], v[:w.prompt_len], q[:, w.prompt_len - 1:w.prompt_len])
    b = np.array([u.step(q[:, w.prompt_len + s], k[w.prompt_len + s], v[w.prompt_len + s]) for s in range(60)])
    assert np.array_equal(a, b) and np.array_equal(ua.positions(), u.positions())


def test_current_scales_surviving_weights_by_the_evicted_mass(oracle):
    # one window row (G = 1, R = 2 so that the older row has lived through one eviction): its weight on a survivor
    # is the stored weight divided by 1 - (mass it had on the token evicted meanwhile)
    w = TINY.replace(n_q_heads=2, n_kv_heads=2, prompt_len=6, steps=3, C=3, R=2)
    q, k, v = unit_inputs(w, 0, 0, 0, np.arange(9))
    sh = ShadowMorphKV(1, w.head_dim, 3, 2, "sum", norm="current")
    u = oracle.Unit(1, w.head_dim, 3, 2, "sum", norm="current")
    for x in (u, sh):
        x.prefill(k[:6], v[:6], q[:, 4:6])
    for t in (6, 7):
        u.step(q[:, t], k[t], v[t]); sh.step(q[:, t], k[t], v[t])
    pos, F = u.last_scores()
    older, newer = 6, 7                       # window rows at the selection of step 7
    gone = [p for p in sh.profile[older][0] if p not in sh.cached and p not in sh.last_dropped and p <= older]
    assert gone                               # the older row did see a token that has been evicted since
    lost = sum(sh.profile[older][0][p] for p in gone)
    for p, f in zip(pos, F):
        want = sh.profile[older][0][p] / (1.0 - lost) + sh.profile[newer][0][p]
        assert abs(f - want) < 1e-13


def test_t1_is_default(oracle):
    w = synth.WORKLOADS["c0"].replace(steps=30)
    a, ua, _ = _run(oracle, w)
    b, ub, _ = _run(oracle, w, T=1)
    assert np.array_equal(a, b)


# ---- argument checking ----
def test_rejects_bad_parameters(oracle):
    with pytest.raises(ValueError):
        oracle.Unit(0, 16, 4, 2, "sum")
    u = oracle.Unit(1, 4, 2, 2, "sum")
    with pytest.raises(RuntimeError):
        u.step(np.zeros((1, 4)), np.zeros(4), np.zeros(4))      # decode before prefill


def test_forced_eviction_is_followed(oracle):
    w = TINY.replace(steps=1, prompt_len=8)
    q, k, v = unit_inputs(w, 0, 0, 0, np.arange(9))
    u = oracle.Unit(w.group, w.head_dim, 3, 2, "sum")
    u.prefill(k[:8], v[:8], q[:, 6:8])
    cand = sorted(set(u.positions().tolist()) - {6, 7}) + [6]
    u.step(q[:, 8], k[8], v[8], forced=[cand[0]])
    assert cand[0] not in u.positions().tolist() and u.last_evicted().tolist() == [cand[0]]
    with pytest.raises(RuntimeError):
        u.step(q[:, 8], k[8], v[8], forced=[10 ** 6])
