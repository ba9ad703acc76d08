"""Pins of the fp64 oracle against things other than itself (CPU only).

The paper prints no worked numeric example of Algorithm 1, so the oracle is pinned
by: a library routine in the special case where nothing is evicted, closed forms of
the importance recurrence (Sec. 4.2, Eq. 5) on inputs whose attention is known
analytically, brute force over all subsets for the arg-min of Eq. 8, the limits
beta=0 / beta=1, and the invariants the text states.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import mkv_oracle as O
from workloads.synthetic import CONFIGS, SequenceStream


def sdpa_f64(q, K, V, G):
    """Textbook attention through torch's library routine. q [Hq,d]; K,V [Hkv,N,d]."""
    qt = torch.from_numpy(q)[:, None, :]                       # [Hq,1,d]
    Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)       # head h reads KV head h//G
    Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)
    return torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt)[:, 0, :].numpy()


def rand_problem(rng, Hq, Hkv, d, Lp, T, scale=1.0):
    Kp = rng.standard_normal((Hkv, Lp, d)) * scale
    Vp = rng.standard_normal((Hkv, Lp, d))
    q = rng.standard_normal((T, Hq, d)) * scale
    k = rng.standard_normal((T, Hkv, d)) * scale
    v = rng.standard_normal((T, Hkv, d))
    return Kp, Vp, q, k, v


# ---------------------------------------------------------------- P1: library routine
@pytest.mark.parametrize("Hq,Hkv,d,Lp", [(4, 1, 16, 7), (8, 2, 32, 0), (6, 3, 8, 5)])
def test_no_eviction_equals_full_attention(Hq, Hkv, d, Lp):
    """Budget >= generated length: Eq. 7 gives overflow 0, so every step must be plain
    attention (Eq. 2) over all prefill and all generated tokens."""
    rng = np.random.default_rng(1)
    T = 20
    Kp, Vp, q, k, v = rand_problem(rng, Hq, Hkv, d, Lp, T, scale=1.5)
    o = O.OracleSequence(Hq, Hkv, d, budget=T, beta=0.9, prefill_len=Lp)
    o.prefill(Kp, Vp)
    for t in range(T):
        out = o.step(q[t], k[t], v[t])
        Kall = np.concatenate([Kp, k[: t + 1].transpose(1, 0, 2)], axis=1)
        Vall = np.concatenate([Vp, v[: t + 1].transpose(1, 0, 2)], axis=1)
        ref = sdpa_f64(q[t], Kall, Vall, Hq // Hkv)
        np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-14)
        for g in range(Hkv):
            assert o.count(g) == t + 1


def test_output_uses_pool_before_eviction():
    """Algorithm 1 computes attention before the capacity check: the output of a step
    sees budget+1 decode tokens (the retained set of the previous step plus the fresh
    one), whatever is evicted afterwards."""
    rng = np.random.default_rng(2)
    Hq, Hkv, d, Lp, T, B = 4, 2, 16, 6, 40, 5
    Kp, Vp, q, k, v = rand_problem(rng, Hq, Hkv, d, Lp, T, scale=2.0)
    o = O.OracleSequence(Hq, Hkv, d, budget=B, beta=0.7, prefill_len=Lp)
    o.prefill(Kp, Vp)
    for t in range(T):
        before = [o.decode_kv(g) for g in range(Hkv)]
        out = o.step(q[t], k[t], v[t])
        Kall = np.stack([np.concatenate([Kp[g], before[g][0], k[t, g][None]]) for g in range(Hkv)])
        Vall = np.stack([np.concatenate([Vp[g], before[g][1], v[t, g][None]]) for g in range(Hkv)])
        assert Kall.shape[1] == Lp + min(t, B) + 1
        np.testing.assert_allclose(out, sdpa_f64(q[t], Kall, Vall, Hq // Hkv), rtol=1e-12, atol=1e-14)
        assert all(o.count(g) == min(t + 1, B) for g in range(Hkv))


# ---------------------------------------------------------------- P2: closed forms
def test_update_closed_forms():
    beta, n = 0.9, 37
    # constant attention a: I(n) = a (1 - beta^n) / (1 - beta)
    I = np.zeros(3)
    a = np.array([0.25, 0.01, 1.0])
    for _ in range(n):
        I = O.update(I, a, beta)
    np.testing.assert_allclose(I, a * (1 - beta ** n) / (1 - beta), rtol=1e-13)
    # impulse then silence: I(n) = beta^n
    I = O.update(np.zeros(1), np.ones(1), beta)
    for _ in range(n):
        I = O.update(I, np.zeros(1), beta)
    np.testing.assert_allclose(I, beta ** n, rtol=1e-13)
    # on/off square wave (on 3, off 2), closed form = sum of beta^(age) over "on" steps
    pattern = [1, 1, 1, 0, 0] * 6
    I = np.zeros(1)
    for x in pattern:
        I = O.update(I, np.array([0.5 * x]), beta)
    T = len(pattern)
    expect = sum(0.5 * x * beta ** (T - 1 - s) for s, x in enumerate(pattern))
    np.testing.assert_allclose(I, expect, rtol=1e-13)


@pytest.mark.parametrize("mode", [O.GROUP_MEAN, O.LAYER_MEAN])
def test_uniform_attention_closed_form(mode):
    """All keys zero: every logit is 0, attention is uniform 1/(Lp + n_s), the output is
    the mean of V, I_i(t) = sum_{s=t_i..t} beta^(t-s) / (Lp + n_s) (Eq. 5 unrolled), the
    fresh token always has the strictly lowest score, so once the pool is full the
    cache is exactly the first `budget` generated tokens."""
    rng = np.random.default_rng(3)
    Hq, Hkv, d, Lp, T, B, beta = 4, 2, 8, 5, 30, 6, 0.8
    Kp = np.zeros((Hkv, Lp, d)); Vp = rng.standard_normal((Hkv, Lp, d))
    q = rng.standard_normal((T, Hq, d)); k = np.zeros((T, Hkv, d)); v = rng.standard_normal((T, Hkv, d))
    o = O.OracleSequence(Hq, Hkv, d, budget=B, beta=beta, prefill_len=Lp, mode=mode)
    o.prefill(Kp, Vp)
    n_at = lambda s: min(s + 1, B + 1)
    for t in range(T):
        out = o.step(q[t], k[t], v[t])
        for g in range(Hkv):
            kept = list(range(min(t + 1, B)))
            pool_v = np.concatenate([Vp[g], v[kept, g]] + ([v[t, g][None]] if t >= B else []))
            for r in range(Hq // Hkv):
                np.testing.assert_allclose(out[g * (Hq // Hkv) + r], pool_v.mean(0), rtol=1e-12, atol=1e-14)
            pos, sc, ab = o.decode_state(g)
            assert list(pos) == kept
            expect = [sum(beta ** (t - s) / (Lp + n_at(s)) for s in range(i, t + 1)) for i in kept]
            np.testing.assert_allclose(sc, expect, rtol=1e-12)
            ev_pos, ev_sc = o.last_evicted(g)
            if t >= B:
                assert list(ev_pos) == [t]
                np.testing.assert_allclose(ev_sc, [1.0 / (Lp + B + 1)], rtol=1e-12)
            else:
                assert len(ev_pos) == 0


def _one_hot_problem(targets, Hq, Hkv, Lp, T, d, big=60.0):
    """Token j of KV head g (prefill tokens first, then decode tokens in step order) has
    key sqrt(d)*e_j, so logit(q, key_j) = q[j].  q_h(t) = big * e_{targets[t][h]} makes the
    softmax one-hot up to exp(-big)."""
    assert d >= Lp + T
    Kp = np.zeros((Hkv, Lp, d)); k = np.zeros((T, Hkv, d))
    for g in range(Hkv):
        for j in range(Lp):
            Kp[g, j, j] = np.sqrt(d)
        for t in range(T):
            k[t, g, Lp + t] = np.sqrt(d)
    q = np.zeros((T, Hq, d))
    for t in range(T):
        for h in range(Hq):
            q[t, h, targets[t][h]] = big
    rng = np.random.default_rng(4)
    return Kp, rng.standard_normal((Hkv, Lp, d)), q, k, rng.standard_normal((T, Hkv, d))


def test_head_grouping_and_decode_slice_closed_form():
    """One-hot attention with chosen targets pins (a) which query heads feed which KV
    head (h // G), (b) the 1/G (GROUP) or 1/H (LAYER, Eq. 4 as printed) mean, (c) that
    only the decode slice A[|Phi_p|:] is scored and prefill attention is discarded."""
    Hq, Hkv, Lp, T, d, beta = 4, 2, 3, 6, 16, 0.5
    G = Hq // Hkv
    # targets[t][h] = global token index (0..Lp-1 prefill, Lp+s = decode token of step s)
    targets = [
        [Lp + 0, Lp + 0, Lp + 0, 1],          # t=0: heads 0,1,2 -> fresh token; head 3 -> prefill 1
        [Lp + 0, Lp + 1, 0, Lp + 1],          # t=1
        [Lp + 2, Lp + 2, Lp + 0, Lp + 0],     # t=2
        [2, 2, Lp + 3, Lp + 1],               # t=3: group 0 looks only at prefill
        [Lp + 1, Lp + 4, Lp + 4, Lp + 4],     # t=4
        [Lp + 5, Lp + 0, Lp + 2, Lp + 5],     # t=5
    ]
    Kp, Vp, q, k, v = _one_hot_problem(targets, Hq, Hkv, Lp, T, d)
    for mode in (O.GROUP_MEAN, O.LAYER_MEAN):
        o = O.OracleSequence(Hq, Hkv, d, budget=T, beta=beta, prefill_len=Lp, mode=mode)
        o.prefill(Kp, Vp)
        expect = np.zeros((Hkv, T))
        for t in range(T):
            out = o.step(q[t], k[t], v[t])
            abar = np.zeros((Hkv, T))
            for h in range(Hq):
                tgt = targets[t][h]
                if tgt >= Lp:
                    if mode == O.GROUP_MEAN:
                        abar[h // G, tgt - Lp] += 1.0 / G
                    else:
                        abar[:, tgt - Lp] += 1.0 / Hq
                # output of a one-hot head is the value row of its target
                vt = Vp[h // G, tgt] if tgt < Lp else v[tgt - Lp, h // G]
                np.testing.assert_allclose(out[h], vt, atol=1e-12)
            expect = beta * expect + abar
            for g in range(Hkv):
                _, sc, ab = o.decode_state(g)
                np.testing.assert_allclose(sc, expect[g, : t + 1], atol=1e-12)
                np.testing.assert_allclose(ab, abar[g, : t + 1], atol=1e-12)


def test_eviction_order_hand_built():
    """Budget 3, one KV head, two query heads, one-hot attention.  The scores, and so the
    evictions, follow by hand from Eq. 5-8 (beta = 0.5):
      t=0 both heads on tok0                     I = [1]
      t=1 both on tok1                           I = [.5, 1]
      t=2 h0 tok0, h1 tok2                       I = [.75, .5, .5]
      t=3 both on tok0        I = [1.375, .25, .25, 0(+eps)] -> fresh tok3 (about 0) leaves
      t=4 both on tok4        I = [.6875, .125, .125, 1] -> tie tok1/tok2: older tok1 leaves
      t=5 h0 tok2, h1 tok5    I = [.34375, .5625, .5, .5] (tok0,tok2,tok4,tok5): tok0 leaves
    The last step shows an old, once-dominant token being evicted purely by score, and
    t=4 shows a token older than the fresh one being evicted while the fresh one stays."""
    Lp, T, d = 2, 6, 8
    targets = [[Lp + 0, Lp + 0], [Lp + 1, Lp + 1], [Lp + 0, Lp + 2], [Lp + 0, Lp + 0],
               [Lp + 4, Lp + 4], [Lp + 2, Lp + 5]]
    Kp, Vp, q, k, v = _one_hot_problem(targets, 2, 1, Lp, T, d)
    # make the t=4 tie exact: tokens 1 and 2 must carry bit-identical scores.  Their
    # one-hot leak terms differ by O(exp(-big)); big = 800 makes exp(-big) == 0 in fp64.
    q[q != 0] = 800.0
    o = O.OracleSequence(2, 1, d, budget=3, beta=0.5, prefill_len=Lp)
    o.prefill(Kp, Vp)
    evicted, kept = [], []
    for t in range(T):
        o.step(q[t], k[t], v[t])
        evicted.append(list(o.last_evicted(0)[0]))
        kept.append(list(o.decode_state(0)[0]))
    assert evicted == [[], [], [], [3], [1], [0]]
    assert kept[-1] == [2, 4, 5]
    np.testing.assert_allclose(o.decode_state(0)[1], [0.5625, 0.5, 0.5], atol=1e-12)


# ---------------------------------------------------------------- P4: limits of beta
def test_beta_limits():
    rng = np.random.default_rng(5)
    Hq, Hkv, d, Lp, T = 4, 2, 8, 4, 15
    Kp, Vp, q, k, v = rand_problem(rng, Hq, Hkv, d, Lp, T, scale=2.0)
    o0 = O.OracleSequence(Hq, Hkv, d, budget=T, beta=0.0, prefill_len=Lp)
    o1 = O.OracleSequence(Hq, Hkv, d, budget=T, beta=1.0, prefill_len=Lp)
    o0.prefill(Kp, Vp); o1.prefill(Kp, Vp)
    run_sum = [np.zeros(T) for _ in range(Hkv)]
    for t in range(T):
        o0.step(q[t], k[t], v[t]); o1.step(q[t], k[t], v[t])
        for g in range(Hkv):
            _, sc0, ab0 = o0.decode_state(g)
            np.testing.assert_array_equal(sc0, ab0)            # beta=0: instantaneous attention
            _, sc1, ab1 = o1.decode_state(g)
            run_sum[g][: t + 1] += ab1
            np.testing.assert_allclose(sc1, run_sum[g][: t + 1], rtol=1e-13)  # beta=1: plain accumulation


# ---------------------------------------------------------------- P5: brute force
def test_select_is_the_min_sum_subset_bruteforce():
    """Eq. 8: E = argmin over subsets of size k of the summed importance.  Enumerate all
    subsets; the sort-based choice must reach the minimum and, among minimisers, be the
    lexicographically smallest index set (ties to the older token)."""
    rng = np.random.default_rng(6)
    for trial in range(60):
        n = int(rng.integers(1, 10))
        k = int(rng.integers(0, n + 1))
        if trial % 2:
            score = rng.integers(0, 4, size=n).astype(np.float64) * 0.25   # many ties
        else:
            score = rng.random(n)
        got = sorted(O.select(score, None, k).tolist())
        best, best_sets = None, []
        for S in itertools.combinations(range(n), k):
            tot = float(sum(score[i] for i in S))
            if best is None or tot < best - 1e-15:
                best, best_sets = tot, [S]
            elif abs(tot - best) <= 1e-15:
                best_sets.append(S)
        assert tuple(got) == min(best_sets)


def test_select_ties_use_position_id_not_storage_order():
    score = np.array([0.5, 0.1, 0.1, 0.1])
    pos = np.array([7, 30, 10, 20])
    assert O.select(score, pos, 2).tolist() == [2, 3]       # pos 10 then pos 20


# ---------------------------------------------------------------- P3: invariants
@pytest.mark.parametrize("variant", ["literal", "hot"])
def test_invariants_on_tiny_workload(variant):
    w = CONFIGS["tiny"].with_(variant=variant)
    s = SequenceStream(w, 0, 0)
    Kp, Vp = s.prefill()
    o = O.OracleSequence(w.q_heads, w.kv_heads, w.head_dim, w.budget, w.beta, s.Lp)
    o.prefill(Kp, Vp)
    Kp0, Vp0 = Kp.copy(), Vp.copy()
    q, k, v = s.next(w.steps)
    bound = 1.0 / (1.0 - w.beta)
    prev = set()
    for t in range(w.steps):
        o.attend_update(q[t], k[t], v[t])
        pos, sc, ab = o.decode_state(0)
        assert len(pos) == min(t, w.budget) + 1 and pos[-1] == t
        assert sc[-1] == ab[-1] > 0.0                       # Eq. 6: fresh score = own attention > 0
        assert 0.0 < ab.sum() <= 1.0 + 1e-12                # decode slice of a probability vector
        assert (sc > 0).all() and sc.max() <= bound and sc.sum() <= bound + 1e-9
        o.evict()
        pos2, sc2, _ = o.decode_state(0)
        ev_pos, ev_sc = o.last_evicted(0)
        assert len(pos2) <= w.budget                        # Eq. 3
        assert set(pos2) | set(ev_pos) == prev | {t} and not (set(pos2) & set(ev_pos))
        assert len(set(pos2)) == len(pos2)
        if len(ev_sc):
            assert sc2.min() >= ev_sc.max()                 # retained >= evicted
        prev = set(pos2)
    # frozen prefill pool (Sec. 4.2 "Prefill pool (frozen)")
    import ctypes
    L = O.lib()
    L.mko_prefill_k.restype = ctypes.POINTER(ctypes.c_double)
    L.mko_prefill_v.restype = ctypes.POINTER(ctypes.c_double)
    L.mko_prefill_k.argtypes = L.mko_prefill_v.argtypes = [ctypes.c_void_p]
    n = Kp0.size
    np.testing.assert_array_equal(np.ctypeslib.as_array(L.mko_prefill_k(o._h), (n,)), Kp0.ravel())
    np.testing.assert_array_equal(np.ctypeslib.as_array(L.mko_prefill_v(o._h), (n,)), Vp0.ravel())
    # the planted heavy hitters survive to the end (Sec. 3.1 behaviour the method targets)
    assert all(int(tj) in prev for tj in w.heavy_steps())


def test_no_prefill_probabilities_sum_to_one():
    rng = np.random.default_rng(8)
    Hq, Hkv, d, T = 4, 2, 8, 12
    _, _, q, k, v = rand_problem(rng, Hq, Hkv, d, 0, T)
    o = O.OracleSequence(Hq, Hkv, d, budget=4, beta=0.9, prefill_len=0)
    o.prefill(np.zeros((Hkv, 0, d)), np.zeros((Hkv, 0, d)))
    for t in range(T):
        o.attend_update(q[t], k[t], v[t])
        for g in range(Hkv):
            np.testing.assert_allclose(o.decode_state(g)[2].sum(), 1.0, rtol=1e-13)
        o.evict()


def test_forced_eviction_and_budget_shrink():
    rng = np.random.default_rng(9)
    Hq, Hkv, d, Lp, T = 2, 1, 8, 3, 12
    Kp, Vp, q, k, v = rand_problem(rng, Hq, Hkv, d, Lp, T)
    o = O.OracleSequence(Hq, Hkv, d, budget=8, beta=0.9, prefill_len=Lp)
    o.prefill(Kp, Vp)
    for t in range(8):
        o.step(q[t], k[t], v[t])
    o.set_budget(4)                                         # overflow 5 at the next step (Eq. 7)
    o.attend_update(q[8], k[8], v[8])
    pos, sc, _ = o.decode_state(0)
    want = pos[np.lexsort((pos, sc))[:5]]
    assert sorted(o.choose(0).tolist()) == sorted(want.tolist())
    o.evict()
    assert o.count(0) == 4
    # forcing a different (valid) eviction is honoured
    o.attend_update(q[9], k[9], v[9])
    pos, _, _ = o.decode_state(0)
    o.evict(force=[[int(pos[0])]])
    assert int(pos[0]) not in o.decode_state(0)[0] and o.count(0) == 4


@pytest.mark.parametrize("mode", [O.GROUP_MEAN, O.LAYER_MEAN])
def test_loaded_state_continues_like_the_uninterrupted_run(mode):
    """The state loader holds no arithmetic: an oracle whose decode pools are loaded from
    another oracle's state (in a different slot order: Algorithm 1 does not depend on the order
    of the pool, and ties go by position id) continues with exactly the same evictions and, up
    to summation order, the same outputs and scores."""
    rng = np.random.default_rng(21)
    Hq, Hkv, d, Lp, T0, T1, budget = 6, 2, 16, 9, 20, 12, 7
    Kp, Vp, q, k, v = rand_problem(rng, Hq, Hkv, d, Lp, T0 + T1, scale=1.5)
    a = O.OracleSequence(Hq, Hkv, d, budget, 0.85, Lp, mode)
    a.prefill(Kp, Vp)
    for t in range(T0):
        a.step(q[t], k[t], v[t])
    b = O.OracleSequence(Hq, Hkv, d, budget, 0.85, Lp, mode)
    b.prefill(Kp, Vp)
    perm = rng.permutation(budget)                           # the same order in every KV head
    for g in range(Hkv):
        pos, sc, _ = a.decode_state(g)
        Kd, Vd = a.decode_kv(g)
        b.load_decode_state(g, Kd[perm], Vd[perm], sc[perm], pos[perm], T0)
    assert b.steps_done() == T0
    for t in range(T0, T0 + T1):
        oa, ob = a.attend_update(q[t], k[t], v[t]), b.attend_update(q[t], k[t], v[t])
        np.testing.assert_allclose(ob, oa, rtol=1e-12, atol=1e-14)
        for g in range(Hkv):
            assert sorted(a.choose(g).tolist()) == sorted(b.choose(g).tolist())
        a.evict(); b.evict()
        for g in range(Hkv):
            pa, sa, _ = a.decode_state(g)
            pb, sb, _ = b.decode_state(g)
            np.testing.assert_array_equal(np.sort(pa), np.sort(pb))
            np.testing.assert_allclose(sb[np.argsort(pb)], sa[np.argsort(pa)], rtol=1e-12)
