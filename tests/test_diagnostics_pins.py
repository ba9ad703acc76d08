"""Pins of the recency-window diagnostics oracle against things other than itself (CPU only).

The paper shows the analysis as figures (Sec. 3.2, Sec. 7.1) and prints no numbers for it, so
the oracle is pinned by closed forms (uniform, one-hot and geometric attention), by exact
window counts, by the properties every such curve has, and -- through the Algorithm 1 oracle
-- by the fact that the attention of a step sums to one over prompt and generated tokens.
"""
import numpy as np
import pytest

from oracle import mkv_diagnostics as D
from oracle import mkv_oracle as O


def test_uniform_attention_gives_the_uniform_baseline():
    """Equal attention on every token of the window: the curve is the straight line the paper
    draws as its baseline, and the mass is count times the common value."""
    t, W = 99, 32
    pos = np.arange(100)
    mass, count, curve = D.recency_window(np.full(100, 0.004), pos, t, W)
    assert count == W
    assert mass == pytest.approx(W * 0.004, rel=1e-12)
    np.testing.assert_allclose(curve, D.uniform_baseline(W), rtol=1e-12)


def test_all_attention_on_one_token_saturates_at_once():
    pos = np.arange(50)
    ab = np.zeros(50)
    ab[41] = 0.3
    mass, count, curve = D.recency_window(ab, pos, 49, 16)
    assert count == 16 and mass == pytest.approx(0.3)
    np.testing.assert_allclose(curve, np.ones(16))
    # the attended token lies outside a shorter window: nothing left inside
    mass, count, curve = D.recency_window(ab, pos, 49, 8)
    assert count == 8 and mass == 0.0 and not curve.any()


@pytest.mark.parametrize("r", [0.5, 0.9])
def test_geometric_attention_closed_form(r):
    """abar_i = c r^age: the j+1 most attended tokens are the j+1 youngest, so
    curve[j] = (1 - r^(j+1)) / (1 - r^count) and mass = c (1 - r^count) / (1 - r)."""
    t, W, c = 199, 64, 0.01
    pos = np.arange(200)
    ab = c * r ** (t - pos)
    rng = np.random.default_rng(0)
    perm = rng.permutation(200)                       # slot order must not matter
    mass, count, curve = D.recency_window(ab[perm], pos[perm], t, W)
    assert count == W
    assert mass == pytest.approx(c * (1 - r ** W) / (1 - r), rel=1e-12)
    j = np.arange(W)
    np.testing.assert_allclose(curve, (1 - r ** (j + 1)) / (1 - r ** W), rtol=1e-12)


def test_window_counts_are_exact_at_the_edges():
    """The window holds the token of the current step and the W-1 before it -- no more, no
    fewer -- and only those still cached."""
    t = 20
    pos = np.arange(t + 1)
    ab = np.full(t + 1, 0.01)
    for W in (1, 2, 5, 21, 22, 1000):
        _, count, _ = D.recency_window(ab, pos, t, W)
        assert count == min(W, t + 1)
    _, count, _ = D.recency_window(ab, pos, t, 1)
    assert count == 1                                   # only the fresh token
    keep = np.array([0, 3, 15, 18, 20])                 # the rest was evicted
    mass, count, _ = D.recency_window(ab[keep], pos[keep], t, 6)    # ids 15..20 qualify
    assert count == 3 and mass == pytest.approx(0.03)


def test_curve_properties_on_random_attention():
    """Non-decreasing, ends at one, concave (increments sorted), at or above the uniform
    baseline; the mass grows with the window and equals the total for a window that holds all."""
    rng = np.random.default_rng(3)
    n, t = 300, 400
    pos = np.sort(rng.choice(t + 1, size=n, replace=False))
    ab = rng.random(n) ** 4
    ab *= 0.6 / ab.sum()
    last = -1.0
    for W in (1, 7, 64, 256, 401):
        mass, count, curve = D.recency_window(ab, pos, t, W)
        assert count == int(((pos > t - W) & (pos <= t)).sum())
        assert mass >= last
        last = mass
        if count:
            inc = np.diff(np.concatenate([[0.0], curve]))
            assert (inc >= -1e-15).all() and (np.diff(inc) <= 1e-15).all()
            assert curve[-1] == pytest.approx(1.0, rel=1e-12)
            assert (curve >= D.uniform_baseline(count) - 1e-12).all()
    assert last == pytest.approx(0.6, rel=1e-12)


def test_mass_is_a_share_of_the_steps_attention():
    """With a window that holds every generated token, the mass and the attention the prompt
    received add up to one: the per-token values are those of Eq. 4, whose softmax (Eq. 2) runs
    over prompt and generated tokens together.  The prompt's share is computed here from the
    textbook softmax, independently of the oracle."""
    rng = np.random.default_rng(5)
    Hq, Hkv, d, Lp, T = 4, 2, 16, 9, 12
    G = Hq // Hkv
    Kp = rng.standard_normal((Hkv, Lp, d))
    Vp = rng.standard_normal((Hkv, Lp, d))
    q = rng.standard_normal((T, Hq, d)) * 2.0
    k = rng.standard_normal((T, Hkv, d))
    v = rng.standard_normal((T, Hkv, d))
    o = O.OracleSequence(Hq, Hkv, d, budget=T, beta=0.9, prefill_len=Lp)
    o.prefill(Kp, Vp)
    for t in range(T):
        o.attend_update(q[t], k[t], v[t])
        for g in range(Hkv):
            pos, _, ab = o.decode_state(g)
            mass, count, _ = D.recency_window(ab, pos, t, T + 5)
            assert count == t + 1
            keys = np.concatenate([Kp[g], k[: t + 1, g]], axis=0)
            prompt_share = 0.0
            for h in range(g * G, (g + 1) * G):
                s = keys @ q[t, h] / np.sqrt(d)
                p = np.exp(s - s.max())
                p /= p.sum()
                prompt_share += p[:Lp].sum() / G
            assert mass + prompt_share == pytest.approx(1.0, abs=1e-12)
        o.evict()
