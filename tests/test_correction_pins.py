"""Pins of the correction oracle (Eq. 2, 4, 5, 6, 16, 17) against what the paper and the
mathematics fix: a hand-worked example, closed forms and invariants, brute force."""
import json
import os

import numpy as np
import pytest

from oracle import correction_oracle as C

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")))["correction"]


def test_hand_example():
    p_d, p_t = C.softmax(GOLD["z_d"]), C.softmax(GOLD["z_t"])
    assert np.allclose(p_d, GOLD["p_d"], atol=1e-12) and np.allclose(p_t, GOLD["p_t"], atol=1e-12)
    assert C.margin(p_d) == pytest.approx(GOLD["margin"], abs=1e-12)
    assert C.gate(C.margin(p_d), 0.25) == 0 and C.gate(C.margin(p_d), 0.35) == 1
    r, mass = C.residual(p_t, p_d)
    assert mass == pytest.approx(GOLD["resid_mass"], abs=1e-12) and np.allclose(r, GOLD["r"], atol=1e-12)
    assert C.accept_probability(p_t, p_d, 2) == pytest.approx(GOLD["accept_token2"], abs=1e-12)
    assert C.accept_probability(p_t, p_d, 0) == GOLD["accept_token0"]
    for x, w in GOLD["samples"]:
        assert C.sample(r, x) == w


def test_softmax_invariants():
    rng = np.random.default_rng(0)
    z = rng.normal(size=1000) * 4
    p = C.softmax(z)
    assert p.sum() == pytest.approx(1.0, abs=1e-12) and (p > 0).all()
    assert np.allclose(C.softmax(z + 123.4), p, rtol=1e-12)            # shift invariance
    assert np.argmax(p) == np.argmax(z)
    assert np.allclose(np.log(p[1:] / p[:-1]), z[1:] - z[:-1], atol=1e-9)   # ratios follow the logits
    assert np.allclose(C.softmax(np.zeros(7)), 1 / 7)


def test_margin_and_gate():
    assert C.margin([0.5, 0.5]) == 0.0                                  # tie: no margin
    assert C.margin([0.7, 0.1, 0.2]) == pytest.approx(0.5)
    assert C.gate(0.3, 0.3) == 0 and C.gate(0.2999, 0.3) == 1           # m >= gamma commits locally
    p = C.softmax([10.0, 0.0, 0.0])
    assert C.margin(p) == pytest.approx((np.e ** 10 - 1) / (np.e ** 10 + 2))


def test_accept_or_resample_reproduces_the_target_distribution():
    # Speculative sampling is exact: p_d(w) a(w) + (1 - sum_u p_d(u) a(u)) r(w) = p_t(w) for all w.
    rng = np.random.default_rng(1)
    for n in (2, 5, 300):
        p_d, p_t = C.softmax(rng.normal(size=n) * 3), C.softmax(rng.normal(size=n) * 3)
        a = np.array([C.accept_probability(p_t, p_d, w) for w in range(n)])
        r, mass = C.residual(p_t, p_d)
        out = p_d * a + (1.0 - (p_d * a).sum()) * r
        assert np.allclose(out, p_t, atol=1e-14)
        assert mass == pytest.approx(1.0 - (p_d * a).sum(), abs=1e-14)  # rejection probability
        assert mass == pytest.approx(0.5 * np.abs(p_t - p_d).sum(), abs=1e-14)   # total variation
        assert r.sum() == pytest.approx(1.0, abs=1e-12) and (r[p_d >= p_t] == 0).all()


def test_identical_distributions_fall_back_to_the_target():
    p = C.softmax([0.3, -1.0, 2.0])
    r, mass = C.residual(p, p)
    assert mass == 0.0 and np.array_equal(r, p)
    assert C.accept_probability(p, p, 1) == 1.0


def test_inverse_cdf_brute_force():
    rng = np.random.default_rng(2)
    r = rng.random(50)
    r[rng.random(50) < 0.5] = 0.0
    r /= r.sum()
    for x in np.concatenate([rng.random(200), [0.0, 0.999999999]]):
        acc, want = 0.0, None
        for w, v in enumerate(r):
            acc += v
            if acc > x and want is None:
                want = w
        if want is None:
            want = int(np.nonzero(r)[0][-1])
        got = C.sample(r, x)
        assert got == want or abs(np.cumsum(r)[min(got, want)] - x) < 1e-12
        assert r[got] > 0                                              # never a zero-probability token


def test_sampling_frequencies_follow_the_residual():
    rng = np.random.default_rng(3)
    p_d, p_t = C.softmax(rng.normal(size=6)), C.softmax(rng.normal(size=6))
    r, _ = C.residual(p_t, p_d)
    xs = (np.arange(20000) + 0.5) / 20000                              # stratified uniforms
    counts = np.bincount([C.sample(r, x) for x in xs], minlength=6) / len(xs)
    assert np.allclose(counts, r, atol=1e-4)


def test_correct_position_bundles_the_definitions():
    out = C.correct_position(GOLD["z_d"], GOLD["z_t"], 0.75, 0.35, y=2)
    assert out["token"] == 3 and out["gate"] == 1 and out["accept"] == pytest.approx(0.4)


def test_fanout_sequence():
    # Eq. 23 by hand: F_0 = 8, rho = 0.5 -> 8, 4, 2, 1, ceil(0.5) = 1; F_0 = 5, rho = 0.7 -> 5, 4, 3, 2, 2
    assert [C.fanout(8, 0.5, j) for j in range(5)] == [8, 4, 2, 1, 1]
    assert [C.fanout(5, 0.7, j) for j in range(5)] == [5, 4, 3, 2, 2]
    assert C.fanout(3, 0.999999, 0) == 3


def test_bonus_candidates_hand_and_brute_force():
    z = [0.5, 2.0, 2.0, -1.0, 3.0, 2.0]
    assert C.bonus_candidates(z, 4, 2).tolist() == [1, 2]        # 3.0 is drafted; ties 2.0 -> lowest ids
    assert C.bonus_candidates(z, None, 3).tolist() == [1, 2, 4]
    assert C.bonus_candidates(z, 1, 3).tolist() == [2, 4, 5]
    rng = np.random.default_rng(5)
    zr = np.round(rng.normal(size=40), 1)                         # many ties
    for y in (None, 0, 17):
        got = C.bonus_candidates(zr, y, 7)
        assert len(set(got.tolist())) == 7 and (y is None or y not in got)
        rest = [w for w in range(40) if w not in got and w != y]
        assert min(zr[got]) >= max(zr[rest])                      # nothing outside beats anything inside
