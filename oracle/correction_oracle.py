"""CPU oracle for the device-side gating and correction step of CoVSpec (Eq. 2, 4, 5, 6, 16, 17 and
Sec. III-C.2: the device completes residual sampling locally from its own draft logits and the
target logits of the first rejected position).

TEST INFRASTRUCTURE ONLY: float64 numpy, one definition per function, no fusion.  Shares no code
with the CUDA library; imported only by the tests and the benchmark's CPU-baseline leg.

Pinned by tests/test_correction_pins.py: a hand-worked example, softmax invariances, the identity
that accept-or-resample reproduces the target distribution exactly, brute-force inverse CDF.
Reading where the paper is silent: when the residual of Eq. 6 is identically zero (target and draft
distributions coincide) the correction is drawn from the target distribution; ties between the two
largest draft probabilities give margin 0; the sample for a uniform number x in [0, 1) is the first
token whose cumulative residual exceeds x.
"""
from __future__ import annotations

import numpy as np


def softmax(z):
    """Eq. 2 / Eq. 4: p(w) = exp(z_w) / sum_u exp(z_u)."""
    z = np.asarray(z, dtype=np.float64)
    e = np.exp(z - z.max())
    return e / e.sum()


def margin(p_d):
    """Eq. 16: largest minus second-largest probability of the draft distribution."""
    s = np.sort(np.asarray(p_d, dtype=np.float64))
    return float(s[-1] - s[-2]) if len(s) > 1 else float(s[-1])


def gate(m, gamma):
    """Eq. 17: 1 (verify) when the margin is below the threshold, else 0 (commit locally)."""
    return 1 if m < gamma else 0


def accept_probability(p_t, p_d, y):
    """Eq. 5: min(1, p_t(y) / p_d(y))."""
    return float(min(1.0, p_t[y] / p_d[y])) if p_d[y] > 0.0 else 1.0


def residual(p_t, p_d):
    """Eq. 6: max(p_t - p_d, 0) normalised; returns (r, mass) with mass the normalising sum."""
    pos = np.maximum(np.asarray(p_t, dtype=np.float64) - np.asarray(p_d, dtype=np.float64), 0.0)
    mass = pos.sum()
    if mass == 0.0:
        return np.asarray(p_t, dtype=np.float64).copy(), 0.0
    return pos / mass, float(mass)


def sample(r, x):
    """Inverse CDF: the first token whose cumulative probability exceeds x (x in [0, 1))."""
    c = np.cumsum(np.asarray(r, dtype=np.float64))
    w = int(np.searchsorted(c, x * c[-1], side="right"))
    last = int(np.nonzero(r)[0][-1])
    return min(w, last)


def correct_position(z_d, z_t, x, gamma, y=None):
    """One position: everything the device computes from the two logit rows."""
    p_d, p_t = softmax(z_d), softmax(z_t)
    m = margin(p_d)
    r, mass = residual(p_t, p_d)
    out = dict(margin=m, gate=gate(m, gamma), resid_mass=mass, token=sample(r, x), cdf=np.cumsum(r))
    if y is not None:
        out["accept"] = accept_probability(p_t, p_d, int(y))
    return out


def fanout(f0, rho, j):
    """Eq. 23: F_j = ceil(F_0 * rho^j)."""
    import math
    return int(math.ceil(f0 * rho ** j - 1e-9))


def bonus_candidates(z_d, y, f):
    """Sec. III-C.1: the f largest draft logits, the drafted token y excluded (y None: nothing
    excluded); equal logits are taken in order of increasing token id; ids returned ascending."""
    z = np.asarray(z_d, dtype=np.float64)
    order = sorted((w for w in range(len(z)) if w != y), key=lambda w: (-z[w], w))
    return np.array(sorted(order[:f]), dtype=np.int64)
