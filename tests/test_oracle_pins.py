"""Pins of the CPU oracle against what the paper's definitions and the mathematics fix: hand-worked
values (tests/golden/hand_examples.json), closed forms, invariances, brute force on tiny inputs and
independently written algorithms.  No GPU, no compiled library."""
import itertools
import json
import math
import os

import numpy as np
import pytest

from oracle import covspec_oracle as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")))
RNG = np.random.default_rng(1234)


def A(x):
    return np.asarray(x, dtype=np.float64)


# ------------------------------------------------------------------ Eq. 10
def test_eq10_hand_identity():
    g = GOLD["eq10_identity"]
    np.testing.assert_allclose(O.query_relevance(A(g["X"]), A(g["Q"])), g["S_query"], atol=1e-15)


def test_eq10_hand_two_heads():
    g = GOLD["eq10_two_heads"]
    W = A(g["W"])
    kw = dict(Wq=W, Wk=W, n_heads=g["n_heads"], head_dim=g["head_dim"])
    np.testing.assert_allclose(O.query_relevance(A(g["X"]), A(g["Q"]), **kw),
                               g["S_query_max"], atol=1e-15)
    np.testing.assert_allclose(O.query_relevance(A(g["X"]), A(g["Q"]), head_reduce="mean", **kw),
                               g["S_query_mean"], atol=1e-15)


def test_eq10_weight_orientation():
    # e(x) = W x with W [P, d]: a projection that keeps coordinate 2 only (P=1... padded to 2)
    X = A([[5, 1, 2], [7, -3, -1]])
    Q = A([[0, 0, 1]])
    W = A([[0, 0, 1], [0, 0, 0]])          # [P=2, d=3], one head of width 2
    s = O.query_relevance(X, Q, Wq=W, Wk=W, n_heads=1, head_dim=2)
    np.testing.assert_allclose(s, [1.0, -1.0], atol=1e-15)


def _loops_eq10(X, Q, Wq, Wk, H, hd):
    """Eq. 10 spelled with scalar loops."""
    N, d = X.shape
    out = []
    for i in range(N):
        best = -math.inf
        for j in range(Q.shape[0]):
            for h in range(max(H, 1)):
                if H == 0:
                    ev, eq = list(X[i]), list(Q[j])
                else:
                    ev = [sum(Wk[h * hd + k][c] * X[i][c] for c in range(d)) for k in range(hd)]
                    eq = [sum(Wq[h * hd + k][c] * Q[j][c] for c in range(d)) for k in range(hd)]
                num = sum(a * b for a, b in zip(ev, eq))
                den = math.sqrt(sum(a * a for a in ev)) * math.sqrt(sum(b * b for b in eq))
                best = max(best, num / den if den > 0 else 0.0)
        out.append(best)
    return np.array(out)


@pytest.mark.parametrize("H,hd", [(0, 0), (1, 3), (3, 2)])
def test_eq10_vs_scalar_loops(H, hd):
    N, T, d = 7, 4, 5
    X, Q = RNG.normal(size=(N, d)), RNG.normal(size=(T, d))
    Wq = RNG.normal(size=(max(H * hd, 1), d))
    Wk = RNG.normal(size=(max(H * hd, 1), d))
    got = O.query_relevance(X, Q, Wq if H else None, Wk if H else None, H, hd)
    np.testing.assert_allclose(got, _loops_eq10(X, Q, Wq, Wk, H, hd), rtol=1e-12, atol=1e-14)


def test_eq10_bounds_and_invariances():
    N, T, d, H, hd = 40, 6, 16, 2, 4
    X, Q = RNG.normal(size=(N, d)), RNG.normal(size=(T, d))
    Wq, Wk = RNG.normal(size=(H * hd, d)), RNG.normal(size=(H * hd, d))
    kw = dict(Wq=Wq, Wk=Wk, n_heads=H, head_dim=hd)
    s = O.query_relevance(X, Q, **kw)
    assert s.shape == (N,) and np.all(s <= 1 + 1e-12) and np.all(s >= -1 - 1e-12)
    # positive rescaling of any token, any query element, any head of either map
    sv = np.exp(RNG.normal(size=(N, 1)))
    sq = np.exp(RNG.normal(size=(T, 1)))
    np.testing.assert_allclose(O.query_relevance(X * sv, Q * sq, **kw), s, rtol=1e-12)
    Wk2 = Wk.copy()
    Wk2[:hd] *= 7.5
    Wq2 = Wq.copy()
    Wq2[hd:] *= 0.01
    np.testing.assert_allclose(
        O.query_relevance(X, Q, Wq=Wq2, Wk=Wk2, n_heads=H, head_dim=hd), s, rtol=1e-12)
    # token permutation permutes the scores
    p = RNG.permutation(N)
    np.testing.assert_allclose(O.query_relevance(X[p], Q, **kw), s[p], rtol=1e-12)
    # more query elements can only raise the max
    s_more = O.query_relevance(X, np.vstack([Q, RNG.normal(size=(3, d))]), **kw)
    assert np.all(s_more >= s - 1e-15)


def test_eq10_special_cases():
    d = 8
    X = RNG.normal(size=(5, d))
    # a query element equal to (a positive multiple of) token 2 => that token scores exactly 1
    Q = np.vstack([RNG.normal(size=(2, d)), 3.0 * X[2]])
    s = O.query_relevance(X, Q)
    assert abs(s[2] - 1.0) < 1e-14
    # a query element equal to minus a token is the worst possible match for it
    s = O.query_relevance(X, -X[1:2])
    assert abs(s[1] + 1.0) < 1e-14
    # queries orthogonal to every token => 0
    Xo = np.zeros((3, 6))
    Xo[:, :3] = RNG.normal(size=(3, 3))
    Qo = np.zeros((2, 6))
    Qo[:, 3:] = RNG.normal(size=(2, 3))
    np.testing.assert_allclose(O.query_relevance(Xo, Qo), 0.0, atol=1e-15)


# ------------------------------------------------------------------ Eq. 11
def test_eq11_hand():
    g = GOLD["eq11"]
    np.testing.assert_allclose(O.token_activity([A(h) for h in g["Hs"]]), g["S_act"], atol=1e-14)


def test_eq11_constructed_steps():
    N, d, K = 9, 12, 5
    u = RNG.normal(size=(N, d))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    a = RNG.normal(size=(K, N))
    Hs = [RNG.normal(size=(N, d))]
    for l in range(K):
        Hs.append(Hs[-1] + a[l][:, None] * u)
    s = O.token_activity(Hs)
    np.testing.assert_allclose(s, np.abs(a).mean(axis=0), rtol=1e-10)
    # adding one constant vector to every snapshot changes nothing
    c = RNG.normal(size=(1, d))
    np.testing.assert_allclose(O.token_activity([h + c for h in Hs]), s, rtol=1e-10)
    # global scaling by alpha scales by |alpha|
    np.testing.assert_allclose(O.token_activity([-2.5 * h for h in Hs]), 2.5 * s, rtol=1e-12)
    # K = 1 is a plain row norm of the difference
    np.testing.assert_allclose(O.token_activity(Hs[:2]), np.linalg.norm(Hs[1] - Hs[0], axis=1),
                               rtol=1e-12)
    # the order of the layers matters only through consecutive pairs: reversing keeps the score
    np.testing.assert_allclose(O.token_activity(Hs[::-1]), s, rtol=1e-12)


# ------------------------------------------------------------------ Eq. 12
def test_eq12_hand():
    g = GOLD["eq12"]
    np.testing.assert_allclose(O.fuse(A(g["S_query"]), A(g["S_act"]), g["lam"]), g["S"], atol=1e-15)


def test_eq12_zscore_hand():
    # the z-score reading divides by the population deviation; the sample deviation (n - 1) or a
    # missing mean would fail these hand-worked values
    g = GOLD["eq12_zscore"]
    np.testing.assert_allclose(O.normalise(A(g["S"]), "zscore"), g["z"], atol=1e-15)
    np.testing.assert_allclose(O.normalise(A(g["S3"]), "zscore"), g["z3"], atol=1e-15)
    np.testing.assert_allclose(O.fuse(A(g["S3"]), A(g["S3_act"]), g["lambda"], "zscore"), g["fused3"],
                               atol=1e-15)
    # zero mean, unit population variance, invariant to a positive affine change; constant -> 0
    z = O.normalise(RNG.normal(size=40) * 3 + 7, "zscore")
    assert abs(z.mean()) < 1e-14 and abs(np.mean(z * z) - 1.0) < 1e-13
    s = RNG.normal(size=40)
    np.testing.assert_allclose(O.normalise(5 * s - 2, "zscore"), O.normalise(s, "zscore"), atol=1e-13)
    np.testing.assert_allclose(O.normalise(np.full(5, 3.0), "zscore"), np.zeros(5), atol=0)
    np.testing.assert_allclose(O.normalise(A(g["S3"]), "none"), g["S3"], atol=0)


def test_eq12_properties():
    sq, sa = RNG.normal(size=50), np.abs(RNG.normal(size=50))
    s = O.fuse(sq, sa, 0.3)
    assert s.min() >= 0 and s.max() <= 1
    # lambda = 1 / 0 reduce to a single ranking
    assert list(np.argsort(-O.fuse(sq, sa, 1.0), kind="stable")) == list(np.argsort(-sq, kind="stable"))
    assert list(np.argsort(-O.fuse(sq, sa, 0.0), kind="stable")) == list(np.argsort(-sa, kind="stable"))
    # invariant to a positive affine change of either raw score
    np.testing.assert_allclose(O.fuse(3 * sq + 5, 0.1 * sa - 2, 0.3), s, rtol=1e-12, atol=1e-14)
    # a constant score normalises to zero
    np.testing.assert_allclose(O.fuse(np.full(50, 2.0), sa, 0.3), 0.7 * O.normalise(sa), atol=1e-15)
    # no activity stack: the fused score is the normalised query score
    np.testing.assert_allclose(O.fuse(sq, None, 0.3), O.normalise(sq), atol=0)


# ------------------------------------------------------------------ top-k
def test_topk_ties_and_order():
    assert list(O.top_k([1, 3, 3, 3, 0], 2)) == [1, 2]
    assert list(O.top_k([1, 3, 3, 3, 0], 4)) == [0, 1, 2, 3]
    assert list(O.top_k([5, 4, 9, 9, 1], 1)) == [2]
    assert list(O.top_k([2.0, 2.0, 2.0], 3)) == [0, 1, 2]
    assert list(O.top_k([0.5], 1)) == [0]


def test_topk_brute_force():
    for n in range(1, 9):
        s = RNG.integers(0, 4, size=n).astype(float)     # many ties
        for k in range(1, n + 1):
            got = O.top_k(s, k)
            assert len(got) == k and len(set(got)) == k and list(got) == sorted(got)
            best = max(sum(s[list(c)]) for c in itertools.combinations(range(n), k))
            assert sum(s[got]) == best
            # among the maximising subsets, ties go to the lower index: lexicographically smallest
            cands = [c for c in itertools.combinations(range(n), k) if sum(s[list(c)]) == best]
            # rank by (scores descending, then index): the chosen set is the first k of that order
            order = sorted(range(n), key=lambda i: (-s[i], i))[:k]
            assert tuple(sorted(order)) in cands and tuple(got) == tuple(sorted(order))


# ------------------------------------------------------------------ Eq. 13-15
def test_eq15_hand():
    g = GOLD["eq15_2x2"]
    c, s = O.subspace_energy(A(g["Z"]), g["r"])
    np.testing.assert_allclose(c, g["c"], rtol=1e-13)
    np.testing.assert_allclose(s ** 2, g["svals_sq"], rtol=1e-13)
    g = GOLD["eq15_orthogonal"]
    c, _ = O.subspace_energy(A(g["Z"]), g["r"])
    np.testing.assert_allclose(c, g["c"], atol=1e-13)


def test_eq13_stack_is_d_by_M():
    X = RNG.normal(size=(10, 4))
    Z = O.stack(X, [7, 2, 5])
    assert Z.shape == (4, 3)
    np.testing.assert_array_equal(Z[:, 0], X[7])
    np.testing.assert_array_equal(Z[:, 2], X[5])


def _power_iteration_energy(Z, r, iters=3000):
    """c_i from r rounds of scalar power iteration with deflation on G = Z^T Z (own loops)."""
    M = Z.shape[1]
    G = [[float(np.dot(Z[:, i], Z[:, j])) for j in range(M)] for i in range(M)]
    c = [0.0] * M
    for _ in range(r):
        v = [1.0 / (1 + i) for i in range(M)]
        lam = 0.0
        for _ in range(iters):
            w = [sum(G[i][j] * v[j] for j in range(M)) for i in range(M)]
            nrm = math.sqrt(sum(x * x for x in w))
            if nrm == 0:
                break
            v = [x / nrm for x in w]
            lam = nrm
        for i in range(M):
            c[i] += lam * v[i] * v[i]
            for j in range(M):
                G[i][j] -= lam * v[i] * v[j]
    return np.array(c)


def test_eq15_vs_power_iteration():
    d, M, r = 6, 5, 2
    Z = RNG.normal(size=(d, M)) * np.array([3.0, 1.0, 2.0, 0.5, 1.5])[None, :]
    c, _ = O.subspace_energy(Z, r)
    np.testing.assert_allclose(c, _power_iteration_energy(Z, r), rtol=1e-8)


def test_eq15_closed_forms():
    d, M, r = 20, 12, 4
    # exactly rank <= r: every token lies in the retained subspace, c_i = ||z_i||^2
    Z = RNG.normal(size=(d, r)) @ RNG.normal(size=(r, M))
    c, s = O.subspace_energy(Z, r)
    np.testing.assert_allclose(c, np.sum(Z * Z, axis=0), rtol=1e-10)
    # all columns equal, r = 1
    a = RNG.normal(size=(d, 1))
    c, _ = O.subspace_energy(np.repeat(a, 5, axis=1), 1)
    np.testing.assert_allclose(c, np.full(5, float((a * a).sum())), rtol=1e-12)
    # orthogonal columns with distinct norms (random rotation of a scaled partial identity)
    Rm, _ = np.linalg.qr(RNG.normal(size=(d, d)))
    norms = np.array([5.0, 0.5, 3.0, 4.0, 1.0, 2.0])
    Z = Rm[:, :6] * norms[None, :]
    c, _ = O.subspace_energy(Z, 3)
    np.testing.assert_allclose(c, [25.0, 0, 9.0, 16.0, 0, 0], atol=1e-10)


def test_eq15_sums_bounds_invariances():
    d, M, r = 15, 11, 4
    Z = RNG.normal(size=(d, M))
    c, s = O.subspace_energy(Z, r)
    # squared singular values from an independent route: eigenvalues of the d x d matrix Z Z^T
    ev = np.sort(np.linalg.eigvalsh(Z @ Z.T))[::-1]
    np.testing.assert_allclose(c.sum(), ev[:r].sum(), rtol=1e-10)
    col2 = np.sum(Z * Z, axis=0)
    assert np.all(c >= -1e-12) and np.all(c <= col2 + 1e-12)
    # Eckart-Young: total residual = discarded spectrum, and no other rank-r subspace does better
    np.testing.assert_allclose((col2 - c).sum(), ev[r:].sum(), rtol=1e-9)
    for _ in range(20):
        Ub, _ = np.linalg.qr(RNG.normal(size=(d, r)))
        assert np.sum((Ub.T @ Z) ** 2) <= c.sum() + 1e-10
    # c_i is the energy of z_i inside the top-r left singular subspace (from Z Z^T's eigenvectors)
    w, Uf = np.linalg.eigh(Z @ Z.T)
    Ur = Uf[:, np.argsort(-w)[:r]]
    np.testing.assert_allclose(c, np.sum((Ur.T @ Z) ** 2, axis=0), rtol=1e-9)
    # rotation of the feature space leaves c unchanged; permuting tokens permutes c
    Rm, _ = np.linalg.qr(RNG.normal(size=(d, d)))
    np.testing.assert_allclose(O.subspace_energy(Rm @ Z, r)[0], c, rtol=1e-9)
    p = RNG.permutation(M)
    np.testing.assert_allclose(O.subspace_energy(Z[:, p], r)[0], c[p], rtol=1e-9)
    # r = min(M, d) - 0 would keep everything; the largest admissible r keeps less than all
    c_all, _ = O.subspace_energy(Z, M)
    np.testing.assert_allclose(c_all, col2, rtol=1e-10)


# ------------------------------------------------------------------ budgets and the whole request
def test_budgets():
    assert O.budgets(576, 64, 1024) == (64, 128, 32)
    assert O.budgets(576, 144, 2048) == (144, 288, 72)
    assert O.budgets(2880, 288, 4096) == (288, 576, 128)
    assert O.budgets(16384, 1024, 3584) == (1024, 2048, 128)
    g = GOLD["paper_budget"]
    B, M, r = O.budgets(g["N"], g["B_vis"], 4096)
    assert B == 64 and B < M <= g["N"] and r < min(M, 4096)
    assert O.budgets(5, 9, 16) == (5, 5, 3)              # N <= B_vis: keep everything
    assert O.budgets(2, 1, 16) == (1, 2, 1)
    assert O.budgets(100, 3, 2)[2] == 1                  # r < d


def _tiny_request(N=10, T=3, d=6, A_=2):
    X = RNG.normal(size=(N, d))
    Q = RNG.normal(size=(T, d))
    Hs = [RNG.normal(size=(N, d)) for _ in range(A_ + 1)]
    return X, Q, Hs


def test_request_keepset_brute_force():
    for trial in range(5):
        X, Q, Hs = _tiny_request()
        res = O.prune_request(X, Q, Hs, 3, lam=0.4)
        B, M, r = res["B_vis"], res["M"], res["r"]
        assert (B, M, r) == (3, 6, 2)
        keep, presel = res["keep"], res["presel"]
        assert len(keep) == B and len(set(keep)) == B and list(keep) == sorted(keep)
        assert set(keep) <= set(presel) and len(presel) == M
        # stage 1: the M best fused scores, by exhaustive search
        S = res["s_fused"]
        best1 = max(itertools.combinations(range(len(S)), M), key=lambda c: sum(S[list(c)]))
        assert tuple(presel) == best1
        # stage 2: the B preselected tokens of largest subspace energy, by exhaustive search
        c = res["energy"]
        best2 = max(itertools.combinations(range(M), B), key=lambda cc: sum(c[list(cc)]))
        assert tuple(keep) == tuple(presel[list(best2)])
        np.testing.assert_array_equal(res["compact"], X[keep])


def test_request_degenerate_sizes():
    X, Q, Hs = _tiny_request(N=4)
    res = O.prune_request(X, Q, Hs, 4)
    assert list(res["keep"]) == [0, 1, 2, 3] and res["energy"] is None
    res = O.prune_request(X, Q, Hs, 9)
    assert list(res["keep"]) == [0, 1, 2, 3]
    res = O.prune_request(X[:1], Q, [h[:1] for h in Hs], 1)
    assert list(res["keep"]) == [0]
    res = O.prune_request(X, Q, [], 1)                   # no activity stack
    assert res["s_act"] is None and len(res["keep"]) == 1
    res = O.prune_request(X, Q[:1], Hs, 2, presel_factor=1.0)   # M == B_vis: stage 2 is skipped
    assert list(res["keep"]) == list(res["presel"]) and res["energy"] is None


def test_request_planted_anchors_survive():
    # r orthogonal, long "anchor" tokens plus shorter noisy near-copies of them: the low-rank
    # stage must keep the anchors (largest energy in the retained subspace), not the copies.
    d, r = 32, 4
    basis, _ = np.linalg.qr(RNG.normal(size=(d, d)))
    anchors = 10.0 * basis[:, :r].T * np.array([1.0, 1.1, 1.2, 1.3])[:, None]
    copies = np.vstack([0.5 * anchors[k] + 0.01 * RNG.normal(size=d) for k in range(r)])
    filler = 0.01 * RNG.normal(size=(8, d))
    X = np.vstack([copies, filler[:4], anchors, filler[4:]])
    scores = np.zeros(16)
    scores[[0, 1, 2, 3, 8, 9, 10, 11]] = 1.0             # copies and anchors are preselected
    res = O.prune_request(X, RNG.normal(size=(2, d)), [], 4, forced_scores=scores, rank_frac=1.0)
    assert (res["M"], res["r"]) == (8, 4)
    assert list(res["keep"]) == [8, 9, 10, 11]


def test_forced_preselect_and_ambiguity():
    X, Q, Hs = _tiny_request(N=12)
    res = O.prune_request(X, Q, Hs, 3, forced_presel=[11, 0, 5, 7, 2, 9])
    assert list(res["presel"]) == [0, 2, 5, 7, 9, 11] and set(res["keep"]) <= {0, 2, 5, 7, 9, 11}
    # distinct singular values: nothing is ambiguous
    Z = O.stack(X, res["presel"])
    np.testing.assert_array_equal(O.energy_ambiguity(Z, 2), 0.0)
    # two equal singular values straddling the cut: both directions are reported
    Zt = np.zeros((4, 3))
    Zt[0, 0], Zt[1, 1], Zt[2, 2] = 3.0, 2.0, 2.0
    np.testing.assert_allclose(O.energy_ambiguity(Zt, 2), [0.0, 4.0, 4.0])


# ------------------------------------------------------------------ greedy pivoted variant
def test_greedy_lowrank_hand_and_properties():
    # columns e1*3, e1*2, e2*1, (e1+e2): norms^2 9, 4, 1, 2.  First pick 0 (9).  Residuals after
    # projecting out e1: 0, 0, 1, 1 -> tie between 2 and 3 goes to the lower index 2.
    Z = np.array([[3.0, 2.0, 0.0, 1.0], [0.0, 0.0, 1.0, 1.0]])
    picks, en = O.greedy_lowrank_select(Z, 2)
    assert picks.tolist() == [0, 2] and np.allclose(en, [9.0, 1.0])
    rng = np.random.default_rng(11)
    Z = rng.normal(size=(20, 12))
    picks, en = O.greedy_lowrank_select(Z, 6)
    assert len(set(picks.tolist())) == 6
    assert np.all(np.diff(en) <= 1e-12)                  # residual energies never grow
    # the energies are the squared pivots of a QR with column pivoting: their product is the squared
    # volume of the picked columns
    sub = Z[:, picks]
    assert np.isclose(np.prod(en), np.linalg.det(sub.T @ sub), rtol=1e-9)
    # each pick is the brute-force argmax of the distance to the span of the previous picks
    for k in range(1, 6):
        Q, _ = np.linalg.qr(Z[:, picks[:k]])
        resid = ((Z - Q @ (Q.T @ Z)) ** 2).sum(0)
        resid[picks[:k]] = -1
        assert int(np.argmax(resid)) == picks[k]
    # following its own sequence is valid; following a bad one is not
    assert O.greedy_lowrank_select(Z, 6, follow=picks)[2]
    bad = picks.copy(); bad[0] = int(np.argmin((Z ** 2).sum(0)))
    assert not O.greedy_lowrank_select(Z, 6, follow=bad)[2]


def test_greedy_lowrank_exhausted_rank():
    # rank 2 data, 4 picks: after two picks every residual is ~0 and the remaining picks are the
    # lowest unpicked indices
    rng = np.random.default_rng(12)
    Z = rng.normal(size=(2, 6))
    picks, en = O.greedy_lowrank_select(Z, 4)
    assert len(set(picks.tolist())) == 4 and np.all(np.abs(en[2:]) < 1e-12 * en[0])
