"""CPU oracle for CoVSpec's training-free visual token selection (Sec. III-A, Eq. 10-15).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the selection path
computes, in float64 numpy, one paper definition per function, with no blocking, fusion or
reordering.  It shares no code with the CUDA library and is imported only by the tests, by the
smoke check and by the benchmark's CPU-baseline leg.  The product path never calls it.

Pinned by tests/test_oracle_pins.py against closed forms, invariances, brute force on tiny inputs
and independently written power iteration.  Parity unpinned by the paper (it gives no values):
lambda, the number of late layers, the preselect size M, the rank r, the normalisation used in
"normalize the two scores to the same scale", and how heads combine; the defaults below are this
library's reading and are passed in explicitly.

Inputs are numpy arrays already rounded to the storage dtype and upcast to float64; nothing is
rounded in between.
"""
from __future__ import annotations

import math

import numpy as np


# ----------------------------------------------------------------------------------------------
# Eq. 10: query-aware score
# ----------------------------------------------------------------------------------------------
def embed(F, W, n_heads, head_dim):
    """e(.) of Sec. III-A.1.  W is [n_heads*head_dim, d] (one output feature per row) or None for
    the identity map.  Returns [n_heads_eff, rows, width]."""
    F = np.asarray(F, dtype=np.float64)
    if W is None or n_heads == 0:
        return F[None, :, :]
    W = np.asarray(W, dtype=np.float64)
    E = F @ W.T                                            # [rows, P]
    return E.reshape(F.shape[0], n_heads, head_dim).transpose(1, 0, 2)


def cosine_table(EV, EQ):
    """cos[h, i, j] = <e(v_i), e(q_j)> / (||e(v_i)|| ||e(q_j)||) per head; 0 where a norm is 0."""
    inner = EV @ EQ.transpose(0, 2, 1)                    # [h, i, j]
    nv = np.sqrt(np.sum(EV * EV, axis=2))                  # [h, i]
    nq = np.sqrt(np.sum(EQ * EQ, axis=2))                  # [h, j]
    den = nv[:, :, None] * nq[:, None, :]
    cos = np.zeros_like(inner)
    np.divide(inner, den, out=cos, where=den > 0.0)
    return cos


def query_relevance(X, Q, Wq=None, Wk=None, n_heads=0, head_dim=0, head_reduce="max"):
    """Eq. 10: S_i^query = max over query elements of the cosine similarity.  With several heads
    every (query element, head) pair counts as one element of the max ("max"), or the per-head
    cosines are averaged before the max over query elements ("mean")."""
    cos = cosine_table(embed(X, Wk, n_heads, head_dim), embed(Q, Wq, n_heads, head_dim))
    if head_reduce == "max":
        return cos.max(axis=(0, 2))
    if head_reduce == "mean":
        return cos.mean(axis=0).max(axis=1)
    raise ValueError(head_reduce)


# ----------------------------------------------------------------------------------------------
# Eq. 11: token activity score
# ----------------------------------------------------------------------------------------------
def token_activity(Hs):
    """Eq. 11 with K = len(Hs) - 1 late layers: the mean over consecutive layers of the Euclidean
    norm of the change of token i's hidden state.  Hs[l] is [N, d]; Hs[0] is layer L-K."""
    K = len(Hs) - 1
    acc = np.zeros(np.asarray(Hs[0]).shape[0], dtype=np.float64)
    for l in range(1, K + 1):
        diff = np.asarray(Hs[l], dtype=np.float64) - np.asarray(Hs[l - 1], dtype=np.float64)
        acc += np.sqrt(np.sum(diff * diff, axis=1))
    return acc / K


# ----------------------------------------------------------------------------------------------
# Eq. 12: normalise to a common scale and fuse
# ----------------------------------------------------------------------------------------------
def normalise(S, mode="minmax"):
    S = np.asarray(S, dtype=np.float64)
    if mode == "minmax":
        lo, hi = S.min(), S.max()
        return np.zeros_like(S) if hi == lo else (S - lo) / (hi - lo)
    if mode == "zscore":
        sd = S.std()
        return np.zeros_like(S) if sd == 0.0 else (S - S.mean()) / sd
    if mode == "none":
        return S.copy()
    raise ValueError(mode)


def fuse(S_query, S_act, lam, mode="minmax"):
    """Eq. 12: S_i = lam * norm(S^query)_i + (1 - lam) * norm(S^act)_i.  S_act None means the
    activity term is absent (no late-layer stack): S = norm(S^query)."""
    if S_act is None:
        return normalise(S_query, mode)
    return lam * normalise(S_query, mode) + (1.0 - lam) * normalise(S_act, mode)


# ----------------------------------------------------------------------------------------------
# "retain the M highest-scoring tokens" / "retain the B_vis tokens with the largest energies"
# ----------------------------------------------------------------------------------------------
def top_k(scores, k):
    """Indices of the k largest scores; equal scores are taken in order of increasing index.
    Returned in ascending index order."""
    scores = np.asarray(scores, dtype=np.float64)
    order = sorted(range(len(scores)), key=lambda i: (-scores[i], i))
    return np.array(sorted(order[:k]), dtype=np.int64)


# ----------------------------------------------------------------------------------------------
# Eq. 13-15: low-rank redundancy reduction
# ----------------------------------------------------------------------------------------------
def stack(X, presel):
    """Eq. 13: Z_M = [z_1 ... z_M] in R^{d x M}, z_i the representation of preselected token i."""
    return np.asarray(X, dtype=np.float64)[np.asarray(presel)].T


def subspace_energy(Z_M, r):
    """Eq. 14-15: truncated SVD Z_M ~ U_r S_r V_r^T and c_i = ||(V_r S_r)_{i,:}||_2^2.
    Returns (c [M], singular values [min(d, M)])."""
    _, s, Vt = np.linalg.svd(Z_M, full_matrices=False)     # Z_M = U diag(s) Vt, s descending
    Vr = Vt[:r].T                                          # [M, r]
    VS = Vr * s[:r][None, :]                               # V_r Sigma_r
    return np.sum(VS * VS, axis=1), s


# ----------------------------------------------------------------------------------------------
# Budgets (host integer logic; the paper only requires r < min(M, d) and B_vis < M <= N)
# ----------------------------------------------------------------------------------------------
def budgets(N, B_vis, d, presel_factor=2.0, rank_frac=0.5, rank_cap=128):
    """Returns (B_vis, M, r).  M = min(N, ceil(presel_factor * B_vis)) but at least B_vis;
    r = clamp(ceil(rank_frac * B_vis), 1, min(rank_cap, M - 1, d - 1))."""
    B = min(int(B_vis), N)
    M = min(N, max(B, int(math.ceil(presel_factor * B - 1e-9))))
    r = max(1, min(int(math.ceil(rank_frac * B - 1e-9)), rank_cap, M - 1, d - 1))
    return B, M, r


# ----------------------------------------------------------------------------------------------
# One request, all steps in the paper's order
# ----------------------------------------------------------------------------------------------
def prune_request(X, Q, Hs, B_vis, *, Wq=None, Wk=None, n_heads=0, head_dim=0, lam=0.5,
                  norm_mode="minmax", head_reduce="max", presel_factor=2.0, rank_frac=0.5,
                  rank_cap=128, forced_presel=None, forced_scores=None):
    """Sec. III-A end to end for one request.  X [N, d] (any float dtype, upcast here), Q [T, d],
    Hs list of A+1 arrays [N, d] or empty.  `forced_presel` replaces the stage-1 result (to check
    stage 2 when stage 1 legitimately differs inside the tolerance band); `forced_scores` replaces
    the fused score S.  Returns a dict of every intermediate."""
    Xd = np.asarray(X, dtype=np.float64)
    N, d = Xd.shape
    B, M, r = budgets(N, B_vis, d, presel_factor, rank_frac, rank_cap)
    out = dict(N=N, B_vis=B, M=M, r=r)
    if forced_scores is None:
        out["s_query"] = query_relevance(Xd, Q, Wq, Wk, n_heads, head_dim, head_reduce)
        out["s_act"] = token_activity(Hs) if len(Hs) > 1 else None
        out["s_fused"] = fuse(out["s_query"], out["s_act"], lam, norm_mode)
    else:
        out["s_fused"] = np.asarray(forced_scores, dtype=np.float64)
    presel = top_k(out["s_fused"], M) if forced_presel is None else \
        np.array(sorted(int(i) for i in forced_presel), dtype=np.int64)
    out["presel"] = presel
    if B >= M:
        # Nothing to reduce (B_vis < M does not hold): the preselected set is the keep-set.
        out["energy"] = None
        out["svals"] = None
        keep = presel
    else:
        c, s = subspace_energy(stack(Xd, presel), r)
        out["energy"] = c
        out["svals"] = s
        keep = presel[top_k(c, B)]
    out["keep"] = keep
    out["compact"] = np.asarray(X)[keep]
    return out


def prune_batch(wl, requests=None, **kw):
    """Run prune_request on the requests of a workload object (fields X, Q, Wq, Wk, Hs as torch
    tensors, vis_offsets, txt_offsets, keep).  Returns a list of per-request dicts."""
    import torch

    def f64(t):
        return None if t is None else t.detach().cpu().to(dtype=torch.float64).numpy()
    Wq, Wk = f64(wl.Wq), f64(wl.Wk)
    res = []
    for b in (range(len(wl.keep)) if requests is None else requests):
        v0, v1 = int(wl.vis_offsets[b]), int(wl.vis_offsets[b + 1])
        t0, t1 = int(wl.txt_offsets[b]), int(wl.txt_offsets[b + 1])
        args = dict(Wq=Wq, Wk=Wk, n_heads=wl.n_heads, head_dim=wl.head_dim, lam=wl.lam)
        args.update(kw)
        res.append(prune_request(f64(wl.X[v0:v1]), f64(wl.Q[t0:t1]),
                                 [f64(h[v0:v1]) for h in wl.Hs], int(wl.keep[b]), **args))
    return res


# ----------------------------------------------------------------------------------------------
# Diagnostics used by the parity rule
# ----------------------------------------------------------------------------------------------
def energy_ambiguity(Z_M, r, delta=1e-3):
    """Energy of token i in singular directions whose squared singular value lies within
    delta * sigma_1^2 of sigma_r^2 or sigma_{r+1}^2: c_i is defined only up to a rotation inside
    (nearly) repeated singular values that straddle the cut."""
    _, s, Vt = np.linalg.svd(Z_M, full_matrices=False)
    lam = s * s
    if r >= len(lam):
        return np.zeros(Z_M.shape[1])
    if lam[r - 1] - lam[r] > delta * lam[0]:
        return np.zeros(Z_M.shape[1])
    near = (np.abs(lam - lam[r - 1]) <= delta * lam[0]) | (np.abs(lam - lam[r]) <= delta * lam[0])
    return np.sum((Vt[near].T ** 2) * lam[near][None, :], axis=1)


# ----------------------------------------------------------------------------------------------
# Variant (not in the paper): greedy pivoted low-rank selection
# ----------------------------------------------------------------------------------------------
def greedy_lowrank_select(Z_M, B, follow=None, tol=0.0):
    """Alternative to Eq. 14-15 that the library offers as `lowrank_mode = 1`: pick, B times, the
    preselected token whose representation has the largest residual energy after projecting out
    the span of the tokens already picked, then update the residuals (pivoted Cholesky of
    G = Z_M^T Z_M: argmax of the residual diagonal, rank-1 update).  Ties go to the lower index; a
    picked token is never picked again.

    Returns (picks in order, residual energy of every pick at the time it was picked).  With
    `follow` (a pick sequence from another implementation) the same loop takes that sequence
    instead of its own argmax and returns, as a third value, whether every followed pick was within
    tol * max(diag G) of the largest residual at its step (several orders are valid at near-ties)."""
    Z = np.asarray(Z_M, dtype=np.float64)
    G = Z.T @ Z
    M = G.shape[0]
    e = np.diag(G).copy()
    scale = e.max() if M else 0.0
    C = np.zeros((0, M))
    picked = np.zeros(M, dtype=bool)
    picks, energies, valid = [], [], True
    for k in range(B):
        cand = np.where(picked, -np.inf, e)
        best = int(np.argmax(cand))                      # first index of the maximum
        if follow is not None:
            p = int(follow[k])
            if picked[p] or cand[p] < cand[best] - tol * scale:
                valid = False
        else:
            p = best
        picks.append(p)
        energies.append(float(e[p]))
        picked[p] = True
        if e[p] > 0.0:
            c = (G[:, p] - C.T @ C[:, p]) / np.sqrt(e[p])
            C = np.vstack([C, c[None, :]])
            e = e - c * c
    if follow is not None:
        return np.array(picks), np.array(energies), valid
    return np.array(picks), np.array(energies)
