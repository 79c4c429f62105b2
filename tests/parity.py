"""Parity rule between the CUDA path and the CPU oracle (used by the -m gpu tests).

Floating-point scores: |got - want| <= TAU * scale, scale = the request's largest |want| (a cosine
near zero has no meaningful relative error); energies additionally get the oracle's ambiguity for
(nearly) repeated singular values at the cut.  Integer results: every token whose oracle score
clears the cut by more than TAU * scale must be kept, every token that misses it by more must be
dropped; inside the band either answer is valid; size, uniqueness and order always hold.  When
stage 1 differs inside its band, stage 2 is checked against the oracle re-run on the GPU's own
preselected set.
"""
import numpy as np
import torch

from oracle import covspec_oracle as O

TAU = 2e-3


def f64(t):
    return None if t is None else t.detach().cpu().to(torch.float64).numpy()


def check_scores(got, want, what, extra=None, tau=TAU):
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    scale = np.abs(want).max()
    tol = tau * scale + (0.0 if extra is None else extra)
    err = np.abs(got - want)
    bad = err > tol
    assert not bad.any(), (f"{what}: {bad.sum()} of {len(want)} outside tolerance; worst "
                           f"{(err / max(scale, 1e-300)).max():.3e} x scale at {int(np.argmax(err - tol))}")
    return float((err / max(scale, 1e-300)).max())


def check_topk(got_idx, want_scores, k, what, extra=None, tau=TAU):
    """got_idx: selected positions (ascending).  Returns number of positions that differ from the
    oracle's own top-k (all of them inside the band)."""
    want_scores = np.asarray(want_scores, dtype=np.float64)
    got_idx = np.asarray(got_idx)
    n = len(want_scores)
    assert len(got_idx) == k, f"{what}: size {len(got_idx)} != {k}"
    assert len(np.unique(got_idx)) == k and np.all(np.diff(got_idx) > 0), f"{what}: not unique/ascending"
    assert got_idx.min() >= 0 and got_idx.max() < n, f"{what}: index out of range"
    want_idx = O.top_k(want_scores, k)
    if k == n:
        return 0
    order = np.sort(want_scores)[::-1]
    theta = 0.5 * (order[k - 1] + order[k])
    band = tau * np.abs(want_scores).max() + (0.0 if extra is None else np.asarray(extra))
    sel = np.zeros(n, dtype=bool)
    sel[got_idx] = True
    must_keep = want_scores > theta + band
    must_drop = want_scores < theta - band
    assert not (must_keep & ~sel).any(), \
        f"{what}: {int((must_keep & ~sel).sum())} tokens clearly above the cut were dropped"
    assert not (must_drop & sel).any(), \
        f"{what}: {int((must_drop & sel).sum())} tokens clearly below the cut were kept"
    return int(len(set(got_idx.tolist()) ^ set(want_idx.tolist())) // 2)


def oracle_kwargs(wl, **kw):
    args = dict(Wq=f64(wl.Wq), Wk=f64(wl.Wk), n_heads=wl.n_heads, head_dim=wl.head_dim, lam=wl.lam)
    args.update(kw)
    return args


def check_request(wl, b, gpu, stats, **oracle_kw):
    """gpu: dict with s_query, s_act, s_fused (numpy, request slice), presel, energy, keep, out."""
    v0, v1 = int(wl.vis_offsets[b]), int(wl.vis_offsets[b + 1])
    t0, t1 = int(wl.txt_offsets[b]), int(wl.txt_offsets[b + 1])
    X, Q = f64(wl.X[v0:v1]), f64(wl.Q[t0:t1])
    Hs = [f64(h[v0:v1]) for h in wl.Hs]
    kw = oracle_kwargs(wl, **oracle_kw)
    ref = O.prune_request(X, Q, Hs, int(wl.keep[b]), **kw)
    tag = f"{wl.name}[{b}]"
    stats["err_query"] = max(stats.get("err_query", 0), check_scores(gpu["s_query"], ref["s_query"], tag + " s_query"))
    if ref["s_act"] is not None:
        rel = np.abs(gpu["s_act"] - ref["s_act"]) / np.maximum(np.abs(ref["s_act"]), 1e-300)
        assert rel.max() <= TAU, f"{tag} s_act: max relative error {rel.max():.3e}"
        stats["err_act"] = max(stats.get("err_act", 0), float(rel.max()))
    stats["err_fused"] = max(stats.get("err_fused", 0), check_scores(gpu["s_fused"], ref["s_fused"], tag + " s_fused"))
    M, B = ref["M"], ref["B_vis"]
    assert len(gpu["presel"]) == M and len(gpu["keep"]) == B
    d1 = check_topk(gpu["presel"], ref["s_fused"], M, tag + " preselect")
    stats["presel_diff"] = stats.get("presel_diff", 0) + d1
    if d1:
        ref = O.prune_request(X, Q, Hs, int(wl.keep[b]), forced_presel=gpu["presel"], **kw)
    if ref["energy"] is not None:
        Z = O.stack(X, ref["presel"])
        amb = O.energy_ambiguity(Z, ref["r"])
        stats["err_energy"] = max(stats.get("err_energy", 0),
                                  check_scores(gpu["energy"], ref["energy"], tag + " energy", extra=amb))
        pos = np.searchsorted(ref["presel"], gpu["keep"])
        assert np.array_equal(ref["presel"][pos], gpu["keep"]), f"{tag}: keep is not a subset of presel"
        d2 = check_topk(pos, ref["energy"], B, tag + " final select", extra=amb)
        stats["keep_diff"] = stats.get("keep_diff", 0) + d2
    else:
        assert np.array_equal(gpu["keep"], gpu["presel"]), f"{tag}: stage 2 skipped but keep != presel"
    exact = np.array_equal(gpu["keep"], ref["keep"])
    stats["keep_exact"] = stats.get("keep_exact", 0) + int(exact)
    stats["requests"] = stats.get("requests", 0) + 1
    want_rows = wl.X[v0:v1].cpu()[torch.from_numpy(np.asarray(gpu["keep"], dtype=np.int64))]
    assert torch.equal(gpu["out"], want_rows), f"{tag}: compacted rows are not bit copies of X[keep]"
    return ref


def run_gpu(wl, pruner_kw=None, requests=None, stats=None, **oracle_kw):
    """Runs score / select / compact and the fused prune through the C ABI on cuda:0 and checks the
    chosen requests against the oracle.  Returns the stats dict."""
    from paper_2605_02218_b200 import api
    stats = {} if stats is None else stats
    dev = wl.to("cuda:0")
    pr = api.Pruner.for_workload(dev, **(pruner_kw or {}))
    m = pr.marshal(dev)
    sq, sa, sf = pr.score(m)
    keep_idx, ko, presel, po, energy = pr.select(m, sf)
    out, pos = pr.compact(m, keep_idx, ko)
    out2, keep2, ko2 = pr.prune(m)
    stats["launches"] = pr.last_launch_count
    pr.check_device_status()
    assert np.array_equal(ko, ko2)
    assert torch.equal(keep_idx, keep2), "fused prune and the separate calls disagree on keep_idx"
    assert torch.equal(out, out2), "fused prune and the separate calls disagree on the compacted rows"
    assert torch.equal(pos, keep_idx)
    sq, sf = sq.cpu().numpy(), sf.cpu().numpy()
    sa = None if sa is None else sa.cpu().numpy()
    keep_idx, presel, energy, out = keep_idx.cpu().numpy(), presel.cpu().numpy(), energy.cpu().numpy(), out.cpu()
    for b in (range(wl.batch) if requests is None else requests):
        v0, v1 = int(wl.vis_offsets[b]), int(wl.vis_offsets[b + 1])
        gpu = dict(s_query=sq[v0:v1], s_act=None if sa is None else sa[v0:v1], s_fused=sf[v0:v1],
                   presel=presel[po[b]:po[b + 1]], energy=energy[po[b]:po[b + 1]],
                   keep=keep_idx[ko[b]:ko[b + 1]], out=out[ko[b]:ko[b + 1]])
        check_request(wl, b, gpu, stats, **oracle_kw)
    pr.close()
    return stats
