"""Seeded synthetic workloads shaped like the visual-token-reduction inputs of CoVSpec (Sec. III-A).

This module only draws random tensors.  It contains none of the method's arithmetic (no score,
no selection, no SVD): both the CUDA path and the CPU oracle consume what it returns.

Inputs of one batch (notation of Sec. III-A):
  X    [sum N_b, d]   visual token representations v_i / z_i, request-major packed rows
  Q    [sum T_b, d]   query-element embeddings q_j (the keyword subset is taken as given)
  Wq,Wk [P, d]        per-head embedding maps e(.), P = n_heads*head_dim, one output feature per
                      row (the layout of a linear layer's weight); None = identity embedding
  Hs   A+1 tensors shaped like X: hidden states h^(L-A) .. h^(L) of the late layers (Eq. 11)
  vis_offsets, txt_offsets  int32 [batch+1] row offsets of every request
  keep  int32 [batch]       B_vis per request

The recipe (ranks, noise levels, log-normal norms, planted text/visual correlation) is stated in
the functions below; the five named configurations are in CONFIGS.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch


@dataclass
class Workload:
    name: str
    dtype: torch.dtype
    d: int
    n_heads: int
    head_dim: int
    act_layers: int
    lam: float
    vis_offsets: np.ndarray
    txt_offsets: np.ndarray
    keep: np.ndarray
    X: torch.Tensor
    Q: torch.Tensor
    Wq: Optional[torch.Tensor]
    Wk: Optional[torch.Tensor]
    Hs: List[torch.Tensor] = field(default_factory=list)

    @property
    def batch(self) -> int:
        return len(self.keep)

    @property
    def total_vis(self) -> int:
        return int(self.vis_offsets[-1])

    @property
    def total_txt(self) -> int:
        return int(self.txt_offsets[-1])

    def request(self, b: int) -> "Workload":
        """A one-request view (same tensors, sliced)."""
        v0, v1 = int(self.vis_offsets[b]), int(self.vis_offsets[b + 1])
        t0, t1 = int(self.txt_offsets[b]), int(self.txt_offsets[b + 1])
        return Workload(
            name=f"{self.name}[{b}]", dtype=self.dtype, d=self.d, n_heads=self.n_heads,
            head_dim=self.head_dim, act_layers=self.act_layers, lam=self.lam,
            vis_offsets=np.array([0, v1 - v0], dtype=np.int32),
            txt_offsets=np.array([0, t1 - t0], dtype=np.int32),
            keep=self.keep[b:b + 1].copy(),
            X=self.X[v0:v1], Q=self.Q[t0:t1], Wq=self.Wq, Wk=self.Wk,
            Hs=[h[v0:v1] for h in self.Hs])

    def to(self, device) -> "Workload":
        mv = lambda t: None if t is None else t.to(device)
        return Workload(self.name, self.dtype, self.d, self.n_heads, self.head_dim,
                        self.act_layers, self.lam, self.vis_offsets, self.txt_offsets, self.keep,
                        mv(self.X), mv(self.Q), mv(self.Wq), mv(self.Wk), [mv(h) for h in self.Hs])


def keep_from_ratio(n: int, ratio: float) -> int:
    """Integer budget of a keep ratio: max(1, ceil(ratio*n - 1e-6)), evaluated in double."""
    return max(1, int(math.ceil(ratio * n - 1e-6)))


def _randn(gen, *shape, device):
    return torch.randn(*shape, generator=gen, device=device, dtype=torch.float32)


def _mixture_tokens(gen, n, d, rank, cluster_of_token, n_clusters, device):
    """Rank-`rank` Gaussian mixture: x_i = (mu_c(i) + 0.5 g_i) @ basis, basis ~ N(0, 1/rank)."""
    basis = _randn(gen, rank, d, device=device) / math.sqrt(rank)
    mu = _randn(gen, n_clusters, rank, device=device)
    w = mu[cluster_of_token] + 0.5 * _randn(gen, n, rank, device=device)
    return w @ basis


def _finish_tokens(gen, sig, noise, lognorm_sigma, device):
    """Add iid noise of `noise` x the signal's per-coordinate std, then rescale every token's norm
    by a log-normal factor exp(lognorm_sigma * g)."""
    n, d = sig.shape
    sigma_sig = sig.std().item()
    x = sig + noise * sigma_sig * _randn(gen, n, d, device=device)
    scale = torch.exp(lognorm_sigma * _randn(gen, n, 1, device=device))
    return x * scale


def _visual_request(gen, kind, n, d, rank, n_clusters, device):
    if kind == "mixture":
        cl = torch.randint(0, n_clusters, (n,), generator=gen, device=device)
        return _finish_tokens(gen, _mixture_tokens(gen, n, d, rank, cl, n_clusters, device),
                              0.1, 0.5, device)
    if kind == "tiles":
        # anyres-style: `n_clusters` equal tiles, every tile draws from its own cluster of one
        # shared rank-`rank` basis.
        per = -(-n // n_clusters)
        cl = (torch.arange(n, device=device) // per).clamp_(max=n_clusters - 1)
        return _finish_tokens(gen, _mixture_tokens(gen, n, d, rank, cl, n_clusters, device),
                              0.1, 0.5, device)
    if kind == "video":
        # frames of 512 tokens; frame f = frame f-1 + 0.05 sigma perturbation.
        per = min(512, n)
        cl = torch.randint(0, n_clusters, (per,), generator=gen, device=device)
        f0 = _finish_tokens(gen, _mixture_tokens(gen, per, d, rank, cl, n_clusters, device),
                            0.1, 0.5, device)
        sigma = f0.std().item()
        frames = [f0]
        while len(frames) * per < n:
            frames.append(frames[-1] + 0.05 * sigma * _randn(gen, per, d, device=device))
        return torch.cat(frames, 0)[:n]
    raise ValueError(kind)


def _text_request(gen, x, t, device):
    """N(0, I) query elements; the first t//2 are correlated with 8 randomly chosen visual tokens:
    q_j = 0.7 x_a / rms(x_a) + 0.3 N(0, I)."""
    n, d = x.shape
    q = _randn(gen, t, d, device=device)
    n_anchor = min(8, n)
    perm = torch.randperm(n, generator=gen, device=device)[:n_anchor]
    for j in range(t // 2):
        xa = x[perm[j % n_anchor]]
        rms = xa.pow(2).mean().sqrt().clamp_min(1e-20)
        q[j] = 0.7 * xa / rms + 0.3 * q[j]
    return q


def _xavier_heads(gen, n_heads, head_dim, d, device):
    bound = math.sqrt(6.0 / (d + head_dim))
    w = torch.rand(n_heads * head_dim, d, generator=gen, device=device, dtype=torch.float32)
    return (2.0 * w - 1.0) * bound


def make_workload(name="custom", *, seed=0, dtype=torch.bfloat16, batch=1, n_vis=576,
                  n_txt=32, d=1024, n_heads=1, head_dim=128, rank=32, n_clusters=8,
                  kind="mixture", keep=None, keep_ratio=None, act_layers=4, lam=0.5,
                  device="cpu", sizes=None) -> Workload:
    """Build one batch.  `n_vis` / `n_txt` are an int (uniform) or an inclusive (lo, hi) range
    drawn per request.  `n_heads=0` gives the identity embedding (Wq = Wk = None).  `sizes`
    = (list of N_b, list of T_b) fixes the request sizes instead (another batch of the same shape
    with different contents); the size draws are still consumed so that the rest of the stream
    does not depend on it."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)

    def draw(spec):
        if isinstance(spec, (tuple, list)):
            lo, hi = spec
            return [int(v) for v in
                    torch.randint(lo, hi + 1, (batch,), generator=gen, device=device).tolist()]
        return [int(spec)] * batch

    ns, ts = draw(n_vis), draw(n_txt)
    if sizes is not None:
        ns, ts = [int(v) for v in sizes[0]], [int(v) for v in sizes[1]]
        assert len(ns) == batch and len(ts) == batch
    xs, qs = [], []
    hs = [[] for _ in range(act_layers + 1)] if act_layers > 0 else []
    for b in range(batch):
        x = _visual_request(gen, kind, ns[b], d, rank, n_clusters, device).to(dtype)
        xs.append(x)
        qs.append(_text_request(gen, x.float(), ts[b], device).to(dtype))
        if act_layers > 0:
            rms = x.float().pow(2).mean().sqrt().item()
            a = torch.exp(0.5 * _randn(gen, ns[b], 1, device=device))
            h = x.clone()
            hs[0].append(h)
            for l in range(1, act_layers + 1):
                h = (h.float() + 0.1 * rms * a * _randn(gen, ns[b], d, device=device)).to(dtype)
                hs[l].append(h)
    if n_heads > 0:
        wq = _xavier_heads(gen, n_heads, head_dim, d, device).to(dtype)
        wk = _xavier_heads(gen, n_heads, head_dim, d, device).to(dtype)
    else:
        wq = wk = None
    if keep is not None:
        kp = [int(keep)] * batch if np.isscalar(keep) else [int(k) for k in keep]
    else:
        kp = [keep_from_ratio(n, keep_ratio) for n in ns]
    return Workload(
        name=name, dtype=dtype, d=d, n_heads=n_heads, head_dim=head_dim, act_layers=act_layers,
        lam=lam,
        vis_offsets=np.concatenate([[0], np.cumsum(ns)]).astype(np.int32),
        txt_offsets=np.concatenate([[0], np.cumsum(ts)]).astype(np.int32),
        keep=np.asarray(kp, dtype=np.int32),
        X=torch.cat(xs, 0), Q=torch.cat(qs, 0), Wq=wq, Wk=wk,
        Hs=[torch.cat(h, 0) for h in hs])


# The five named configurations (shapes, dtypes, budgets).  `batch` can be overridden to take a
# bounded sample of the same workload.
CONFIGS = {
    "c1": dict(seed=0, dtype=torch.float32, batch=1, n_vis=576, n_txt=32, d=1024, n_heads=1,
               rank=32, n_clusters=8, kind="mixture", keep=64),
    "c2": dict(seed=1, dtype=torch.bfloat16, batch=16, n_vis=576, n_txt=64, d=2048, n_heads=16,
               rank=64, n_clusters=8, kind="mixture", keep_ratio=0.25),
    "c3": dict(seed=2, dtype=torch.bfloat16, batch=32, n_vis=2880, n_txt=128, d=4096, n_heads=32,
               rank=128, n_clusters=5, kind="tiles", keep_ratio=0.10),
    "c4": dict(seed=3, dtype=torch.bfloat16, batch=64, n_vis=(256, 4096), n_txt=(16, 256), d=1536,
               n_heads=12, rank=64, n_clusters=8, kind="mixture", keep_ratio=0.20),
    "c5": dict(seed=4, dtype=torch.bfloat16, batch=8, n_vis=16384, n_txt=64, d=3584, n_heads=28,
               rank=64, n_clusters=8, kind="video", keep=1024),
}


def make_config(name: str, device="cpu", **overrides) -> Workload:
    kw = dict(CONFIGS[name])
    kw.update(overrides)
    return make_workload(name, device=device, **kw)


def make_logits(*, seed=0, rows=64, vocab=151674, dtype=torch.float16, spread=3.0, disagreement=1.0,
                device="cpu"):
    """Seeded draft / target logit rows for the device-side correction step: draft logits
    spread * N(0, 1), target logits = draft + disagreement * N(0, 1) (the two models mostly agree),
    uniform numbers in [0, 1) for the correction draw and uniformly drawn drafted token ids.  Rows are
    padded to a multiple of 8 elements (16-byte rows); the padding holds zeros and is not part of the
    vocabulary.  Returns a dict of tensors and sizes; draws only, none of the method's arithmetic."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    ld = (vocab + 7) // 8 * 8
    zd = torch.zeros(rows, ld, dtype=torch.float32, device=device)
    zt = torch.zeros(rows, ld, dtype=torch.float32, device=device)
    base = spread * torch.randn(rows, vocab, generator=gen, device=device)
    zd[:, :vocab] = base
    zt[:, :vocab] = base + disagreement * torch.randn(rows, vocab, generator=gen, device=device)
    uniforms = torch.rand(rows, generator=gen, device=device, dtype=torch.float32)
    drafted = torch.randint(0, vocab, (rows,), generator=gen, device=device, dtype=torch.int32)
    return dict(z_draft=zd.to(dtype), z_target=zt.to(dtype), uniforms=uniforms, drafted=drafted,
                rows=rows, vocab=vocab, ld=ld)
