"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element on seeded
inputs: small shapes that span several tiles with ragged tails, the degenerate cases, and the
named configurations."""
import numpy as np
import pytest
import torch

from paper_2605_02218_b200 import workloads
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2605_02218_b200 import build
    build.build()


def _report(name, stats):
    print(f"\n[parity] {name}: " + ", ".join(f"{k}={v:.3g}" if isinstance(v, float) else f"{k}={v}"
                                             for k, v in sorted(stats.items())))


SMALL = [
    # identity embedding, fp32 and bf16, odd sizes
    dict(seed=11, dtype=torch.float32, batch=3, n_vis=(50, 300), n_txt=(1, 9), d=72, n_heads=0,
         rank=8, keep_ratio=0.3),
    dict(seed=12, dtype=torch.bfloat16, batch=4, n_vis=(100, 700), n_txt=(3, 40), d=264, n_heads=0,
         rank=16, keep_ratio=0.2),
    # projection heads, ragged, tails that are not multiples of any tile
    dict(seed=13, dtype=torch.bfloat16, batch=5, n_vis=(65, 900), n_txt=(1, 70), d=136, n_heads=3,
         rank=12, keep_ratio=0.25),
    dict(seed=14, dtype=torch.float32, batch=2, n_vis=(129, 257), n_txt=(2, 33), d=200, n_heads=2,
         rank=10, keep=40),
    # many late layers / no activity term
    dict(seed=15, dtype=torch.bfloat16, batch=2, n_vis=333, n_txt=7, d=128, n_heads=1, rank=8,
         keep_ratio=0.1, act_layers=9),
    dict(seed=16, dtype=torch.bfloat16, batch=2, n_vis=333, n_txt=7, d=128, n_heads=1, rank=8,
         keep_ratio=0.1, act_layers=0),
    # video-like near-duplicate frames: low-rank dependency dominates
    dict(seed=17, dtype=torch.bfloat16, batch=2, n_vis=1536, n_txt=16, d=256, n_heads=2, rank=16,
         kind="video", keep=128),
    # more query elements than the four logits tiles one pass of the relevance kernel holds
    dict(seed=18, dtype=torch.bfloat16, batch=2, n_vis=(130, 400), n_txt=(257, 330), d=128, n_heads=3,
         rank=8, keep_ratio=0.2),
]


@pytest.mark.parametrize("kw", SMALL, ids=lambda kw: f"seed{kw['seed']}")
def test_small_shapes(kw):
    wl = workloads.make_workload(f"small{kw['seed']}", **kw)
    _report(wl.name, parity.run_gpu(wl))


@pytest.mark.parametrize("d,heads", [(200, 3), (64, 1), (328, 2)])
def test_float32_on_the_tensor_cores_with_padded_width(d, heads):
    # float32 inputs reach the tensor-core kernels as three bf16 terms laid side by side; every term
    # is padded to a multiple of 64 columns (d = 200 -> 256, 328 -> 384), several requests, ragged sizes
    wl = workloads.make_workload(f"f32-d{d}", seed=60 + heads, dtype=torch.float32, batch=3,
                                 n_vis=(140, 700), n_txt=(3, 70), d=d, n_heads=heads, rank=12,
                                 keep_ratio=0.25)
    stats = parity.run_gpu(wl)
    _report(wl.name, stats)
    assert stats["launches"] == 11


def test_zero_token_on_the_tensor_core_path():
    # an all-zero visual token has cosine 0 with every query element (zero-norm reading), also when
    # the query elements lean negative
    wl = workloads.make_workload("zero-token", seed=19, dtype=torch.bfloat16, batch=2, n_vis=(130, 260),
                                 n_txt=(3, 9), d=128, n_heads=2, rank=8, keep_ratio=0.2)
    wl.Q = -wl.Q.abs()
    wl.X[5] = 0
    wl.X[77] = 0
    wl.Hs = [wl.X.clone()] + wl.Hs[1:]
    _report(wl.name, parity.run_gpu(wl))


@pytest.mark.parametrize("kw", [SMALL[2], SMALL[7]], ids=lambda kw: f"seed{kw['seed']}")
def test_two_sm_relevance_kernel(kw):
    # relevance_path = 2: the cta_group::2 form of the relevance kernel (pairs of token tiles on pairs
    # of SMs) gives the same scores; ragged sizes, an odd number of tiles, more than 256 query elements
    wl = workloads.make_workload(f"pair{kw['seed']}", **kw)
    _report(wl.name, parity.run_gpu(wl, pruner_kw=dict(relevance_path=2)))


@pytest.mark.parametrize("d", [136, 1104])
def test_relevance_kernel_several_items_per_block(d):
    # more (token tile, head pair) items than SMs, so that every block of the relevance kernel walks
    # through several of them (its ring and accumulator phases wrap); three and eighteen k-chunks; an
    # odd number of heads leaves a single head in the last pair
    wl = workloads.make_workload(f"items-d{d}", seed=23, dtype=torch.bfloat16, batch=3, n_vis=(3000, 9000),
                                 n_txt=(5, 64), d=d, n_heads=5, rank=8, keep_ratio=0.02)
    _report(wl.name, parity.run_gpu(wl))


def test_more_requests_than_sms_and_more_tiles_than_sms():
    # 170 stage-2 requests of two to six row tiles: every request is one group of the subspace kernel's
    # schedule and the CTAs carry more than one request; then 24 requests with up to twelve tiles, whose
    # tiles are split into groups so that the slowest request's step is as short as the CTAs allow
    many = workloads.make_workload("many-requests", seed=104, dtype=torch.bfloat16, batch=170, n_vis=(260, 700),
                                   n_txt=(2, 20), d=128, n_heads=1, rank=8, keep_ratio=0.3)
    _report(many.name, parity.run_gpu(many))
    ragged = workloads.make_workload("many-tiles", seed=101, dtype=torch.bfloat16, batch=24, n_vis=(500, 3000),
                                     n_txt=(4, 60), d=256, n_heads=2, rank=24, keep_ratio=0.25)
    _report(ragged.name, parity.run_gpu(ragged))


def test_degenerate_requests():
    # N = 1; B_vis >= N (keep everything); B_vis = N - 1; B_vis = 1; T = 1
    wl = workloads.make_workload("degenerate", seed=21, dtype=torch.bfloat16, batch=6,
                                 n_vis=(2, 40), n_txt=1, d=64, n_heads=0, rank=4, keep=1)
    n = np.diff(wl.vis_offsets)
    wl.keep[:] = [1, n[1], n[2] - 1, 1, n[4] + 5, max(1, n[5] // 2)]
    _report(wl.name, parity.run_gpu(wl))
    one = workloads.make_workload("single-token", seed=22, dtype=torch.float32, batch=2, n_vis=1,
                                  n_txt=3, d=32, n_heads=0, rank=2, keep=1)
    _report(one.name, parity.run_gpu(one))


@pytest.mark.parametrize("mode", ["zscore", "none"])
def test_norm_modes(mode):
    wl = workloads.make_workload("norm-" + mode, seed=23, dtype=torch.bfloat16, batch=2, n_vis=400,
                                 n_txt=12, d=128, n_heads=2, rank=8, keep_ratio=0.2)
    _report(wl.name, parity.run_gpu(wl, pruner_kw=dict(norm_mode=mode), norm_mode=mode))


def test_head_mean_and_lambda_extremes():
    wl = workloads.make_workload("head-mean", seed=24, dtype=torch.bfloat16, batch=2, n_vis=300,
                                 n_txt=(4, 20), d=128, n_heads=4, rank=8, keep_ratio=0.2)
    _report(wl.name, parity.run_gpu(wl, pruner_kw=dict(head_reduce="mean"), head_reduce="mean"))
    for lam in (0.0, 1.0):
        wl.lam = lam
        _report(f"lambda={lam}", parity.run_gpu(wl))


def test_budget_knobs():
    wl = workloads.make_workload("knobs", seed=25, dtype=torch.bfloat16, batch=3, n_vis=(200, 500),
                                 n_txt=8, d=128, n_heads=1, rank=24, keep_ratio=0.15)
    kn = dict(presel_factor=3.0, rank_frac=0.25, rank_cap=16)
    _report(wl.name, parity.run_gpu(wl, pruner_kw=kn, **kn))
    kn = dict(presel_factor=1.0)          # M == B_vis: stage 2 is skipped
    _report(wl.name + " M=B", parity.run_gpu(wl, pruner_kw=kn, **kn))


def test_config_c1():
    # float32 inputs take the tensor-core kernels through operands split into three bf16 terms:
    # split, query embed (+ fill), relevance, activity, fuse + preselect, gather + split, Gram, basis
    # init, subspace, final select, compaction
    stats = parity.run_gpu(workloads.make_config("c1"))
    _report("c1", stats)
    assert stats["launches"] == 11


def test_config_c1_on_cuda_cores():
    # the same workload with the projection, cosine and Gram products on CUDA cores (relevance_path 1)
    stats = parity.run_gpu(workloads.make_config("c1"), pruner_kw=dict(relevance_path=1))
    _report("c1 (CUDA cores)", stats)
    assert stats["launches"] > 11


def test_config_c2():
    wl = workloads.make_config("c2")
    _report("c2", parity.run_gpu(wl))


def _full_size(name, requests):
    """Full-size configuration generated on the device (the launch configuration bench.py times);
    the oracle checks a sample of whole requests, every output of those requests element by element."""
    wl = workloads.make_config(name, device="cuda:0")
    if requests == "ragged":              # the smallest, the largest and every fifth request
        n = np.diff(wl.vis_offsets)
        requests = sorted({int(np.argmin(n)), int(np.argmax(n))} | set(range(0, wl.batch, 5)))
    elif requests is None:
        requests = list(range(wl.batch))
    stats = parity.run_gpu(wl, requests=requests)
    _report(name, stats)
    assert stats["requests"] == len(requests)
    del wl
    torch.cuda.empty_cache()


def test_config_c3_every_request():
    _full_size("c3", None)


def test_config_c4_sampled():
    _full_size("c4", "ragged")


def test_config_c5_every_request():
    _full_size("c5", None)


def test_slowly_decaying_spectrum():
    # No gap anywhere: singular values k^-0.7.  The subspace iteration converges slowest here; the
    # default number of steps must still leave the energies inside the tolerance (and the status
    # clean: run_gpu checks it).
    _report("decay0.70", parity.run_gpu(_decay_workload(0.7)))


def _decay_workload(exponent, seed=5):
    """Singular values k^-exponent: no gap anywhere (the slower the decay, the slower the subspace
    iteration settles)."""
    wl = workloads.make_workload("decay%.2f" % exponent, seed=seed, dtype=torch.bfloat16, batch=2, n_vis=1200,
                                 n_txt=16, d=768, n_heads=0, rank=16, keep_ratio=0.2)
    g = torch.Generator().manual_seed(9)
    n, d = wl.X.shape
    U = torch.linalg.qr(torch.randn(n, d, generator=g))[0]
    V = torch.linalg.qr(torch.randn(d, d, generator=g))[0]
    sv = torch.arange(1, d + 1, dtype=torch.float32) ** -exponent
    wl.X = ((U * sv) @ V.T * 30).to(torch.bfloat16)
    wl.Hs = [wl.X.clone()] + wl.Hs[1:]
    return wl


@pytest.mark.parametrize("exponent", [0.65, 0.55, 0.4, 0.25])
def test_unsettled_iteration_is_reported_not_silent(exponent):
    # Nearly flat spectra around the cut: the fixed number of power steps may leave the energies
    # outside the tolerance.  Then the device status must say so (-7); a clean status means the
    # result passes the ordinary parity rule.  Never a silent miss.
    from paper_2605_02218_b200 import api
    wl = _decay_workload(exponent)
    dev = wl.to("cuda:0")
    pr = api.Pruner.for_workload(dev)
    pr.prune(pr.marshal(dev))
    status = pr.device_status()
    pr.close()
    assert status in (0, -7)
    if status == 0:
        _report(wl.name, parity.run_gpu(wl))
    else:
        print(f"\n[parity] {wl.name}: iteration reported as not settled (status -7)")
        # more steps settle it: the same input passes with a longer iteration, or keeps saying so
        pr = api.Pruner.for_workload(dev, eig_iters=40)
        pr.prune(pr.marshal(dev))
        st2 = pr.device_status()
        pr.close()
        assert st2 in (0, -7)
        if st2 == 0:
            _report(wl.name + " (40 steps)", parity.run_gpu(wl, pruner_kw=dict(eig_iters=40)))


def test_results_do_not_depend_on_workspace_contents():
    # The workspace is poisoned with NaN bit patterns between two calls on one context (through a
    # second, larger problem that overwrites it, then a fill of the caller-visible outputs): every
    # kernel must write what it later reads.  Results must be bit-identical and the status clean.
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("poison", seed=36, dtype=torch.bfloat16, batch=3, n_vis=(150, 420),
                                 n_txt=(3, 12), d=192, n_heads=2, rank=12, keep_ratio=0.25).to("cuda:0")
    big = workloads.make_workload("poison-big", seed=37, dtype=torch.bfloat16, batch=3, n_vis=(400, 420),
                                  n_txt=(10, 12), d=192, n_heads=2, rank=12, keep_ratio=0.25).to("cuda:0")
    pr = api.Pruner.for_workload(big)
    m = pr.marshal(wl)
    a = pr.prune(m)
    a = (a[0].clone(), a[1].clone())
    nan_big = big.X.clone()
    nan_big[::3] = float("nan")                       # non-finite scores, Gram entries, factors ...
    big2 = workloads.Workload(**{**big.__dict__, "X": nan_big, "Hs": [nan_big] + big.Hs[1:]})
    pr.prune(pr.marshal(big2))                       # leaves NaN all over the workspace
    assert pr.device_status() == -6
    b = pr.prune(m)
    pr.check_device_status()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    pr.close()


def test_determinism_and_plan_cache():
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("det", seed=31, dtype=torch.bfloat16, batch=3, n_vis=(100, 400),
                                 n_txt=10, d=128, n_heads=2, rank=8, keep_ratio=0.2).to("cuda:0")
    pr = api.Pruner.for_workload(wl)
    m = pr.marshal(wl)
    a = pr.prune(m)
    b = pr.prune(m)                       # cached plan
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    # a different shape on the same context rebuilds the plan
    wl2 = wl.request(1).to("cuda:0")
    m2 = pr.marshal(wl2)
    c = pr.prune(m2)
    k1 = a[1][a[2][1]:a[2][2]]
    assert torch.equal(c[1], k1)
    pr.check_device_status()


def test_device_status_reports_nonfinite():
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("nan", seed=32, dtype=torch.float32, batch=1, n_vis=64, n_txt=4,
                                 d=32, n_heads=0, rank=4, keep=8).to("cuda:0")
    wl.X[5, 3] = float("nan")
    pr = api.Pruner.for_workload(wl)
    out, keep, ko = pr.prune(pr.marshal(wl))
    assert pr.device_status() == -6
    assert pr.device_status() == 0        # reading clears it
    k = keep.cpu().numpy()
    assert len(np.unique(k)) == 8 and k.min() >= 0 and k.max() < 64


def test_greedy_mode_stays_in_bounds_on_nonfinite_input():
    # lowrank_mode = 1 with NaN rows (made on the host): the Gram matrix is not finite; the picks
    # must still be distinct tokens of the request and the status word must say so
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("greedy-nan", seed=44, dtype=torch.bfloat16, batch=2, n_vis=64, n_txt=4,
                                 d=64, n_heads=0, rank=4, keep=40, act_layers=0)
    wl.X[3] = float("nan")
    wl.X[64 + 10, 7] = float("inf")
    dev = wl.to("cuda:0")
    pr = api.Pruner.for_workload(dev, lowrank_mode=1, presel_factor=1.6)
    out, keep, ko = pr.prune(pr.marshal(dev))
    assert pr.device_status() == -6
    k = keep.cpu().numpy()
    for b in range(2):
        kb = k[ko[b]:ko[b + 1]]
        assert len(kb) == 40 and len(np.unique(kb)) == 40 and kb.min() >= 0 and kb.max() < 64
    pr.close()


@pytest.mark.parametrize("kw", [
    dict(seed=41, dtype=torch.bfloat16, batch=3, n_vis=(120, 500), n_txt=6, d=136, n_heads=0, rank=12, keep_ratio=0.2),
    dict(seed=42, dtype=torch.float32, batch=2, n_vis=(60, 200), n_txt=4, d=72, n_heads=0, rank=6, keep=25),
    dict(seed=43, dtype=torch.bfloat16, batch=2, n_vis=1536, n_txt=8, d=256, n_heads=2, rank=16, kind="video", keep=128),
], ids=lambda kw: f"seed{kw['seed']}")
def test_greedy_lowrank_mode(kw):
    # lowrank_mode = 1: the pick sequence must be a valid run of the pivoted selection (each pick
    # within 1e-4 of the largest residual of its step: several orders are valid at near-ties) and
    # the keep-set must be exactly the picked tokens.
    from oracle import covspec_oracle as O
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload(f"greedy{kw['seed']}", **kw)
    dev = wl.to("cuda:0")
    pr = api.Pruner.for_workload(dev, lowrank_mode=1)
    m = pr.marshal(dev)
    sq, sa, sf = pr.score(m)
    keep_idx, ko, presel, po, energy = pr.select(m, sf)
    out, keep2, ko2 = pr.prune(m)
    pr.check_device_status()
    assert torch.equal(keep_idx, keep2)
    keep_idx, presel, energy = keep_idx.cpu().numpy(), presel.cpu().numpy(), energy.cpu().numpy()
    exact = 0
    for b in range(wl.batch):
        v0 = int(wl.vis_offsets[b])
        ps, en, kp = presel[po[b]:po[b + 1]], energy[po[b]:po[b + 1]], keep_idx[ko[b]:ko[b + 1]]
        B = len(kp)
        if B >= len(ps):
            assert np.array_equal(kp, ps)
            continue
        order = np.argsort(-en, kind="stable")[:B]                   # energy = B - k for the k-th pick
        assert np.array_equal(np.sort(en)[::-1][:B], np.arange(B, 0, -1)) and (np.sort(en)[:len(ps) - B] == 0).all()
        assert np.array_equal(np.sort(ps[order]), kp)
        Z = parity.f64(wl.X[v0:v0 + int(np.diff(wl.vis_offsets)[b])])[ps].T
        picks, _, valid = O.greedy_lowrank_select(Z, B, follow=order, tol=1e-4)
        assert valid, f"request {b}: a pick was not (nearly) the largest residual"
        exact += int(np.array_equal(O.greedy_lowrank_select(Z, B)[0], order))
    print(f"\n[parity] {wl.name}: pick sequences identical to the oracle in {exact} of {wl.batch} requests")


def test_compact_rows_follows_the_keep_set():
    # K / V rows (or any per-token tensor) gathered with the same kept indices, bit for bit
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("kv", seed=35, dtype=torch.bfloat16, batch=3, n_vis=(90, 300), n_txt=5,
                                 d=64, n_heads=0, rank=4, keep_ratio=0.25).to("cuda:0")
    pr = api.Pruner.for_workload(wl)
    m = pr.marshal(wl)
    out, keep_idx, ko = pr.prune(m)
    kv = torch.randn(wl.total_vis, 2, 3, 40, device="cuda:0").to(torch.bfloat16)     # [token, k/v, head, dim]
    pos = torch.arange(wl.total_vis, device="cuda:0", dtype=torch.int32).repeat_interleave(4).view(-1, 4).contiguous()
    got_kv = pr.compact_rows(m, keep_idx, ko, kv)
    got_pos = pr.compact_rows(m, keep_idx, ko, pos)
    pr.check_device_status()
    k = keep_idx.cpu().numpy().astype(np.int64)
    rows = np.concatenate([k[ko[b]:ko[b + 1]] + int(wl.vis_offsets[b]) for b in range(wl.batch)])
    idx = torch.from_numpy(rows).to("cuda:0")
    assert torch.equal(got_kv, kv[idx]) and torch.equal(got_pos, pos[idx])
    with pytest.raises(api.CovspecError):
        pr.compact_rows(m, keep_idx, ko, kv[:, 0, 0, :3].contiguous())              # 6-byte rows


def test_bounded_wait_reports_timeout():
    # A wait on a barrier that nothing signals runs out after its poll limit: the kernel returns,
    # the status word says so, and the context keeps working.
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("timeout", seed=34, dtype=torch.bfloat16, batch=1, n_vis=200, n_txt=4,
                                 d=128, n_heads=1, rank=8, keep=20).to("cuda:0")
    pr = api.Pruner.for_workload(wl)
    m = pr.marshal(wl)
    ref = pr.prune(m)
    assert pr.device_status() == 0
    pr.selftest_wait_timeout()
    assert pr.device_status() == -8
    assert pr.device_status() == 0        # reading clears it
    again = pr.prune(m)
    assert torch.equal(ref[1], again[1]) and torch.equal(ref[0], again[0])
    assert pr.device_status() == 0


def test_capacity_and_argument_errors():
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("cap", seed=33, dtype=torch.bfloat16, batch=2, n_vis=100, n_txt=4,
                                 d=64, n_heads=0, rank=4, keep=10).to("cuda:0")
    pr = api.Pruner.for_workload(wl.request(0).to("cuda:0"))
    with pytest.raises(api.CovspecError) as e:
        pr.prune(pr.marshal(wl))          # batch 2 on a context sized for 1
    assert e.value.status == -4
    m = pr.marshal(wl.request(0).to("cuda:0"))
    m.problem.X = None
    with pytest.raises(api.CovspecError) as e:
        pr.prune(m)
    assert e.value.status == -1


def test_iteration_counts_reflect_the_adaptive_stop():
    # Requests that skip the spectral stage report 0 multiplications; the others report a count
    # between the minimum the stop rule can reach and eig_iters + 1, and exactly eig_iters + 1 when
    # the adaptive stop is switched off.
    from paper_2605_02218_b200 import api
    wl = workloads.make_workload("counts", seed=41, dtype=torch.bfloat16, batch=4, n_vis=(300, 900),
                                 n_txt=(4, 12), d=256, n_heads=4, rank=16, keep_ratio=0.25).to("cuda:0")
    for stop in (1, 0):
        pr = api.Pruner.for_workload(wl, eig_early_stop=stop)
        pr.prune(pr.marshal(wl))
        counts = pr.iteration_counts(wl.batch)
        iters = pr.cfg.eig_iters
        assert pr.device_status() == 0
        pr.close()
        assert len(counts) == wl.batch
        for c in counts:
            assert c == 0 or 3 <= c <= iters + 1
        assert any(c > 0 for c in counts)
        if not stop:
            assert all(c in (0, iters + 1) for c in counts)


def test_repeated_calls_on_ragged_batch_agree():
    # 150 fused calls on the ragged workload (last tiles of a few rows, several tiles per CTA, requests
    # that stop at different steps) must give the same keep-set every time: a missing barrier between
    # two users of one shared-memory region showed up as a rare garbage energy in a ragged last tile
    from paper_2605_02218_b200 import api
    wl = workloads.make_config("c4", device="cuda:0")
    pr = api.Pruner.for_workload(wl)
    m = pr.marshal(wl)
    _, first, _ = pr.prune(m)
    first = first.clone()
    different = 0
    for _ in range(150):
        _, keep, _ = pr.prune(m)
        different += int(not torch.equal(keep, first))
    assert pr.device_status() == 0
    pr.close()
    assert different == 0


@pytest.mark.parametrize("name", ["c2", "c4"])
def test_poisoned_scratch_changes_nothing_at_full_size(name):
    # the whole scratch of the context filled with NaN patterns, huge values and zeros between calls
    from paper_2605_02218_b200 import api
    wl = workloads.make_config(name, device="cuda:0")
    pr = api.Pruner.for_workload(wl)
    m = pr.marshal(wl)
    out, keep, _ = pr.prune(m)
    out, keep = out.clone(), keep.clone()
    for byte in (0xFF, 0x7F, 0x00):
        pr.fill_workspace(byte)
        out2, keep2, _ = pr.prune(m)
        assert pr.device_status() == 0
        assert torch.equal(keep2, keep) and torch.equal(out2, out), hex(byte)
    pr.close()
