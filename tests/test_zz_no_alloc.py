"""The allocation-free query-score entry point (for callers that cannot call cudaMalloc: serving
loops whose memory pool is fully committed, processes whose device allocator belongs to another
framework) must give what covspec_score gives, and what the CPU oracle's Eq. 10 gives.  Collected last on purpose: a run that stops at the
first failure has then already run every other test.  Works alone in a fresh process and after the
other tests; calls go through the C ABI."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2605_02218_b200 import workloads
from tests.parity import TAU


@pytest.mark.gpu
def test_static_query_score_matches_context_entry_point_twice_in_a_row():
    from paper_2605_02218_b200 import api, build
    build.build()
    # Two different problems back to back: the second call finds the first call's leftovers in the
    # shared scratch array and must not be affected by them.
    specs = [
        dict(seed=41, dtype=torch.bfloat16, batch=5, n_vis=(90, 700), n_txt=(1, 50), d=264),
        dict(seed=42, dtype=torch.float32, batch=3, n_vis=(33, 200), n_txt=(2, 9), d=72),
    ]
    wls = [workloads.make_workload("static", n_heads=0, rank=8, keep_ratio=0.2, act_layers=0,
                                   **kw).to("cuda:0") for kw in specs]
    expected = []
    for wl in wls:
        pr = api.Pruner.for_workload(wl)
        sq, _, _ = pr.score(pr.marshal(wl))
        pr.check_device_status()
        expected.append(sq.clone())
        pr.close()
    outs = [torch.full((wl.total_vis,), float("nan"), device="cuda:0") for wl in wls]
    # warm-up call: the first call on a device looks up the scratch array's address
    api.query_score_static(wls[1].X, wls[1].Q, wls[1].vis_offsets, wls[1].txt_offsets, out=outs[1])
    outs[1].fill_(float("nan"))
    torch.cuda.synchronize()
    # free device memory as the driver sees it: an allocation made inside the library (which
    # torch's own counters cannot see) would lower it
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = torch.cuda.memory_allocated()
    for wl, out in zip(wls, outs):                       # two calls in a row, no sync in between
        api.query_score_static(wl.X, wl.Q, wl.vis_offsets, wl.txt_offsets, out=out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the call changed the device's free memory"
    assert torch.cuda.memory_allocated() == torch_before
    from oracle import covspec_oracle as oracle
    for wl, out, want in zip(wls, outs, expected):
        err = (out - want).abs().max().item()
        scale = want.abs().max().item()
        assert err <= TAU * scale, f"static entry point differs from covspec_score: {err:.3e}"
        got = out.cpu().double().numpy()
        for b in range(wl.batch):                        # and against the definition itself
            v0, v1 = int(wl.vis_offsets[b]), int(wl.vis_offsets[b + 1])
            t0, t1 = int(wl.txt_offsets[b]), int(wl.txt_offsets[b + 1])
            ref = oracle.query_relevance(wl.X[v0:v1].cpu().double().numpy(), wl.Q[t0:t1].cpu().double().numpy())
            assert np.abs(got[v0:v1] - ref).max() <= TAU * np.abs(ref).max()
    # and once more on the first problem, after the scratch held the second one
    again = api.query_score_static(wls[0].X, wls[0].Q, wls[0].vis_offsets, wls[0].txt_offsets)
    assert (again - expected[0]).abs().max().item() <= TAU * expected[0].abs().max().item()


@pytest.mark.gpu
def test_static_entry_point_rejects_what_does_not_fit():
    from paper_2605_02218_b200 import api, build
    build.build()
    lib = api.load_library()
    d = 1024
    t = api.STATIC_MAX_QUERY_ELEMS // d + 1              # one query element too many
    X = torch.zeros((4, d), dtype=torch.bfloat16, device="cuda:0")
    Q = torch.zeros((t, d), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(api.CovspecError) as e:
        api.query_score_static(X, Q, [0, 4], [0, t])
    assert e.value.status == -9 and "capacity" in str(e.value)
    nb = api.STATIC_MAX_BATCH + 1                        # one request too many
    with pytest.raises(api.CovspecError) as e:
        api.query_score_static(X.new_zeros((nb, d)), Q[:nb], np.arange(nb + 1), np.arange(nb + 1))
    assert e.value.status == -9
    # a problem exactly at the limit is accepted
    t = api.STATIC_MAX_QUERY_ELEMS // d
    out = api.query_score_static(X, Q[:t], [0, 4], [0, t])
    torch.cuda.synchronize()
    assert out.shape == (4,)
