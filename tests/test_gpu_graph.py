"""The fused call inside a CUDA graph: once the plan of a batch shape is cached, covspec_prune copies
nothing from the host and waits for nothing, so stream capture can record it; the replayed graph
must give what the direct call gives, also after the inputs' contents have changed in place."""
import numpy as np
import pytest
import torch

from paper_2605_02218_b200 import api, workloads

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c1", "c2"])
def test_captured_prune_call_replays(name):
    wl = workloads.make_config(name, device="cuda:0")
    other = workloads.make_config(name, device="cuda:0", seed=4321)       # same shapes, other contents
    pr = api.Pruner.for_workload(wl)
    m = pr.marshal(wl)
    out, idx, ko = pr.prune(m)                       # direct call: uploads the plan
    torch.cuda.synchronize()
    want = (out.clone(), idx.clone())
    assert pr.last_launch_count in (10, 11)

    out.zero_(); idx.zero_()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        pr.prune(m, out=out, keep_idx=idx)
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want[0]) and torch.equal(idx, want[1])
    assert pr.device_status() == 0

    # new contents in the buffers the graph points to
    def flat(t):
        return [x for x in t[:4] if x is not None] + list(t[4] or ())
    for dst, src in zip(flat(m.tensors), flat(pr.marshal(other).tensors)):
        dst.copy_(src)
    graph.replay()
    torch.cuda.synchronize()
    got = (out.clone(), idx.clone())
    out2, idx2, ko2 = pr.prune(m)
    torch.cuda.synchronize()
    assert np.array_equal(ko, ko2)
    assert torch.equal(got[0], out2) and torch.equal(got[1], idx2)
    assert not torch.equal(got[1], want[1])          # the other contents keep other tokens
    assert pr.device_status() == 0
