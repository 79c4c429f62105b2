"""Parity of the whole selection path on randomly drawn shapes and settings (seeded): dtype, batch,
ragged token and query counts, feature width, head count, generator kind, number of late layers,
budgets and the preselect / rank knobs.  Every request of every drawn workload goes through the
same element-by-element checks against the oracle as the named configurations."""
import numpy as np
import pytest
import torch

from paper_2605_02218_b200 import workloads
from tests import parity

pytestmark = pytest.mark.gpu


def _draw(rng, it):
    dtype = torch.bfloat16 if rng.random() < 0.75 else torch.float32
    kw = dict(seed=int(rng.integers(1, 10**6)), dtype=dtype, batch=int(rng.integers(1, 6)),
              n_vis=(int(rng.integers(1, 200)), int(rng.integers(200, 1100))),
              n_txt=(int(rng.integers(1, 20)), int(rng.integers(20, 320))),
              d=int(rng.choice([64, 72, 128, 200, 264, 520])), n_heads=int(rng.choice([0, 1, 2, 3, 5])),
              rank=int(rng.choice([4, 8, 16, 32])), kind=str(rng.choice(["mixture", "tiles", "video"])),
              act_layers=int(rng.choice([0, 1, 4, 6])))
    if rng.random() < 0.5:
        kw["keep_ratio"] = float(rng.choice([0.05, 0.1, 0.25, 0.5, 0.9]))
    else:
        kw["keep"] = int(rng.integers(1, 150))
    knobs = {}
    if rng.random() < 0.3:
        knobs = dict(presel_factor=float(rng.choice([1.5, 3.0])), rank_frac=float(rng.choice([0.25, 0.75])))
    return kw, knobs


@pytest.mark.parametrize("seed", [1, 2])
def test_random_shapes(seed):
    from paper_2605_02218_b200 import build
    build.build()
    rng = np.random.default_rng(seed)
    requests = exact = 0
    for it in range(10):
        kw, knobs = _draw(rng, it)
        wl = workloads.make_workload(f"random{seed}-{it}", **kw)
        st = parity.run_gpu(wl, pruner_kw=knobs, **knobs)
        requests += st["requests"]
        exact += st["keep_exact"]
    print(f"\n[parity] random shapes seed {seed}: {exact} of {requests} keep-sets identical to the oracle")
    assert exact >= requests - 2          # the rest differ only inside the tolerance band (checked above)
