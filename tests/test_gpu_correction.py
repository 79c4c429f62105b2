"""Parity of covspec_correct (through the C ABI) with the float64 oracle: margin, gate, acceptance
probability, residual mass and the drawn token, for the three logit types, vocabulary sizes that
are not multiples of the vector width, and the degenerate rows (identical distributions, ties)."""
import numpy as np
import pytest
import torch

from oracle import correction_oracle as C
from paper_2605_02218_b200 import workloads

pytestmark = pytest.mark.gpu

TOL = 2e-4        # float32 softmax sums over up to 152k terms against float64; relative to 1


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2605_02218_b200 import build
    build.build()


def _check(data, gamma, got, rows=None):
    margin, gate, accept, mass, token = [t.cpu().numpy() for t in got]
    zd = data["z_draft"].cpu().double().numpy()[:, :data["vocab"]]
    zt = data["z_target"].cpu().double().numpy()[:, :data["vocab"]]
    xs, ys = data["uniforms"].cpu().numpy(), data["drafted"].cpu().numpy()
    exact = 0
    for i in (range(data["rows"]) if rows is None else rows):
        ref = C.correct_position(zd[i], zt[i], float(xs[i]), gamma, y=int(ys[i]))
        assert abs(margin[i] - ref["margin"]) <= TOL, (i, margin[i], ref["margin"])
        if abs(ref["margin"] - gamma) > TOL:
            assert gate[i] == ref["gate"]
        assert abs(accept[i] - ref["accept"]) <= TOL * max(1.0, ref["accept"]) + 2e-3 * ref["accept"]
        assert abs(mass[i] - ref["resid_mass"]) <= TOL
        tk, cdf, x = int(token[i]), ref["cdf"], float(xs[i])
        assert 0 <= tk < data["vocab"]
        # the token is the oracle's, or the uniform number sits within the tolerance of a step of the
        # oracle's cumulative distribution between the two
        assert cdf[tk] > x - TOL and (tk == 0 or cdf[tk - 1] <= x + TOL), (i, tk, ref["token"])
        assert cdf[tk] - (cdf[tk - 1] if tk else 0.0) > 0.0          # never a zero-probability token
        exact += tk == ref["token"]
    return exact


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16, torch.float32])
@pytest.mark.parametrize("vocab", [2, 37, 1000, 5003, 40000])
def test_small_vocabularies(dtype, vocab):
    from paper_2605_02218_b200 import api
    data = workloads.make_logits(seed=vocab, rows=24, vocab=vocab, dtype=dtype, device="cuda:0")
    got = api.correct(data["z_draft"], data["z_target"], data["uniforms"], 0.05, data["drafted"], vocab=vocab)
    torch.cuda.synchronize()
    exact = _check(data, 0.05, got)
    assert exact >= 22


def test_full_vocabulary_sampled_rows():
    from paper_2605_02218_b200 import api
    data = workloads.make_logits(seed=7, rows=512, vocab=151674, dtype=torch.float16, device="cuda:0")
    got = api.correct(data["z_draft"], data["z_target"], data["uniforms"], 0.02, data["drafted"], vocab=151674)
    torch.cuda.synchronize()
    exact = _check(data, 0.02, got, rows=[0, 1, 100, 255, 511])
    assert exact >= 4


def test_degenerate_rows():
    from paper_2605_02218_b200 import api
    vocab = 96
    data = workloads.make_logits(seed=3, rows=6, vocab=vocab, dtype=torch.float32, device="cuda:0")
    zd, zt = data["z_draft"], data["z_target"]
    zt[0] = zd[0]                                    # identical distributions: draw from p_t
    zd[1, :vocab] = 0.0                              # uniform draft: tie for the top, margin 0
    zd[2, :vocab] = -30.0; zd[2, 5] = 30.0           # one-hot draft: margin 1
    zt[3, :vocab] = -30.0; zt[3, 95] = 30.0          # one-hot target on the last token
    data["uniforms"][4] = 0.0
    data["uniforms"][5] = 0.99999994
    got = api.correct(zd, zt, data["uniforms"], 0.5, data["drafted"], vocab=vocab)
    torch.cuda.synchronize()
    _check(data, 0.5, got)
    margin, gate, accept, mass, token = [t.cpu().numpy() for t in got]
    assert mass[0] == 0.0 and margin[1] == 0.0 and gate[1] == 1
    assert margin[2] > 0.999 and gate[2] == 0 and token[3] == 95


def test_argument_errors():
    from paper_2605_02218_b200 import api
    z = torch.zeros(2, 12, dtype=torch.float16, device="cuda:0")          # 24-byte rows
    u = torch.zeros(2, device="cuda:0")
    with pytest.raises(api.CovspecError) as e:
        api.correct(z, z, u, 0.1)
    assert e.value.status == -2


@pytest.mark.parametrize("dtype", [torch.float16, torch.float32])
def test_branch_candidates(dtype):
    from paper_2605_02218_b200 import api
    for vocab, rows in [(37, 6), (5003, 8), (151674, 4)]:
        data = workloads.make_logits(seed=vocab + 1, rows=rows, vocab=vocab, dtype=dtype, device="cuda:0")
        fan = [api.fanout(8, 0.6, j) for j in range(rows)]
        assert fan == [C.fanout(8, 0.6, j) for j in range(rows)]
        if vocab == 5003:
            fan[0] = 1500                                         # beyond the direct-ranking size
        cand, off = api.branch_candidates(data["z_draft"], fan, data["drafted"], vocab=vocab)
        torch.cuda.synchronize()
        cand = cand.cpu().numpy()
        zd = data["z_draft"].cpu().double().numpy()[:, :vocab]
        ys = data["drafted"].cpu().numpy()
        for i in range(rows):
            want = C.bonus_candidates(zd[i], int(ys[i]), min(fan[i], vocab - 1))
            assert np.array_equal(cand[off[i]:off[i + 1]], want), (vocab, i)
