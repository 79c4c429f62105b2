"""Host logic of the benchmark: the algorithmic work of one fused call (the numerator of the roofline
fraction), the `config` object both arms print, and the bounded CPU sample."""
import numpy as np

import bench
from oracle import covspec_oracle as O


def _work(name):
    n, t, keep = bench.config_sizes(name)
    d = bench.workloads.CONFIGS[name]["d"]
    return bench.algorithmic_work(name, n, t, keep, lambda a, k: O.budgets(a, k, d))


def test_algorithmic_work_of_the_named_configurations():
    # per stage: projection 2 N d P, logits 2 T N P, Gram 2 M^2 d, eight multiplications by the
    # Gram matrix with r + 32 vectors; bytes: every input once (X, five snapshots, Q, both weights),
    # the M preselected and B kept rows gathered, the kept rows written
    w = _work("c2")
    np.testing.assert_allclose(w["relevance_flops"], 16 * (2 * 576 * 2048 * 2048 + 2 * 64 * 576 * 2048))
    np.testing.assert_allclose(w["gram_flops"], 16 * 2 * 288 ** 2 * 2048)
    np.testing.assert_allclose(w["eig_flops"], 16 * 8 * 2 * 288 ** 2 * (72 + 32))
    assert abs(w["flops"] / 1e9 - 96) < 1.5 and abs(w["bytes"] / 1e6 - 285) < 3
    w5 = _work("c5")
    assert abs(w5["flops"] / 1e9 - 3767) < 40 and abs(w5["bytes"] / 1e6 - 5927) < 40
    w3 = _work("c3")
    assert abs(w3["flops"] / 1e9 - 3441) < 40 and abs(w3["bytes"] / 1e6 - 4933) < 40
    w1 = _work("c1")
    assert abs(w1["bytes"] / 1e6 - 16.4) < 0.3


def test_fused_roofline_picks_the_binding_resource():
    peaks = dict(hbm=6500.0, tf_burst=1680.0, tf_sust=1390.0, source="test")
    r = bench.fused_roofline(_work("c5"), 5.0, peaks, False)
    assert r["bound"] == "tensor" and abs(r["frac"] - r["t_tensor_ms"] / 5.0) < 1e-12
    r1 = bench.fused_roofline(_work("c1"), 0.5, peaks, True)
    assert r1["bound"] == "hbm" and abs(r1["frac"] - r1["t_hbm_ms"] / 0.5) < 1e-12


def test_both_arms_print_the_same_config_object():
    n, t, keep = bench.config_sizes("c5")
    a = bench.config_dict("c5", n, t, keep, 1)
    b = bench.config_dict("c5", list(n), list(t), [int(k) for k in np.asarray(keep)], 1)
    assert a == b and a["workload"].startswith("c5: ") and set(a) == {"workload", "l2", "parallelism"}
    assert bench.config_sizes("c4") is None


def test_cpu_sample_is_bounded():
    wl, what = bench.oracle_sample("c5")
    assert wl.batch == 1 and wl.total_vis == 2048 and int(wl.keep[0]) == 128 and "2048" in what
    wl2, what2 = bench.oracle_sample("c2")
    assert wl2.batch == 16 and wl2.total_vis == 16 * 576
