"""The C-ABI library loads without a GPU, exports every symbol the header declares, and its
host-only entry points (budgets, plan sizes, defaults, error text) agree with the oracle's integer
logic.  No kernel is launched here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import covspec_oracle as O
from paper_2605_02218_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "covspec.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(covspec_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_defaults(lib):
    cfg = api.default_config()
    assert (cfg.lam, cfg.presel_factor, cfg.rank_frac, cfg.rank_cap) == (0.5, 2.0, 0.5, 128)
    assert cfg.act_layers == 4 and cfg.norm_mode == 0 and cfg.head_reduce == 0
    assert cfg.dtype == api.COVSPEC_BF16 and cfg.head_dim == 128


@pytest.mark.parametrize("n,keep,d", [(576, 64, 1024), (576, 144, 2048), (2880, 288, 4096),
                                      (16384, 1024, 3584), (768, 64, 4096), (5, 9, 16), (2, 1, 16),
                                      (1, 1, 8), (100, 3, 8), (4096, 820, 1536), (256, 52, 1536),
                                      (300, 299, 64), (300, 150, 64), (300, 151, 64)])
def test_budgets_match_oracle(lib, n, keep, d):
    cfg = api.default_config(d=d)
    assert api.budgets(cfg, n, keep) == O.budgets(n, keep, d)


def test_budgets_other_factors(lib):
    cfg = api.default_config(d=512, presel_factor=1.0, rank_frac=1.0, rank_cap=16)
    for n, keep in [(100, 10), (100, 30), (7, 3)]:
        assert api.budgets(cfg, n, keep) == O.budgets(n, keep, 512, 1.0, 1.0, 16)
    cfg = api.default_config(d=512, presel_factor=3.5, rank_frac=0.25)
    for n, keep in [(1000, 10), (1000, 333), (64, 9)]:
        assert api.budgets(cfg, n, keep) == O.budgets(n, keep, 512, 3.5, 0.25, 128)


def _problem(vis, txt, keep=None, ratio=0.0):
    vis = np.asarray(vis, dtype=np.int32)
    txt = np.asarray(txt, dtype=np.int32)
    ip = C.POINTER(C.c_int)
    kp = None
    if keep is not None:
        keep = np.asarray(keep, dtype=np.int32)
        kp = keep.ctypes.data_as(ip)
    prob = api.Problem(len(vis) - 1, None, vis.ctypes.data_as(ip), None, txt.ctypes.data_as(ip),
                       None, None, None, kp, ratio)
    return prob, (vis, txt, keep)


def test_plan_sizes_and_ratio_rule(lib):
    from paper_2605_02218_b200.workloads import keep_from_ratio
    cfg = api.default_config(d=1536)
    ns = [256, 4096, 1000, 577, 1]
    vis = np.concatenate([[0], np.cumsum(ns)])
    txt = np.arange(len(ns) + 1) * 3
    prob, hold = _problem(vis, txt, ratio=0.2)
    ko = np.zeros(len(ns) + 1, dtype=np.int32)
    po = np.zeros(len(ns) + 1, dtype=np.int32)
    ip = C.POINTER(C.c_int)
    assert lib.covspec_plan_sizes(C.byref(cfg), C.byref(prob), ko.ctypes.data_as(ip),
                                  po.ctypes.data_as(ip)) == 0
    want = [O.budgets(n, keep_from_ratio(n, 0.2), 1536) for n in ns]
    assert list(np.diff(ko)) == [w[0] for w in want]
    assert list(np.diff(po)) == [w[1] for w in want]
    # 25 % of 576 and 10 % of 2880 are exact integers
    assert keep_from_ratio(576, 0.25) == 144 and keep_from_ratio(2880, 0.10) == 288


def test_host_side_rejections(lib):
    cfg = api.default_config(d=64)
    ip = C.POINTER(C.c_int)
    bad = [
        (_problem([0, 5, 5], [0, 1, 2], keep=[1, 1]), -2),      # empty request
        (_problem([0, 5, 3], [0, 1, 2], keep=[1, 1]), -2),      # offsets not monotone
        (_problem([1, 5, 9], [0, 1, 2], keep=[1, 1]), -2),      # does not start at 0
        (_problem([0, 5, 9], [0, 1, 1], keep=[1, 1]), -2),      # request without query elements
        (_problem([0, 5, 9], [0, 1, 2], keep=[1, 0]), -2),      # zero budget
        (_problem([0, 5, 9], [0, 1, 2], ratio=0.0), -1),        # neither keep nor ratio
        (_problem([0, 5, 9], [0, 1, 2], ratio=1.5), -1),
    ]
    for (prob, hold), code in bad:
        assert lib.covspec_plan_sizes(C.byref(cfg), C.byref(prob), None, None) == code
    assert lib.covspec_plan_sizes(None, None, None, None) == -1
    out = C.c_void_p()
    # configuration errors are reported before any allocation
    for kw, code in [(dict(d=12), -3), (dict(d=64, n_heads=2, head_dim=64), -3),
                     (dict(d=64, lam=1.5), -1), (dict(d=64, rank_cap=150, eig_oversample=32), -3),
                     (dict(d=64, act_layers=40), -3), (dict(d=64, presel_factor=0.5), -1),
                     (dict(d=64, dtype=7), -1), (dict(d=64, relevance_path=3), -1)]:
        c = api.default_config(**kw)
        c.max_batch, c.max_total_vis, c.max_total_txt, c.max_vis_per_req = 1, 8, 8, 8
        assert lib.covspec_prune_init(C.byref(c), C.byref(out)) == code and not out.value
    c = api.default_config(d=64)     # capacities missing
    assert lib.covspec_prune_init(C.byref(c), C.byref(out)) == -1


def test_strerror(lib):
    texts = {lib.covspec_strerror(s).decode() for s in range(0, -11, -1)}
    assert len(texts) == 11 and "unknown status" not in texts
    assert lib.covspec_strerror(-99).decode() == "unknown status"


def test_binding_fails_loudly_without_library(monkeypatch):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "_LIB_PATH", "/nonexistent/libcovspec.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        api.load_library()


def test_checked_build_exports_the_same_interface(lib):
    # libcovspec_debug.so: the same sources with the index tests compiled in
    path = build.build(debug_bounds=True)
    dbg = C.CDLL(path)
    for name in api.EXPORTS:
        assert getattr(dbg, name) is not None
    assert dbg.covspec_build_has_bounds_checks() == 1
    assert lib.covspec_build_has_bounds_checks() == 0
    dbg.covspec_strerror.restype = C.c_char_p
    assert b"out of range" in dbg.covspec_strerror(-10)
