"""ctypes binding of libcovspec.so (declared in include/covspec.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch is
used for device memory and the current stream.  There is no CPU fallback: loading fails loudly
when the compiled library is missing, and every call raises on a non-zero status.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

# COVSPEC_LIBRARY selects another build of the same library (the checked one, libcovspec_debug.so)
_LIB_PATH = os.environ.get("COVSPEC_LIBRARY") or \
    os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcovspec.so")

COVSPEC_F32, COVSPEC_BF16, COVSPEC_F16 = 0, 1, 2
NORM_MODES = {"minmax": 0, "zscore": 1, "none": 2}
HEAD_REDUCE = {"max": 0, "mean": 1}

EXPORTS = [
    "covspec_default_config", "covspec_budgets", "covspec_plan_sizes", "covspec_prune_init",
    "covspec_prune_destroy", "covspec_workspace_bytes", "covspec_score", "covspec_select",
    "covspec_compact", "covspec_compact_rows", "covspec_prune", "covspec_get_device_status",
    "covspec_last_launch_count", "covspec_strerror", "covspec_last_cuda_error",
    "covspec_profile_begin", "covspec_profile_end", "covspec_profile_stage_count",
    "covspec_profile_stage_name", "covspec_query_score_static", "covspec_selftest_wait_timeout",
    "covspec_correct", "covspec_fanout", "covspec_branch_candidates",
    "covspec_uplink_bits", "covspec_downlink_bits", "covspec_comm_latency", "covspec_ema_update",
    "covspec_draft_length", "covspec_get_iteration_counts", "covspec_build_has_bounds_checks",
    "covspec_selftest_fill_workspace",
]
STATIC_MAX_BATCH = 256
STATIC_MAX_QUERY_ELEMS = 1 << 20


class Config(C.Structure):
    _fields_ = [
        ("dtype", C.c_int), ("d", C.c_int), ("n_heads", C.c_int), ("head_dim", C.c_int),
        ("act_layers", C.c_int), ("lam", C.c_float), ("norm_mode", C.c_int),
        ("head_reduce", C.c_int), ("presel_factor", C.c_float), ("rank_frac", C.c_float),
        ("rank_cap", C.c_int), ("eig_iters", C.c_int), ("eig_oversample", C.c_int),
        ("max_batch", C.c_int), ("max_total_vis", C.c_longlong), ("max_total_txt", C.c_longlong),
        ("max_vis_per_req", C.c_int), ("max_presel_per_req", C.c_int),
        ("max_total_presel", C.c_longlong), ("relevance_path", C.c_int), ("lowrank_mode", C.c_int),
        ("ritz_window", C.c_int), ("activity_overlap", C.c_int), ("conv_tol", C.c_float),
        ("eig_early_stop", C.c_int),
    ]


class Problem(C.Structure):
    _fields_ = [
        ("batch", C.c_int), ("X", C.c_void_p), ("vis_offsets", C.POINTER(C.c_int)),
        ("Q", C.c_void_p), ("txt_offsets", C.POINTER(C.c_int)), ("Wq", C.c_void_p),
        ("Wk", C.c_void_p), ("Hs", C.POINTER(C.c_void_p)), ("keep", C.POINTER(C.c_int)),
        ("keep_ratio", C.c_double),
    ]


class CovspecError(RuntimeError):
    def __init__(self, status, where):
        lib = load_library()
        msg = lib.covspec_strerror(status).decode()
        if status == -5:
            msg += " (" + lib.covspec_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {msg} [{status}]")
        self.status = status


_lib = None


def load_library():
    """Loads libcovspec.so (built by paper_2605_02218_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} not found: build it with `python -m paper_2605_02218_b200.build` "
            "(there is no fallback path)")
    lib = C.CDLL(_LIB_PATH)
    vp, ip, fp = C.c_void_p, C.POINTER(C.c_int), C.c_void_p
    lib.covspec_default_config.argtypes = [C.POINTER(Config)]
    lib.covspec_default_config.restype = None
    lib.covspec_budgets.argtypes = [C.POINTER(Config), C.c_int, C.c_int, ip, ip, ip]
    lib.covspec_plan_sizes.argtypes = [C.POINTER(Config), C.POINTER(Problem), ip, ip]
    lib.covspec_prune_init.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    lib.covspec_prune_destroy.argtypes = [vp]
    lib.covspec_workspace_bytes.argtypes = [vp]
    lib.covspec_workspace_bytes.restype = C.c_longlong
    lib.covspec_score.argtypes = [vp, C.POINTER(Problem), fp, fp, fp, vp]
    lib.covspec_select.argtypes = [vp, C.POINTER(Problem), fp, vp, ip, vp, fp, vp]
    lib.covspec_compact.argtypes = [vp, C.POINTER(Problem), vp, ip, vp, vp, vp]
    lib.covspec_prune.argtypes = [vp, C.POINTER(Problem), vp, vp, ip, vp]
    lib.covspec_compact_rows.argtypes = [vp, C.POINTER(Problem), vp, ip, vp, C.c_longlong, vp, vp]
    lib.covspec_get_device_status.argtypes = [vp, vp]
    lib.covspec_selftest_wait_timeout.argtypes = [vp, vp]
    lib.covspec_selftest_fill_workspace.argtypes = [vp, C.c_int, vp]
    lib.covspec_get_iteration_counts.argtypes = [vp, C.c_int, ip, vp]
    lib.covspec_fanout.argtypes = [C.c_int, C.c_double, C.c_int]
    lib.covspec_uplink_bits.argtypes = [C.c_longlong, C.c_int, C.c_longlong, C.c_int]
    lib.covspec_uplink_bits.restype = C.c_double
    lib.covspec_downlink_bits.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_longlong, C.c_int]
    lib.covspec_downlink_bits.restype = C.c_double
    lib.covspec_comm_latency.argtypes = [C.c_double, C.c_double, C.c_double]
    lib.covspec_comm_latency.restype = C.c_double
    lib.covspec_ema_update.argtypes = [C.c_double, C.c_double, C.c_int, C.c_int]
    lib.covspec_ema_update.restype = C.c_double
    lib.covspec_draft_length.argtypes = [C.c_int] + [C.c_double] * 6 + [C.c_int, C.c_int]
    lib.covspec_branch_candidates.argtypes = [C.c_int, C.c_int, C.c_int, C.c_longlong, vp, vp, vp, C.c_int, vp, vp]
    lib.covspec_correct.argtypes = [C.c_int, C.c_int, C.c_int, C.c_longlong, vp, vp, vp, vp, C.c_float,
                                    vp, vp, vp, vp, vp, vp]
    lib.covspec_last_launch_count.argtypes = [vp]
    lib.covspec_strerror.argtypes = [C.c_int]
    lib.covspec_strerror.restype = C.c_char_p
    lib.covspec_last_cuda_error.argtypes = []
    lib.covspec_last_cuda_error.restype = C.c_char_p
    lib.covspec_query_score_static.argtypes = [C.c_int, C.c_int, C.c_int, vp, ip, vp, ip, fp, vp]
    lib.covspec_profile_begin.argtypes = [vp, C.c_int]
    lib.covspec_profile_end.argtypes = [vp, C.POINTER(C.c_double), C.c_int, ip]
    lib.covspec_profile_stage_count.argtypes = []
    lib.covspec_profile_stage_name.argtypes = [C.c_int]
    lib.covspec_profile_stage_name.restype = C.c_char_p
    _lib = lib
    return lib


def default_config(**overrides) -> Config:
    cfg = Config()
    load_library().covspec_default_config(C.byref(cfg))
    for k, v in overrides.items():
        if k == "lambda_":
            k = "lam"
        if k == "norm_mode" and isinstance(v, str):
            v = NORM_MODES[v]
        if k == "head_reduce" and isinstance(v, str):
            v = HEAD_REDUCE[v]
        if not hasattr(cfg, k):
            raise KeyError(k)
        setattr(cfg, k, v)
    return cfg


def budgets(cfg: Config, n: int, keep: int):
    b, m, r = C.c_int(), C.c_int(), C.c_int()
    st = load_library().covspec_budgets(C.byref(cfg), n, keep, C.byref(b), C.byref(m), C.byref(r))
    if st:
        raise CovspecError(st, "covspec_budgets")
    return b.value, m.value, r.value


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.POINTER(C.c_int))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


class _Marshalled:
    """Keeps the host arrays referenced by a Problem alive."""

    def __init__(self, X, Q, vis_offsets, txt_offsets, Wq=None, Wk=None, Hs=None, keep=None,
                 keep_ratio=0.0):
        self.tensors = (X, Q, Wq, Wk, Hs)
        for t in (X, Q, Wq, Wk) + tuple(Hs or ()):
            if t is not None:
                assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors required"
        self.vis, vis_p = _i32(vis_offsets)
        self.txt, txt_p = _i32(txt_offsets)
        self.batch = len(self.vis) - 1
        keep_p = None
        if keep is not None:
            self.keep, keep_p = _i32(keep)
        hs_p = None
        if Hs:
            self.hs = (C.c_void_p * len(Hs))(*[h.data_ptr() for h in Hs])
            hs_p = C.cast(self.hs, C.POINTER(C.c_void_p))
        self.problem = Problem(self.batch, _ptr(X), vis_p, _ptr(Q), txt_p, _ptr(Wq), _ptr(Wk), hs_p,
                               keep_p, float(keep_ratio))


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Pruner:
    """One context (workspace + plan cache) for a fixed configuration and capacity."""

    def __init__(self, cfg: Config):
        self.lib = load_library()
        self.cfg = cfg
        self._ctx = C.c_void_p()
        st = self.lib.covspec_prune_init(C.byref(cfg), C.byref(self._ctx))
        if st:
            raise CovspecError(st, "covspec_prune_init")
        self._keepalive = None

    @classmethod
    def for_workload(cls, wl, **overrides) -> "Pruner":
        """Context sized exactly for a workloads.Workload."""
        lib = load_library()
        cfg = default_config(
            dtype=COVSPEC_BF16 if wl.dtype == torch.bfloat16 else COVSPEC_F32, d=wl.d,
            n_heads=wl.n_heads, head_dim=wl.head_dim if wl.n_heads else 0,
            act_layers=wl.act_layers, lam=wl.lam, **overrides)
        n = np.diff(wl.vis_offsets)
        cfg.max_batch = wl.batch
        cfg.max_total_vis = int(wl.vis_offsets[-1])
        cfg.max_total_txt = int(wl.txt_offsets[-1])
        cfg.max_vis_per_req = int(n.max())
        vis, vis_p = _i32(wl.vis_offsets)
        txt, txt_p = _i32(wl.txt_offsets)
        keep, keep_p = _i32(wl.keep)
        prob = Problem(wl.batch, None, vis_p, None, txt_p, None, None, None, keep_p, 0.0)
        po = np.zeros(wl.batch + 1, dtype=np.int32)
        st = lib.covspec_plan_sizes(C.byref(cfg), C.byref(prob), None,
                                    po.ctypes.data_as(C.POINTER(C.c_int)))
        if st:
            raise CovspecError(st, "covspec_plan_sizes")
        cfg.max_total_presel = int(po[-1])
        cfg.max_presel_per_req = int(np.diff(po).max())
        return cls(cfg)

    def close(self):
        if self._ctx:
            self.lib.covspec_prune_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def workspace_bytes(self) -> int:
        return int(self.lib.covspec_workspace_bytes(self._ctx))

    @property
    def last_launch_count(self) -> int:
        return int(self.lib.covspec_last_launch_count(self._ctx))

    def plan_sizes(self, m: _Marshalled):
        ko = np.zeros(m.batch + 1, dtype=np.int32)
        po = np.zeros(m.batch + 1, dtype=np.int32)
        st = self.lib.covspec_plan_sizes(C.byref(self.cfg), C.byref(m.problem),
                                         ko.ctypes.data_as(C.POINTER(C.c_int)),
                                         po.ctypes.data_as(C.POINTER(C.c_int)))
        if st:
            raise CovspecError(st, "covspec_plan_sizes")
        return ko, po

    def marshal(self, wl=None, **kw) -> _Marshalled:
        if wl is not None:
            kw = dict(X=wl.X, Q=wl.Q, vis_offsets=wl.vis_offsets, txt_offsets=wl.txt_offsets,
                      Wq=wl.Wq, Wk=wl.Wk, Hs=wl.Hs, keep=wl.keep)
        return _Marshalled(**kw)

    # ---- the entry points --------------------------------------------------------------------
    def score(self, m: _Marshalled):
        """covspec_score: returns (s_query, s_act, s_fused) float32 device tensors."""
        n = int(m.vis[-1])
        dev = m.tensors[0].device
        sq = torch.empty(n, dtype=torch.float32, device=dev)
        sa = torch.empty(n, dtype=torch.float32, device=dev)
        sf = torch.empty(n, dtype=torch.float32, device=dev)
        st = self.lib.covspec_score(self._ctx, C.byref(m.problem), _ptr(sq), _ptr(sa), _ptr(sf),
                                    _stream())
        if st:
            raise CovspecError(st, "covspec_score")
        return sq, (sa if self.cfg.act_layers > 0 else None), sf

    def select(self, m: _Marshalled, s_fused: torch.Tensor):
        """covspec_select: returns (keep_idx, keep_offsets, presel_idx, presel_offsets, energy)."""
        ko, po = self.plan_sizes(m)
        dev = s_fused.device
        keep_idx = torch.empty(int(ko[-1]), dtype=torch.int32, device=dev)
        presel = torch.empty(int(po[-1]), dtype=torch.int32, device=dev)
        energy = torch.empty(int(po[-1]), dtype=torch.float32, device=dev)
        ko2 = np.zeros_like(ko)
        st = self.lib.covspec_select(self._ctx, C.byref(m.problem), _ptr(s_fused), _ptr(keep_idx),
                                     ko2.ctypes.data_as(C.POINTER(C.c_int)), _ptr(presel),
                                     _ptr(energy), _stream())
        if st:
            raise CovspecError(st, "covspec_select")
        assert np.array_equal(ko, ko2)
        return keep_idx, ko, presel, po, energy

    def compact(self, m: _Marshalled, keep_idx: torch.Tensor, keep_offsets: np.ndarray):
        """covspec_compact: returns (out_hidden [sum B_vis, d], out_pos)."""
        X = m.tensors[0]
        ko, ko_p = _i32(keep_offsets)
        out = torch.empty((int(ko[-1]), X.shape[1]), dtype=X.dtype, device=X.device)
        pos = torch.empty(int(ko[-1]), dtype=torch.int32, device=X.device)
        st = self.lib.covspec_compact(self._ctx, C.byref(m.problem), _ptr(keep_idx), ko_p, _ptr(out),
                                      _ptr(pos), _stream())
        if st:
            raise CovspecError(st, "covspec_compact")
        return out, pos

    def compact_rows(self, m: _Marshalled, keep_idx: torch.Tensor, keep_offsets: np.ndarray,
                     src: torch.Tensor):
        """covspec_compact_rows: gathers the kept tokens' rows of another per-token tensor
        (first dimension = visual tokens, like X)."""
        assert src.is_cuda and src.is_contiguous() and src.shape[0] == int(m.vis[-1])
        ko, ko_p = _i32(keep_offsets)
        row_bytes = src[0].numel() * src.element_size()
        out = torch.empty((int(ko[-1]),) + tuple(src.shape[1:]), dtype=src.dtype, device=src.device)
        st = self.lib.covspec_compact_rows(self._ctx, C.byref(m.problem), _ptr(keep_idx), ko_p, _ptr(src),
                                           row_bytes, _ptr(out), _stream())
        if st:
            raise CovspecError(st, "covspec_compact_rows")
        return out

    def prune(self, m: _Marshalled, out: Optional[torch.Tensor] = None,
              keep_idx: Optional[torch.Tensor] = None):
        """covspec_prune: the fused path.  Returns (out_hidden, keep_idx, keep_offsets)."""
        X = m.tensors[0]
        ko = np.zeros(m.batch + 1, dtype=np.int32)
        if out is None or keep_idx is None:
            ko, _ = self.plan_sizes(m)
            out = torch.empty((int(ko[-1]), X.shape[1]), dtype=X.dtype, device=X.device)
            keep_idx = torch.empty(int(ko[-1]), dtype=torch.int32, device=X.device)
        st = self.lib.covspec_prune(self._ctx, C.byref(m.problem), _ptr(out), _ptr(keep_idx),
                                    ko.ctypes.data_as(C.POINTER(C.c_int)), _stream())
        if st:
            raise CovspecError(st, "covspec_prune")
        return out, keep_idx, ko

    def profile_begin(self, max_calls: int):
        st = self.lib.covspec_profile_begin(self._ctx, int(max_calls))
        if st:
            raise CovspecError(st, "covspec_profile_begin")

    def profile_end(self):
        """Returns ({stage name: summed milliseconds}, number of profiled prune calls)."""
        n = self.lib.covspec_profile_stage_count()
        ms = (C.c_double * n)()
        calls = C.c_int()
        st = self.lib.covspec_profile_end(self._ctx, ms, n, C.byref(calls))
        if st:
            raise CovspecError(st, "covspec_profile_end")
        names = [self.lib.covspec_profile_stage_name(i).decode() for i in range(n)]
        return dict(zip(names, list(ms))), calls.value

    def selftest_wait_timeout(self):
        """covspec_selftest_wait_timeout: makes one bounded wait run out on purpose."""
        st = self.lib.covspec_selftest_wait_timeout(self._ctx, _stream())
        if st:
            raise CovspecError(st, "covspec_selftest_wait_timeout")

    def iteration_counts(self, batch: int):
        """covspec_get_iteration_counts: multiplications by the Gram matrix per request of the last call."""
        out = np.zeros(batch, dtype=np.int32)
        st = self.lib.covspec_get_iteration_counts(self._ctx, int(batch), out.ctypes.data_as(C.POINTER(C.c_int)),
                                                   _stream())
        if st:
            raise CovspecError(st, "covspec_get_iteration_counts")
        return out

    def fill_workspace(self, byte: int):
        """covspec_selftest_fill_workspace: poisons the context's scratch before the next call."""
        st = self.lib.covspec_selftest_fill_workspace(self._ctx, int(byte), _stream())
        if st:
            raise CovspecError(st, "covspec_selftest_fill_workspace")

    def device_status(self) -> int:
        return int(self.lib.covspec_get_device_status(self._ctx, _stream()))

    def check_device_status(self):
        st = self.device_status()
        if st:
            raise CovspecError(st, "device status")


def query_score_static(X: torch.Tensor, Q: torch.Tensor, vis_offsets, txt_offsets,
                       out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """covspec_query_score_static: Eq. 10 with the identity embedding for callers that must not
    allocate device memory (a serving loop with a fully committed memory pool, a process whose
    allocator belongs to another framework).  The library call itself allocates nothing; pass
    `out` (float32, one element per visual token) to keep this wrapper allocation-free as well."""
    lib = load_library()
    assert X.is_cuda and Q.is_cuda and X.is_contiguous() and Q.is_contiguous() and X.dtype == Q.dtype
    vis, vis_p = _i32(vis_offsets)
    txt, txt_p = _i32(txt_offsets)
    if out is None:
        out = torch.empty(int(vis[-1]), dtype=torch.float32, device=X.device)
    dtype = COVSPEC_BF16 if X.dtype == torch.bfloat16 else COVSPEC_F32
    st = lib.covspec_query_score_static(dtype, X.shape[1], len(vis) - 1, _ptr(X), vis_p, _ptr(Q),
                                        txt_p, _ptr(out), _stream())
    if st:
        raise CovspecError(st, "covspec_query_score_static")
    return out


_LOGIT_DTYPES = {torch.float32: COVSPEC_F32, torch.bfloat16: COVSPEC_BF16, torch.float16: COVSPEC_F16}


def correct(z_draft: torch.Tensor, z_target: torch.Tensor, uniforms: torch.Tensor, gamma: float,
            drafted: Optional[torch.Tensor] = None, vocab: Optional[int] = None):
    """covspec_correct: gating (Eq. 16-17), acceptance probability (Eq. 5) and the residual
    correction draw (Eq. 6) for every row of two logit matrices [rows, ld] (ld >= vocab).
    Returns (margin, gate, accept, resid_mass, token) device tensors."""
    lib = load_library()
    assert z_draft.is_cuda and z_draft.is_contiguous() and z_target.is_contiguous()
    assert z_draft.shape == z_target.shape and z_draft.dtype == z_target.dtype
    rows, ld = z_draft.shape
    vocab = ld if vocab is None else vocab
    dev = z_draft.device
    margin = torch.empty(rows, dtype=torch.float32, device=dev)
    gate = torch.empty(rows, dtype=torch.int32, device=dev)
    accept = torch.empty(rows, dtype=torch.float32, device=dev)
    mass = torch.empty(rows, dtype=torch.float32, device=dev)
    token = torch.empty(rows, dtype=torch.int32, device=dev)
    st = lib.covspec_correct(_LOGIT_DTYPES[z_draft.dtype], rows, vocab, ld, _ptr(z_draft), _ptr(z_target),
                             _ptr(drafted), _ptr(uniforms), float(gamma), _ptr(margin), _ptr(gate),
                             _ptr(accept), _ptr(mass), _ptr(token), _stream())
    if st:
        raise CovspecError(st, "covspec_correct")
    return margin, gate, accept, mass, token


def fanout(f0: int, rho: float, j: int) -> int:
    """covspec_fanout: F_j = ceil(F_0 * rho^j) (Eq. 23)."""
    v = load_library().covspec_fanout(int(f0), float(rho), int(j))
    if v < 0:
        raise CovspecError(v, "covspec_fanout")
    return v


def branch_candidates(z_draft: torch.Tensor, fanouts, drafted: Optional[torch.Tensor] = None,
                      vocab: Optional[int] = None):
    """covspec_branch_candidates: the F_j largest draft logits of every row, the drafted token
    excluded.  `fanouts`: one int per row.  Returns (cand int32 device tensor, offsets numpy)."""
    lib = load_library()
    rows, ld = z_draft.shape
    vocab = ld if vocab is None else vocab
    f = np.asarray(fanouts, dtype=np.int64)
    assert len(f) == rows
    off = np.concatenate([[0], np.cumsum(f)]).astype(np.int32)
    d_off = torch.from_numpy(off).to(z_draft.device)
    cand = torch.empty(max(int(off[-1]), 1), dtype=torch.int32, device=z_draft.device)
    st = lib.covspec_branch_candidates(_LOGIT_DTYPES[z_draft.dtype], rows, vocab, ld, _ptr(z_draft),
                                       _ptr(drafted), _ptr(d_off), int(f.max()) if rows else 0,
                                       _ptr(cand), _stream())
    if st:
        raise CovspecError(st, "covspec_branch_candidates")
    return cand[:int(off[-1])], off
