"""ctypes front end of the CPU oracle (``spec_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  The product package never imports it.
Arguments are numpy arrays on the host; nothing here touches a GPU or the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, "spec_oracle.c"), os.path.join(_HERE, "otlp_oracle.c")]
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over sequences) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(f) for f in _SRCS):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", _LIB] + _SRCS + ["-lm"])
    return _LIB


class _In(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("N", C.c_int32), ("V", C.c_int32), ("logits_dtype", C.c_int32),
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
        ("seq_stride", C.c_int64), ("node_stride", C.c_int64),
        ("parent", C.c_void_p), ("topo_seq_stride", C.c_int64), ("token", C.c_void_p),
        ("temperature", C.c_float), ("top_k", C.c_int32), ("top_p", C.c_float),
        ("temperature_per_seq", C.c_void_p), ("u_accept", C.c_void_p), ("u_bonus", C.c_void_p),
    ]


class _Out(C.Structure):
    _fields_ = [
        ("accepted_node", C.c_void_p), ("accept_len", C.c_void_p), ("out_tokens", C.c_void_p),
        ("bonus_token", C.c_void_p), ("residual", C.c_void_p), ("bonus_margin", C.c_void_p),
        ("trace_node", C.c_void_p), ("trace_thr", C.c_void_p), ("trace_acc", C.c_void_p),
        ("trace_len", C.c_void_p), ("status", C.c_void_p),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_row_probs.restype = C.c_int
        _lib.oracle_row_probs.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_int32, C.c_double,
                                          C.c_void_p, C.c_void_p]
        _lib.oracle_inverse_cdf.restype = C.c_int32
        _lib.oracle_inverse_cdf.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_void_p]
        for name in ("oracle_verify_specinfer", "oracle_verify_traversal"):
            f = getattr(_lib, name)
            f.restype = C.c_int32
            f.argtypes = [C.POINTER(_In), C.POINTER(_Out)]
        _lib.oracle_specinfer_tables.restype = C.c_int32
        _lib.oracle_specinfer_tables.argtypes = [C.POINTER(_In)] + [C.c_void_p] * 4
        _lib.oracle_traversal_tables.restype = C.c_int32
        _lib.oracle_traversal_tables.argtypes = [C.POINTER(_In)] + [C.c_void_p] * 4
        _lib.oracle_tree_probs.restype = C.c_int32
        _lib.oracle_tree_probs.argtypes = [C.POINTER(_In), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.oracle_sample_bonus.restype = C.c_int32
        _lib.oracle_sample_bonus.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                             C.c_void_p, C.c_void_p]
        _lib.oracle_max_threads.restype = C.c_int32
        _lib.oracle_set_threads.restype = None
        _lib.oracle_set_threads.argtypes = [C.c_int32]
        _lib.oracle_spectr_rho.restype = C.c_double
        _lib.oracle_spectr_rho.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32]
        _lib.oracle_verify_otlp.restype = C.c_int32
        _lib.oracle_verify_otlp.argtypes = [C.POINTER(_In), C.c_int32] + [C.c_void_p] * 7
        _lib.oracle_acceptance.restype = C.c_int32
        _lib.oracle_acceptance.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
        _lib.oracle_divergences.restype = C.c_int32
        _lib.oracle_divergences.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        _lib.oracle_branching.restype = C.c_int32
        _lib.oracle_branching.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32,
                                          C.c_void_p]
        _lib.oracle_block_efficiency.restype = C.c_int32
        _lib.oracle_block_efficiency.argtypes = [C.POINTER(_In), C.c_int32] + [C.c_void_p] * 4
        _lib.oracle_node_analysis.restype = C.c_int32
        _lib.oracle_node_analysis.argtypes = [C.POINTER(_In)] + [C.c_void_p] * 3
        _lib.oracle_latency_model.restype = C.c_int32
        _lib.oracle_latency_model.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
                                              C.c_void_p]
        _lib.oracle_tps_estimate.restype = C.c_double
        _lib.oracle_tps_estimate.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32]
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def set_threads(n: int) -> None:
    """Threads the batch loops use from now on (timing only: results do not depend on it)."""
    lib().oracle_set_threads(int(n))


# ---------------------------------------------------------------------------------------------
# row-level entry points
# ---------------------------------------------------------------------------------------------
def row_probs(z, T=1.0, top_k=0, top_p=1.0):
    """Sampling distribution of one row.  Returns (probs float64[V], stats float64[8])."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    probs = np.empty_like(z)
    stats = np.empty(8, dtype=np.float64)
    rc = lib().oracle_row_probs(_ptr(z), z.size, float(T), int(top_k), float(top_p), _ptr(probs), _ptr(stats))
    if rc:
        raise ValueError(f"oracle_row_probs failed with {rc}")
    return probs, stats


def inverse_cdf(w, u):
    """Inverse-CDF draw.  Returns (token, margin)."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    m = C.c_double(0.0)
    t = lib().oracle_inverse_cdf(_ptr(w), w.size, float(u), C.byref(m))
    return int(t), float(m.value)


# ---------------------------------------------------------------------------------------------
# batched tree verification
# ---------------------------------------------------------------------------------------------
@dataclass
class TreeInputs:
    """Host-side inputs of one verification call (all numpy, C-contiguous).

    target_logits / draft_logits: [B,N,V] float32, or uint16 holding bf16 bit patterns.
    parent: [N] or [B,N] int32 (parent[0] = -1, parent[i] < i).  token: [B,N] int32.
    u_accept / u_bonus: [B,N] float32 in [0,1).
    """
    target_logits: np.ndarray
    draft_logits: np.ndarray
    parent: np.ndarray
    token: np.ndarray
    u_accept: np.ndarray
    u_bonus: np.ndarray
    temperature: float = 1.0
    top_k: int = 0
    top_p: float = 1.0
    temperature_per_seq: np.ndarray | None = None
    _keep: list = field(default_factory=list, repr=False)

    def as_struct(self) -> _In:
        tl, dl = self.target_logits, self.draft_logits
        assert tl.ndim == 3 and tl.shape == dl.shape and tl.dtype == dl.dtype
        assert tl.dtype in (np.float32, np.uint16), "logits must be float32 or uint16 (bf16 bits)"
        B, N, V = tl.shape
        arrs = dict(
            tl=np.ascontiguousarray(tl), dl=np.ascontiguousarray(dl),
            parent=np.ascontiguousarray(self.parent, dtype=np.int32),
            token=np.ascontiguousarray(self.token, dtype=np.int32),
            ua=np.ascontiguousarray(self.u_accept, dtype=np.float32),
            ub=np.ascontiguousarray(self.u_bonus, dtype=np.float32),
            tps=None if self.temperature_per_seq is None
            else np.ascontiguousarray(self.temperature_per_seq, dtype=np.float32),
        )
        assert arrs["token"].shape == (B, N) and arrs["ua"].shape == (B, N) and arrs["ub"].shape == (B, N)
        assert arrs["parent"].shape in ((N,), (B, N))
        self._keep = list(arrs.values())
        return _In(B, N, V, 0 if tl.dtype == np.float32 else 1, _ptr(arrs["tl"]), _ptr(arrs["dl"]),
                   N * V, V, _ptr(arrs["parent"]), 0 if arrs["parent"].ndim == 1 else N,
                   _ptr(arrs["token"]), float(self.temperature), int(self.top_k), float(self.top_p),
                   _ptr(arrs["tps"]), _ptr(arrs["ua"]), _ptr(arrs["ub"]))

    @property
    def shape(self):
        return self.target_logits.shape


@dataclass
class VerifyResult:
    accepted_node: np.ndarray   # [B] int32
    accept_len: np.ndarray      # [B] int32 (tau)
    out_tokens: np.ndarray      # [B,N] int32: path tokens, the bonus token, then -1
    bonus_token: np.ndarray     # [B] int32
    residual: np.ndarray | None  # [B,V] float64
    bonus_margin: np.ndarray    # [B] float64
    trace: list                 # per sequence: list of (node, threshold, accepted) in consumption order
    status: np.ndarray          # [B] int32


def _verify(fn, inp: TreeInputs, want_residual: bool) -> VerifyResult:
    B, N, V = inp.shape
    st = inp.as_struct()
    acc = np.empty(B, np.int32); alen = np.empty(B, np.int32)
    toks = np.empty((B, N), np.int32); bonus = np.empty(B, np.int32)
    res = np.empty((B, V), np.float64) if want_residual else None
    bm = np.zeros(B, np.float64)
    tn = np.zeros((B, N), np.int32); tt = np.zeros((B, N), np.float64); ta = np.zeros((B, N), np.int32)
    tl = np.zeros(B, np.int32); status = np.zeros(B, np.int32)
    out = _Out(_ptr(acc), _ptr(alen), _ptr(toks), _ptr(bonus), _ptr(res), _ptr(bm),
               _ptr(tn), _ptr(tt), _ptr(ta), _ptr(tl), _ptr(status))
    rc = fn(C.byref(st), C.byref(out))
    if rc:
        raise ValueError(f"oracle verify failed with {rc}")
    trace = [[(int(tn[b, i]), float(tt[b, i]), bool(ta[b, i])) for i in range(tl[b])] for b in range(B)]
    return VerifyResult(acc, alen, toks, bonus, res, bm, trace, status)


def verify_specinfer(inp: TreeInputs, want_residual: bool = False) -> VerifyResult:
    return _verify(lib().oracle_verify_specinfer, inp, want_residual)


def verify_traversal(inp: TreeInputs, want_residual: bool = False) -> VerifyResult:
    return _verify(lib().oracle_verify_traversal, inp, want_residual)


def specinfer_tables(inp: TreeInputs):
    """(ratio float64[B,N], next_child int32[B,N], bonus_all int32[B,N], status int32[B])."""
    B, N, _ = inp.shape
    st = inp.as_struct()
    ratio = np.zeros((B, N), np.float64); nxt = np.full((B, N), -1, np.int32)
    bonus = np.full((B, N), -1, np.int32); status = np.zeros(B, np.int32)
    rc = lib().oracle_specinfer_tables(C.byref(st), _ptr(ratio), _ptr(nxt), _ptr(bonus), _ptr(status))
    if rc:
        raise ValueError(f"oracle_specinfer_tables failed with {rc}")
    return ratio, nxt, bonus, status


def traversal_tables(inp: TreeInputs):
    """(w_in float64[B,N], w_fin float64[B,N], bonus_all int32[B,N], status int32[B])."""
    B, N, _ = inp.shape
    st = inp.as_struct()
    w_in = np.zeros((B, N), np.float64); w_fin = np.zeros((B, N), np.float64)
    bonus = np.full((B, N), -1, np.int32); status = np.zeros(B, np.int32)
    rc = lib().oracle_traversal_tables(C.byref(st), _ptr(w_in), _ptr(w_fin), _ptr(bonus), _ptr(status))
    if rc:
        raise ValueError(f"oracle_traversal_tables failed with {rc}")
    return w_in, w_fin, bonus, status


def tree_probs(inp: TreeInputs, which: int, want_probs: bool = True):
    """(probs float64[B,N,V] or None, stats float64[B,N,8], status int32[B]) for target (0) / draft (1)."""
    B, N, V = inp.shape
    st = inp.as_struct()
    probs = np.empty((B, N, V), np.float64) if want_probs else None
    stats = np.zeros((B, N, 8), np.float64); status = np.zeros(B, np.int32)
    rc = lib().oracle_tree_probs(C.byref(st), int(which), _ptr(probs), _ptr(stats), _ptr(status))
    if rc:
        raise ValueError(f"oracle_tree_probs failed with {rc}")
    return probs, stats, status


def sample_bonus(weights, u):
    """Batched inverse CDF over float32 rows.  Returns (token int32[R], margin float64[R])."""
    w = np.ascontiguousarray(weights, dtype=np.float32)
    u = np.ascontiguousarray(u, dtype=np.float32)
    R, V = w.shape
    tok = np.empty(R, np.int32); mg = np.zeros(R, np.float64)
    rc = lib().oracle_sample_bonus(_ptr(w), R, V, _ptr(u), _ptr(tok), _ptr(mg))
    if rc:
        raise ValueError(f"oracle_sample_bonus failed with {rc}")
    return tok, mg


# ---------------------------------------------------------------------------------------------
# the other OTLP solvers and the offline analysis (otlp_oracle.c)
# ---------------------------------------------------------------------------------------------
SOLVERS = {"nss": 0, "naive": 1, "spectr": 2, "specinfer": 3, "specinfer_uniform": 4}


def spectr_rho(p, q, k: int) -> float:
    p = np.ascontiguousarray(p, np.float64); q = np.ascontiguousarray(q, np.float64)
    return float(lib().oracle_spectr_rho(_ptr(p), _ptr(q), p.size, int(k)))


@dataclass
class OtlpResult:
    accepted_node: np.ndarray
    accept_len: np.ndarray
    out_tokens: np.ndarray
    bonus_token: np.ndarray
    bonus_margin: np.ndarray    # CDF margin of the last residual draw (0: the last token was an accepted child)
    min_margin: np.ndarray      # smallest |u - threshold| over the acceptance tests made (1: none)
    status: np.ndarray


def verify_otlp(inp: TreeInputs, solver: str) -> OtlpResult:
    """Top-down verification with NSS / Naive / SpecTr (Algorithms 1-3)."""
    B, N, _ = inp.shape
    st = inp.as_struct()
    acc = np.empty(B, np.int32); alen = np.empty(B, np.int32); toks = np.empty((B, N), np.int32)
    bonus = np.empty(B, np.int32); bm = np.zeros(B, np.float64); mm = np.ones(B, np.float64)
    status = np.zeros(B, np.int32)
    rc = lib().oracle_verify_otlp(C.byref(st), SOLVERS[solver], _ptr(acc), _ptr(alen), _ptr(toks), _ptr(bonus),
                                  _ptr(bm), _ptr(mm), _ptr(status))
    if rc:
        raise ValueError(f"oracle_verify_otlp failed with {rc}")
    return OtlpResult(acc, alen, toks, bonus, bm, mm, status)


def acceptance(p, q, k: int):
    """Acceptance rates (Algorithms 6-9): [NSS, Naive, SpecTr, SpecInfer]."""
    p = np.ascontiguousarray(p, np.float64); q = np.ascontiguousarray(q, np.float64)
    out = np.empty(4, np.float64)
    rc = lib().oracle_acceptance(_ptr(p), _ptr(q), p.size, int(k), _ptr(out))
    if rc:
        raise ValueError(f"oracle_acceptance failed with {rc}")
    return out


def divergences(p, q):
    """[L1, KL(p||q), KL(q||p)] in nats."""
    p = np.ascontiguousarray(p, np.float64); q = np.ascontiguousarray(q, np.float64)
    out = np.empty(3, np.float64)
    rc = lib().oracle_divergences(_ptr(p), _ptr(q), p.size, _ptr(out))
    if rc:
        raise ValueError(f"oracle_divergences failed with {rc}")
    return out


def branching(solver: str, p, q, xs):
    """Branching probabilities B(f, xs, xs[i]) (Algorithms 11-14) for every child position."""
    p = np.ascontiguousarray(p, np.float64); q = np.ascontiguousarray(q, np.float64)
    x = np.ascontiguousarray(xs, np.int32)
    out = np.zeros(x.size, np.float64)
    rc = lib().oracle_branching(SOLVERS[solver], _ptr(p), _ptr(q), p.size, _ptr(x), x.size, _ptr(out))
    if rc:
        raise ValueError(f"oracle_branching failed with {rc}")
    return out


def block_efficiency(inp: TreeInputs, solver: str):
    """(E[tau+1 | tree] float64[B], node_reach [B,N], node_branch [B,N], status) -- equation (3)'s inner sum."""
    B, N, _ = inp.shape
    st = inp.as_struct()
    be = np.zeros(B, np.float64); reach = np.zeros((B, N), np.float64); br = np.zeros((B, N), np.float64)
    status = np.zeros(B, np.int32)
    rc = lib().oracle_block_efficiency(C.byref(st), SOLVERS[solver], _ptr(be), _ptr(reach), _ptr(br), _ptr(status))
    if rc:
        raise ValueError(f"oracle_block_efficiency failed with {rc}")
    return be, reach, br, status


def node_analysis(inp: TreeInputs):
    """(acceptance float64[B,N,4], divergences float64[B,N,3], status): NaN at childless nodes."""
    B, N, _ = inp.shape
    st = inp.as_struct()
    acc = np.zeros((B, N, 4), np.float64); dv = np.zeros((B, N, 3), np.float64); status = np.zeros(B, np.int32)
    rc = lib().oracle_node_analysis(C.byref(st), _ptr(acc), _ptr(dv), _ptr(status))
    if rc:
        raise ValueError(f"oracle_node_analysis failed with {rc}")
    return acc, dv, status


def latency_model(t_q, t_p, ctx: int, actions):
    """Equation (8): forward-pass time of every action (K, L1, L2) at context length ctx."""
    t_q = np.ascontiguousarray(t_q, np.float64); t_p = np.ascontiguousarray(t_p, np.float64)
    a = np.ascontiguousarray(actions, np.int32).reshape(-1, 3)
    out = np.zeros(a.shape[0], np.float64)
    rc = lib().oracle_latency_model(_ptr(t_q), _ptr(t_p), t_q.size, int(ctx), _ptr(a), a.shape[0], _ptr(out))
    if rc:
        raise ValueError(f"oracle_latency_model failed with {rc}")
    return out


def tps_estimate(pi, E, T_hat) -> float:
    pi = np.ascontiguousarray(pi, np.float64); E = np.ascontiguousarray(E, np.float64)
    T_hat = np.ascontiguousarray(T_hat, np.float64)
    return float(lib().oracle_tps_estimate(_ptr(pi), _ptr(E), _ptr(T_hat), pi.size))
