"""Thin ctypes binding of libspecverify.so: argument marshalling only.

Every step of the verification path runs inside the CUDA library; this module turns torch tensors
into the plain pointers of the C ABI (``include/specverify.h``), owns the scratch workspace and
allocates output tensors.  There is no CPU fallback: a missing library or a missing CUDA device
raises ``RuntimeError``.

Device-resident API (inputs already in HBM, nothing is synchronised):
    verify_specinfer / verify_traversal / tree_probs / sample_bonus
Host API (pinned host buffers in, host results out; copies and one stream sync inside):
    HostVerifier
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspecverify.so")

SPEC_F32, SPEC_BF16 = 0, 1
ERRORS = {0: "SPEC_OK", -1: "SPEC_ERR_NULL", -2: "SPEC_ERR_SHAPE", -3: "SPEC_ERR_DTYPE",
          -4: "SPEC_ERR_PARAM", -5: "SPEC_ERR_WORKSPACE", -6: "SPEC_ERR_UNSUPPORTED", -7: "SPEC_ERR_CUDA"}
EXPORTS = ("spec_workspace_bytes", "spec_tree_probs", "spec_verify_specinfer", "spec_verify_traversal",
           "spec_sample_bonus", "spec_query_plan", "spec_host_staging_bytes", "spec_verify_host",
           "spec_verify_specinfer_static", "spec_kernel_launches", "spec_analysis_workspace_bytes",
           "spec_tree_analysis", "spec_latency_model", "spec_test_hooks", "spec_row_statistics",
           "spec_verify_otlp")


class SpecIn(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("N", C.c_int32), ("V", C.c_int32), ("logits_dtype", C.c_int32),
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
        ("seq_stride", C.c_int64), ("node_stride", C.c_int64),
        ("parent", C.c_void_p), ("topo_seq_stride", C.c_int64), ("token", C.c_void_p),
        ("temperature", C.c_float), ("top_k", C.c_int32), ("top_p", C.c_float),
        ("temperature_per_seq", C.c_void_p), ("u_accept", C.c_void_p), ("u_bonus", C.c_void_p),
    ]


class SpecOut(C.Structure):
    _fields_ = [
        ("accepted_node", C.c_void_p), ("accept_len", C.c_void_p), ("out_tokens", C.c_void_p),
        ("bonus_token", C.c_void_p), ("status", C.c_void_p), ("residual", C.c_void_p),
        ("node_thr", C.c_void_p), ("node_w_in", C.c_void_p), ("node_features", C.c_void_p),
        ("margin", C.c_void_p),
    ]


class SpecAnalysisOut(C.Structure):
    _fields_ = [("acceptance", C.c_void_p), ("divergence", C.c_void_p), ("branch", C.c_void_p),
                ("reach", C.c_void_p), ("block_eff", C.c_void_p)]


SOLVERS = ("nss", "naive", "spectr", "specinfer", "specinfer_uniform")     # order of the `branch` outputs

_lib = None


def load_library(path: str = LIB_PATH):
    """dlopen the CUDA library (no device needed for this step) and declare the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2602_16994_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(path)
    lib.spec_workspace_bytes.restype = C.c_int32
    lib.spec_workspace_bytes.argtypes = [C.POINTER(SpecIn), C.POINTER(C.c_int64)]
    lib.spec_tree_probs.restype = C.c_int32
    lib.spec_tree_probs.argtypes = [C.POINTER(SpecIn), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_int64, C.c_void_p]
    for name in ("spec_verify_specinfer", "spec_verify_traversal"):
        f = getattr(lib, name)
        f.restype = C.c_int32
        f.argtypes = [C.POINTER(SpecIn), C.POINTER(SpecOut), C.c_void_p, C.c_int64, C.c_void_p]
    lib.spec_verify_specinfer_static.restype = C.c_int32
    lib.spec_verify_specinfer_static.argtypes = [C.POINTER(SpecIn), C.POINTER(SpecOut), C.c_void_p]
    lib.spec_sample_bonus.restype = C.c_int32
    lib.spec_sample_bonus.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_int64, C.c_void_p]
    lib.spec_query_plan.restype = C.c_int32
    lib.spec_query_plan.argtypes = [C.c_int32, C.c_int32] + [C.POINTER(C.c_int32)] * 4
    lib.spec_kernel_launches.restype = C.c_int64
    lib.spec_kernel_launches.argtypes = []
    lib.spec_host_staging_bytes.restype = C.c_int32
    lib.spec_host_staging_bytes.argtypes = [C.POINTER(SpecIn), C.POINTER(C.c_int64)]
    lib.spec_verify_host.restype = C.c_int32
    lib.spec_verify_host.argtypes = [C.POINTER(SpecIn), C.POINTER(SpecOut), C.c_int32, C.c_void_p, C.c_int64,
                                     C.c_void_p]
    lib.spec_analysis_workspace_bytes.restype = C.c_int32
    lib.spec_analysis_workspace_bytes.argtypes = [C.POINTER(SpecIn), C.POINTER(C.c_int64)]
    lib.spec_tree_analysis.restype = C.c_int32
    lib.spec_tree_analysis.argtypes = [C.POINTER(SpecIn), C.POINTER(SpecAnalysisOut), C.c_void_p, C.c_int64, C.c_void_p]
    lib.spec_latency_model.restype = C.c_int32
    lib.spec_latency_model.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                       C.c_void_p]
    lib.spec_verify_otlp.restype = C.c_int32
    lib.spec_verify_otlp.argtypes = [C.POINTER(SpecIn), C.POINTER(SpecOut), C.c_int32, C.c_void_p, C.c_int64, C.c_void_p]
    lib.spec_row_statistics.restype = C.c_int32
    lib.spec_row_statistics.argtypes = [C.POINTER(SpecIn), C.c_void_p, C.c_int64, C.c_void_p]
    lib.spec_test_hooks.restype = C.c_int32
    lib.spec_test_hooks.argtypes = [C.c_int64, C.c_int32]
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"{what} failed: {ERRORS.get(rc, rc)}")


def _require_cuda(t: torch.Tensor, name: str):
    if not t.is_cuda:
        raise RuntimeError(f"{name} must live on a CUDA device (there is no CPU path)")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def set_test_hooks(wait_cycles: int = 0, hold_slot: int = -1):
    """Test hooks: limit of the on-device waits in clock cycles (0: default) and one Traversal weight slot
    (index b * N + node) that is left pending (-1: none)."""
    _check(load_library().spec_test_hooks(int(wait_cycles), int(hold_slot)), "spec_test_hooks")


def kernel_launches() -> int:
    """Kernels the library has enqueued in this process so far."""
    return int(load_library().spec_kernel_launches())


def query_plan(V: int, dtype: int = SPEC_BF16) -> dict:
    lib = load_library()
    c, sl, sm, nt = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
    _check(lib.spec_query_plan(V, dtype, C.byref(c), C.byref(sl), C.byref(sm), C.byref(nt)), "spec_query_plan")
    return dict(cluster_size=c.value, slice_len=sl.value, smem_bytes=sm.value, threads=nt.value)


def make_spec_in(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature=1.0,
                 top_k=0, top_p=1.0, temperature_per_seq=None) -> SpecIn:
    """Marshal tensors into a SpecIn.  Logits: [B,N,V] float32 or bfloat16, last dim contiguous."""
    for name, t in (("target_logits", target_logits), ("draft_logits", draft_logits), ("parent", parent),
                    ("token", token), ("u_accept", u_accept), ("u_bonus", u_bonus)):
        _require_cuda(t, name)
    if target_logits.dtype not in (torch.float32, torch.bfloat16) or draft_logits.dtype != target_logits.dtype:
        raise RuntimeError("logits must both be float32 or both bfloat16")
    if target_logits.dim() != 3 or target_logits.stride(2) != 1 or draft_logits.stride() != target_logits.stride():
        raise RuntimeError("logits must be [B,N,V] with a contiguous vocabulary axis and equal strides")
    B, N, V = target_logits.shape
    for name, t, dt in (("parent", parent, torch.int32), ("token", token, torch.int32),
                        ("u_accept", u_accept, torch.float32), ("u_bonus", u_bonus, torch.float32)):
        if t.dtype != dt or not t.is_contiguous():
            raise RuntimeError(f"{name} must be a contiguous {dt} tensor")
    if tuple(token.shape) != (B, N) or tuple(u_accept.shape) != (B, N) or tuple(u_bonus.shape) != (B, N):
        raise RuntimeError("token, u_accept and u_bonus must be [B,N]")
    if tuple(parent.shape) not in ((N,), (B, N)):
        raise RuntimeError("parent must be [N] or [B,N]")
    return SpecIn(B, N, V, SPEC_F32 if target_logits.dtype == torch.float32 else SPEC_BF16,
                  _ptr(target_logits), _ptr(draft_logits), target_logits.stride(0), target_logits.stride(1),
                  _ptr(parent), 0 if parent.dim() == 1 else N, _ptr(token), float(temperature), int(top_k),
                  float(top_p), _ptr(temperature_per_seq), _ptr(u_accept), _ptr(u_bonus))


def workspace_bytes(spec_in: SpecIn) -> int:
    n = C.c_int64()
    _check(load_library().spec_workspace_bytes(C.byref(spec_in), C.byref(n)), "spec_workspace_bytes")
    return int(n.value)


@dataclass
class VerifyOutputs:
    accepted_node: torch.Tensor
    accept_len: torch.Tensor
    out_tokens: torch.Tensor
    bonus_token: torch.Tensor
    status: torch.Tensor
    residual: torch.Tensor | None = None
    node_thr: torch.Tensor | None = None
    node_w_in: torch.Tensor | None = None
    node_features: torch.Tensor | None = None
    margin: torch.Tensor | None = None

    def as_struct(self) -> SpecOut:
        return SpecOut(_ptr(self.accepted_node), _ptr(self.accept_len), _ptr(self.out_tokens),
                       _ptr(self.bonus_token), _ptr(self.status), _ptr(self.residual), _ptr(self.node_thr),
                       _ptr(self.node_w_in), _ptr(self.node_features), _ptr(self.margin))


def alloc_outputs(B, N, V, device, residual=False, node_thr=False, node_w_in=False, features=False,
                  margin=False) -> VerifyOutputs:
    i32 = dict(dtype=torch.int32, device=device)
    f32 = dict(dtype=torch.float32, device=device)
    return VerifyOutputs(
        torch.empty(B, **i32), torch.empty(B, **i32), torch.empty((B, N), **i32), torch.empty(B, **i32),
        torch.empty(B, **i32),
        torch.empty((B, V), **f32) if residual else None,
        torch.empty((B, N), **f32) if node_thr else None,
        torch.empty((B, N), **f32) if node_w_in else None,
        torch.empty((B, N, 4), **f32) if features else None,
        torch.empty((B, N + 1), **f32) if margin else None)


class Workspace:
    """Scratch memory for the verify calls; grows on demand, one per stream of concurrent calls."""

    def __init__(self, device):
        self.device = device
        self.buf = None

    def get(self, nbytes: int):
        if self.buf is None or self.buf.numel() < nbytes + 256:
            self.buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.buf.data_ptr()
        off = (-base) % 256
        return C.c_void_p(base + off), self.buf.numel() - off


_default_ws = {}


def _ws_for(device) -> Workspace:
    key = str(device)
    if key not in _default_ws:
        _default_ws[key] = Workspace(device)
    return _default_ws[key]


def _verify(fn_name, batch_or_in, outputs, workspace, stream, **alloc):
    lib = load_library()
    if not torch.cuda.is_available():
        raise RuntimeError("no CUDA device: the verification path has no CPU fallback")
    spec_in, keep = batch_or_in
    B, N, V = spec_in.B, spec_in.N, spec_in.V
    device = keep[0].device
    if outputs is None:
        outputs = alloc_outputs(B, N, V, device, **alloc)
    ws = workspace or _ws_for(device)
    ptr, size = ws.get(workspace_bytes(spec_in))
    so = outputs.as_struct()
    _check(getattr(lib, fn_name)(C.byref(spec_in), C.byref(so), ptr, size, _stream_ptr(stream)), fn_name)
    return outputs


def _marshal(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature, top_k, top_p,
             temperature_per_seq):
    si = make_spec_in(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature, top_k,
                      top_p, temperature_per_seq)
    return si, (target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature_per_seq)


def verify_specinfer(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature=1.0,
                     top_k=0, top_p=1.0, temperature_per_seq=None, outputs=None, workspace=None,
                     stream=None, residual=False, node_thr=False, features=False, margin=False):
    """SpecInfer verification of a batch of draft trees (enqueued on the stream; returns device tensors)."""
    m = _marshal(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature, top_k, top_p,
                 temperature_per_seq)
    return _verify("spec_verify_specinfer", m, outputs, workspace, stream, residual=residual,
                   node_thr=node_thr, features=features, margin=margin)


OTLP_SOLVERS = {"nss": 0, "naive": 1, "spectr": 2}


def verify_otlp(solver, target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature=1.0, top_k=0,
                top_p=1.0, temperature_per_seq=None, outputs=None, workspace=None, stream=None):
    """Top-down verification with NSS, NaiveTree or SpecTr (``solver``: "nss", "naive", "spectr")."""
    lib = load_library()
    if not torch.cuda.is_available():
        raise RuntimeError("no CUDA device: the verification path has no CPU fallback")
    spec_in, keep = _marshal(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature, top_k, top_p,
                             temperature_per_seq)
    device = target_logits.device
    if outputs is None:
        outputs = alloc_outputs(spec_in.B, spec_in.N, spec_in.V, device)
    ws = workspace or _ws_for(device)
    ptr, size = ws.get(workspace_bytes(spec_in))
    so = outputs.as_struct()
    _check(lib.spec_verify_otlp(C.byref(spec_in), C.byref(so), OTLP_SOLVERS[solver], ptr, size, _stream_ptr(stream)),
           "spec_verify_otlp")
    return outputs


def verify_specinfer_static(target_logits, draft_logits, parent, token, u_accept, u_bonus, outputs,
                            temperature=1.0, top_k=0, top_p=1.0, stream=None):
    """SpecInfer verification through ``spec_verify_specinfer_static``: the library's built-in scratch
    array is used, so neither this wrapper nor the library allocates anything.  The caller owns every
    buffer, ``outputs`` (a ``VerifyOutputs``) included.  Only for B * N up to 4096 nodes; calls that may
    overlap on the GPU must not share this entry point.  Make the first call on a device outside any
    stream capture.
    """
    lib = load_library()
    if not torch.cuda.is_available():
        raise RuntimeError("no CUDA device: the verification path has no CPU fallback")
    si, keep = _marshal(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature, top_k, top_p,
                        None)
    so = outputs.as_struct()
    _check(lib.spec_verify_specinfer_static(C.byref(si), C.byref(so), _stream_ptr(stream)),
           "spec_verify_specinfer_static")
    return outputs


def verify_traversal(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature=1.0,
                     top_k=0, top_p=1.0, temperature_per_seq=None, outputs=None, workspace=None,
                     stream=None, residual=False, node_thr=False, node_w_in=False, features=False,
                     margin=False):
    """Traversal Verification of a batch of draft trees."""
    m = _marshal(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature, top_k, top_p,
                 temperature_per_seq)
    return _verify("spec_verify_traversal", m, outputs, workspace, stream, residual=residual,
                   node_thr=node_thr, node_w_in=node_w_in, features=features, margin=margin)


class PreparedVerify:
    """One verification call with its arguments marshalled once: ``launch()`` is a single C call.

    For loops that verify the same buffers again and again (a decoding loop reusing its logits
    buffers, a benchmark).  The tensors are kept alive by this object.  ``launch`` may be recorded
    into a CUDA graph after one ordinary call on the device (the first call sets kernel attributes).
    """

    def __init__(self, algorithm, target_logits, draft_logits, parent, token, u_accept, u_bonus,
                 temperature=1.0, top_k=0, top_p=1.0, temperature_per_seq=None, outputs=None, workspace=None,
                 **alloc):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the verification path has no CPU fallback")
        self.fn = getattr(self.lib, {"specinfer": "spec_verify_specinfer",
                                     "traversal": "spec_verify_traversal"}[algorithm])
        self.name = algorithm
        self.spec_in, self.keep = _marshal(target_logits, draft_logits, parent, token, u_accept, u_bonus,
                                           temperature, top_k, top_p, temperature_per_seq)
        B, N, V = self.spec_in.B, self.spec_in.N, self.spec_in.V
        dev = target_logits.device
        self.outputs = outputs if outputs is not None else alloc_outputs(B, N, V, dev, **alloc)
        self.spec_out = self.outputs.as_struct()
        self.workspace = workspace or _ws_for(dev)
        self.ws_ptr, self.ws_size = self.workspace.get(workspace_bytes(self.spec_in))
        self._in_ref, self._out_ref = C.byref(self.spec_in), C.byref(self.spec_out)

    def launch(self, stream=None):
        rc = self.fn(self._in_ref, self._out_ref, self.ws_ptr, self.ws_size, _stream_ptr(stream))
        if rc != 0:
            _check(rc, "spec_verify_" + self.name)
        return self.outputs

    def launch_statistics_only(self, stream=None):
        """Only the row statistics pass of the call (``spec_row_statistics``), for timing it by itself."""
        _check(self.lib.spec_row_statistics(self._in_ref, self.ws_ptr, self.ws_size, _stream_ptr(stream)),
               "spec_row_statistics")


@dataclass
class AnalysisOutputs:
    acceptance: torch.Tensor     # [B,N,4]: NSS, Naive, SpecTr, SpecInfer
    divergence: torch.Tensor     # [B,N,3]: L1, KL(p||q), KL(q||p)
    branch: torch.Tensor         # [5,B,N], order of SOLVERS
    reach: torch.Tensor          # [5,B,N]
    block_eff: torch.Tensor      # [5,B]


def tree_analysis(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature=1.0, top_k=0,
                  top_p=1.0, temperature_per_seq=None, stream=None) -> AnalysisOutputs:
    """Acceptance rates, divergences, branching probabilities and block efficiency of a batch of trees."""
    lib = load_library()
    si, keep = _marshal(target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature, top_k, top_p,
                        temperature_per_seq)
    B, N = si.B, si.N
    dev = target_logits.device
    f32 = dict(dtype=torch.float32, device=dev)
    out = AnalysisOutputs(torch.empty((B, N, 4), **f32), torch.empty((B, N, 3), **f32), torch.empty((5, B, N), **f32),
                          torch.empty((5, B, N), **f32), torch.empty((5, B), **f32))
    n = C.c_int64()
    _check(lib.spec_analysis_workspace_bytes(C.byref(si), C.byref(n)), "spec_analysis_workspace_bytes")
    ptr, size = _ws_for(dev).get(int(n.value))
    so = SpecAnalysisOut(_ptr(out.acceptance), _ptr(out.divergence), _ptr(out.branch), _ptr(out.reach),
                         _ptr(out.block_eff))
    _check(lib.spec_tree_analysis(C.byref(si), C.byref(so), ptr, size, _stream_ptr(stream)), "spec_tree_analysis")
    return out


def latency_model(t_q, t_p, ctx, actions, stream=None):
    """Equation (8): forward-pass time of every action (K, L1, L2) at context length ``ctx`` (device tensors:
    t_q / t_p float64 [n_len], actions int32 [A,3]); returns float64 [A]."""
    lib = load_library()
    for name, t, dt in (("t_q", t_q, torch.float64), ("t_p", t_p, torch.float64), ("actions", actions, torch.int32)):
        _require_cuda(t, name)
        if t.dtype != dt or not t.is_contiguous():
            raise RuntimeError(f"{name} must be a contiguous {dt} tensor")
    if t_q.numel() != t_p.numel() or actions.dim() != 2 or actions.shape[1] != 3:
        raise RuntimeError("t_q and t_p must have the same length, actions must be [A,3]")
    out = torch.empty(actions.shape[0], dtype=torch.float64, device=t_q.device)
    _check(lib.spec_latency_model(_ptr(t_q), _ptr(t_p), t_q.numel(), int(ctx), _ptr(actions), actions.shape[0],
                                  _ptr(out), _stream_ptr(stream)), "spec_latency_model")
    return out


def tree_probs(logits, which=0, temperature=1.0, top_k=0, top_p=1.0, temperature_per_seq=None,
               want_probs=True, want_stats=True, stream=None):
    """Sampling distribution of every row of ``logits`` [B,N,V].  Returns (probs or None, stats or None)."""
    lib = load_library()
    _require_cuda(logits, "logits")
    if logits.dim() != 3 or logits.stride(2) != 1 or logits.dtype not in (torch.float32, torch.bfloat16):
        raise RuntimeError("logits must be [B,N,V] float32 / bfloat16 with a contiguous vocabulary axis")
    B, N, V = logits.shape
    si = SpecIn(B, N, V, SPEC_F32 if logits.dtype == torch.float32 else SPEC_BF16,
                _ptr(logits), _ptr(logits), logits.stride(0), logits.stride(1), None, 0, None,
                float(temperature), int(top_k), float(top_p), _ptr(temperature_per_seq), None, None)
    probs = torch.empty((B, N, V), dtype=torch.float32, device=logits.device) if want_probs else None
    stats = torch.empty((B, N, 6), dtype=torch.float32, device=logits.device) if want_stats else None
    ws_ptr, ws_size = _ws_for(logits.device).get(workspace_bytes(si))       # holds the row cuts when truncating
    _check(lib.spec_tree_probs(C.byref(si), int(which), _ptr(probs), _ptr(stats), ws_ptr, ws_size,
                               _stream_ptr(stream)), "spec_tree_probs")
    return probs, stats


def sample_bonus(weights, u, want_margin=False, stream=None):
    """Inverse-CDF draw from each row of ``weights`` [R,V] float32 with uniforms ``u`` [R]."""
    lib = load_library()
    _require_cuda(weights, "weights")
    _require_cuda(u, "u")
    if weights.dtype != torch.float32 or not weights.is_contiguous() or weights.dim() != 2:
        raise RuntimeError("weights must be a contiguous [R,V] float32 tensor")
    if u.dtype != torch.float32 or not u.is_contiguous() or u.numel() != weights.shape[0]:
        raise RuntimeError("u must be a contiguous float32 tensor with one entry per row")
    R, V = weights.shape
    token = torch.empty(R, dtype=torch.int32, device=weights.device)
    margin = torch.empty(R, dtype=torch.float32, device=weights.device) if want_margin else None
    _check(lib.spec_sample_bonus(_ptr(weights), R, V, _ptr(u), _ptr(token), _ptr(margin), None, 0,
                                 _stream_ptr(stream)), "spec_sample_bonus")
    return (token, margin) if want_margin else token


class HostVerifier:
    """End-to-end call for callers whose logits live in host memory (``spec_verify_host``).

    Owns the device staging buffer for one batch shape and pinned host result arrays.  ``run`` hands
    host pointers to the library, which copies the inputs host->device, runs the verifier, copies the
    decisions device->host and synchronises the stream before returning.
    """

    ALGORITHMS = {"specinfer": 0, "traversal": 1}

    def __init__(self, B, N, V, logits_dtype=torch.bfloat16, device="cuda", algorithm="specinfer",
                 per_sequence_topology=False):
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the verification path has no CPU fallback")
        self.lib = load_library()
        self.device = torch.device(device)
        self.algorithm = self.ALGORITHMS[algorithm]
        self.shape = (B, N, V)
        self.dtype = logits_dtype
        self.per_seq = per_sequence_topology
        probe = SpecIn(B, N, V, SPEC_F32 if logits_dtype == torch.float32 else SPEC_BF16, None, None, N * V, V,
                       None, N if per_sequence_topology else 0, None, 1.0, 0, 1.0, None, None, None)
        n = C.c_int64()
        _check(self.lib.spec_host_staging_bytes(C.byref(probe), C.byref(n)), "spec_host_staging_bytes")
        self.staging = torch.empty(int(n.value) + 256, dtype=torch.uint8, device=self.device)
        self.host_out = {k: torch.empty(shape, dtype=torch.int32).pin_memory()
                         for k, shape in (("accepted_node", (B,)), ("accept_len", (B,)), ("out_tokens", (B, N)),
                                          ("bonus_token", (B,)), ("status", (B,)))}
        self.stream = torch.cuda.Stream(device=self.device)

    def h2d_bytes(self) -> int:
        B, N, V = self.shape
        esz = 4 if self.dtype == torch.float32 else 2
        return 2 * B * N * V * esz + (B if self.per_seq else 1) * N * 4 + 3 * B * N * 4

    def d2h_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.host_out.values())

    def run(self, target_logits, draft_logits, parent, token, u_accept, u_bonus, temperature=1.0, top_k=0,
            top_p=1.0):
        """All arguments are host tensors (pinned for asynchronous copies).  Returns pinned host results."""
        B, N, V = self.shape
        for name, t in (("target_logits", target_logits), ("draft_logits", draft_logits), ("parent", parent),
                        ("token", token), ("u_accept", u_accept), ("u_bonus", u_bonus)):
            if t.is_cuda or not t.is_contiguous():
                raise RuntimeError(f"{name} must be a contiguous host tensor")
        if tuple(target_logits.shape) != (B, N, V) or target_logits.dtype != self.dtype:
            raise RuntimeError("logits do not match the shape / dtype this verifier was built for")
        si = SpecIn(B, N, V, SPEC_F32 if self.dtype == torch.float32 else SPEC_BF16, _ptr(target_logits),
                    _ptr(draft_logits), N * V, V, _ptr(parent), N if parent.dim() == 2 else 0, _ptr(token),
                    float(temperature), int(top_k), float(top_p), None, _ptr(u_accept), _ptr(u_bonus))
        h = self.host_out
        so = SpecOut(_ptr(h["accepted_node"]), _ptr(h["accept_len"]), _ptr(h["out_tokens"]), _ptr(h["bonus_token"]),
                     _ptr(h["status"]), None, None, None, None, None)
        base = self.staging.data_ptr()
        off = (-base) % 256
        _check(self.lib.spec_verify_host(C.byref(si), C.byref(so), self.algorithm, C.c_void_p(base + off),
                                         self.staging.numel() - off, C.c_void_p(self.stream.cuda_stream)),
               "spec_verify_host")
        return h
