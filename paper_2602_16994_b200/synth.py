"""Seeded synthetic workloads: tree shapes, logits, draft tokens and uniforms.

This module only *makes inputs*.  It holds none of the verification arithmetic and imports neither
the CUDA binding nor the CPU checker, so both can be fed the very same arrays.

Recipe (per node, independent draws): ``z_q = 3*g`` and ``z_p = z_q + sigma(node)*h`` with
``g, h ~ N(0,1)`` in fp32, each rounded (nearest-even) to the workload's logit dtype.  Draft tokens
play the role of the draft model's samples: the token of a non-root node is drawn from its
parent's draft distribution (softmax of ``z_q / T`` with the workload's top-k / top-p) by inverse
CDF with a seeded uniform.  Acceptance and bonus uniforms are fp32 in [0, 1), one of each per node.

The shapes follow the paper's draft trees: a root-i.i.d. tree is the union of K i.i.d. length-L
paths (Section 3.2), a delayed tree is a length-L1 trunk followed by K i.i.d. length-L2 branches
(Definition 5.2).  Equal tokens under one parent stay separate nodes.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


# ---------------------------------------------------------------------------------------------
# tree shapes
# ---------------------------------------------------------------------------------------------
def root_iid_tree(K: int, L: int):
    """K chains of length L hanging off the root.  Returns (parent int32[N], depth int32[N])."""
    return delayed_tree(K, 0, L)


def delayed_tree(K: int, L1: int, L2: int):
    """Trunk of L1 nodes, then K chains of L2 nodes from the trunk's end (Definition 5.2).

    Node 0 is the root; parent[i] < i; the children of a node appear in increasing index order,
    which is the order the verifiers try them in.
    """
    parent, depth = [-1], [0]
    for i in range(L1):
        parent.append(i)
        depth.append(i + 1)
    branch = L1
    for _ in range(K if L2 > 0 else 0):
        prev = branch
        for j in range(L2):
            parent.append(prev)
            depth.append(L1 + j + 1)
            prev = len(parent) - 1
    return np.asarray(parent, np.int32), np.asarray(depth, np.int32)


def children_lists(parent):
    ch = [[] for _ in parent]
    for i, p in enumerate(parent):
        if p >= 0:
            ch[int(p)].append(i)
    return ch


# ---------------------------------------------------------------------------------------------
# workloads
# ---------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    V: int
    dtype: str            # "f32" or "bf16"
    K: int
    L1: int
    L2: int
    sigma0: float         # divergence at depth 0
    sigma_per_depth: float = 0.0
    temperature: float = 1.0
    top_k: int = 0
    top_p: float = 1.0
    algorithms: tuple = ("specinfer", "traversal")
    features: bool = False

    @property
    def tree(self):
        return delayed_tree(self.K, self.L1, self.L2)

    @property
    def N(self) -> int:
        return 1 + self.L1 + self.K * self.L2

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def logit_bytes(self) -> int:
        """Bytes of logits one verification call has to read once: a target row for every node
        plus a draft row for every node that has children."""
        parent, _ = self.tree
        internal = len(set(int(p) for p in parent[1:]))
        return self.B * (self.N + internal) * self.V * self.elem_bytes

    def draft_nodes(self) -> int:
        return self.B * (self.N - 1)


def _cfg4(d: int) -> Workload:
    return Workload(f"cfg4_gemma_delayed_d{d}", 16, 262144, "bf16", 4, d, 6 - d, 0.5, 0.25)


WORKLOADS = {
    "cfg1_tiny": Workload("cfg1_tiny", 1, 1000, "f32", 2, 0, 3, 1.0),
    "cfg2_llama3_b8": Workload("cfg2_llama3_b8", 8, 128256, "bf16", 4, 2, 4, 1.0),
    "cfg3_qwen_b32": Workload("cfg3_qwen_b32", 32, 151936, "bf16", 8, 0, 5, 0.7, temperature=0.6,
                              top_p=0.95, algorithms=("specinfer",)),
    **{f"cfg4_gemma_delayed_d{d}": _cfg4(d) for d in range(5)},
    "cfg5_serving_b128": Workload("cfg5_serving_b128", 128, 128256, "bf16", 8, 2, 6, 1.2,
                                  temperature=0.3, top_k=50, algorithms=("specinfer",), features=True),
}


def shrink(w: Workload, **kw) -> Workload:
    """A smaller relative of a workload (tests use it to get cases the CPU checker finishes fast)."""
    return replace(w, **kw)


# ---------------------------------------------------------------------------------------------
# tensors
# ---------------------------------------------------------------------------------------------
@dataclass
class TreeBatch:
    """One batch of inputs as torch tensors on one device.

    target_logits / draft_logits [B,N,V] (float32 or bfloat16); parent / depth [N] int32;
    token [B,N] int32 (token[:,0] = 0, unused); u_accept / u_bonus [B,N] float32.
    """
    workload: Workload
    target_logits: torch.Tensor
    draft_logits: torch.Tensor
    parent: torch.Tensor
    depth: torch.Tensor
    token: torch.Tensor
    u_accept: torch.Tensor
    u_bonus: torch.Tensor

    def to(self, device) -> "TreeBatch":
        f = lambda t: t.to(device)
        return TreeBatch(self.workload, f(self.target_logits), f(self.draft_logits), f(self.parent),
                         f(self.depth), f(self.token), f(self.u_accept), f(self.u_bonus))

    def select(self, idx) -> "TreeBatch":
        """The sub-batch made of the listed sequences (on the same device)."""
        idx = torch.as_tensor(idx, dtype=torch.long, device=self.token.device)
        g = lambda t: t.index_select(0, idx).contiguous()
        return TreeBatch(replace(self.workload, B=int(idx.numel())), g(self.target_logits),
                         g(self.draft_logits), self.parent, self.depth, g(self.token),
                         g(self.u_accept), g(self.u_bonus))

    def numpy(self) -> dict:
        """Host numpy views; bf16 logits come back as uint16 bit patterns."""
        def logits(t):
            t = t.detach().cpu().contiguous()
            if t.dtype == torch.bfloat16:
                return t.view(torch.int16).numpy().view(np.uint16)
            return t.numpy()
        g = lambda t: t.detach().cpu().contiguous().numpy()
        return dict(target_logits=logits(self.target_logits), draft_logits=logits(self.draft_logits),
                    parent=g(self.parent), depth=g(self.depth), token=g(self.token),
                    u_accept=g(self.u_accept), u_bonus=g(self.u_bonus))


def _draft_distribution(zq: torch.Tensor, T: float, top_k: int, top_p: float) -> torch.Tensor:
    """The draft model's sampling distribution for rows of logits (plain sort-based truncation)."""
    work = torch.float64 if zq.device.type == "cpu" else torch.float32
    q = torch.softmax(zq.to(work) / T, dim=-1)
    V = q.shape[-1]
    if 0 < top_k < V:
        kth = torch.topk(q, top_k, dim=-1).values[..., -1:]
        q = torch.where(q >= kth, q, torch.zeros_like(q))
        q = q / q.sum(-1, keepdim=True)
    if top_p < 1.0:
        sq, order = torch.sort(q, dim=-1, descending=True)
        before = torch.cumsum(sq, -1) - sq
        keep_sorted = before < top_p
        keep = torch.zeros_like(keep_sorted).scatter(-1, order, keep_sorted)
        q = torch.where(keep, q, torch.zeros_like(q))
        q = q / q.sum(-1, keepdim=True)
    return q


def make_batch(w: Workload, seed: int = 0, device="cpu", seq_chunk: int = 8) -> TreeBatch:
    """Build one seeded batch of the workload on ``device`` (generated there, chunked by sequence)."""
    device = torch.device(device)
    parent_np, depth_np = w.tree
    N, V, B = w.N, w.V, w.B
    gen = torch.Generator(device=device)
    # python's str hash is salted per process: derive the workload term from the name's bytes
    name_key = int.from_bytes(w.name.encode()[:8].ljust(8, b"\0"), "little") % 999_983
    gen.manual_seed(1_000_003 * int(seed) + name_key)
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    zp = torch.empty((B, N, V), dtype=tdt, device=device)
    zq = torch.empty((B, N, V), dtype=tdt, device=device)
    sigma = torch.tensor([w.sigma0 + w.sigma_per_depth * float(d) for d in depth_np],
                         dtype=torch.float32, device=device).view(1, N, 1)
    token = torch.zeros((B, N), dtype=torch.int32, device=device)
    u_draft = torch.rand((B, N), generator=gen, dtype=torch.float32, device=device)
    u_accept = torch.rand((B, N), generator=gen, dtype=torch.float32, device=device)
    u_bonus = torch.rand((B, N), generator=gen, dtype=torch.float32, device=device)
    par = torch.as_tensor(parent_np, device=device).long()
    for b0 in range(0, B, seq_chunk):
        b1 = min(B, b0 + seq_chunk)
        g = torch.randn((b1 - b0, N, V), generator=gen, dtype=torch.float32, device=device)
        h = torch.randn((b1 - b0, N, V), generator=gen, dtype=torch.float32, device=device)
        zq32 = 3.0 * g
        zp32 = zq32 + sigma * h
        zq[b0:b1] = zq32.to(tdt)
        zp[b0:b1] = zp32.to(tdt)
        del g, h, zq32, zp32
        if N > 1:
            # token of node c ~ q(. | parent(c)), from the rounded draft logits the verifiers will see
            rows = zq[b0:b1].index_select(1, par[1:])                      # [b, N-1, V]
            q = _draft_distribution(rows, w.temperature, w.top_k, w.top_p)
            cdf = torch.cumsum(q, -1)
            target = (u_draft[b0:b1, 1:].to(cdf.dtype) * cdf[..., -1]).unsqueeze(-1)
            tok = torch.searchsorted(cdf, target, right=True).squeeze(-1).clamp_(max=V - 1)
            token[b0:b1, 1:] = tok.to(torch.int32)
            del rows, q, cdf
    return TreeBatch(w, zp, zq, torch.as_tensor(parent_np, device=device),
                     torch.as_tensor(depth_np, device=device), token, u_accept, u_bonus)
