"""The allocation-free SpecInfer entry point against the ordinary one and against the CPU oracle.

``spec_verify_specinfer_static`` serves callers that are not allowed to allocate device memory (a
plugin inside a server that owns the memory pool, a decoding loop in which an allocation would
stall): its scratch is an array inside the library instead of a caller-supplied workspace.  It must
give what ``spec_verify_specinfer`` gives.  Calls come in pairs and the second shape is smaller than
the first, because the second call finds the first one's records, published weights, arrival counters
and row lists still in the array: the every-node path (diagnostic outputs) and the top-k / top-p path
are the ones that depend on the call clearing what must start empty.  This file sorts last on
purpose, so that a run that stops at the first failure has already run every other test; it also
passes on its own in a fresh process.
"""
import numpy as np
import pytest
import torch

from paper_2602_16994_b200 import binding
from paper_2602_16994_b200.synth import Workload, make_batch
from tests.parity import PROB_TOL, compare_decisions, run_oracle

pytestmark = pytest.mark.gpu


def _outputs_equal(a, b, floats=()):
    for name in ("accepted_node", "accept_len", "out_tokens", "bonus_token", "status"):
        np.testing.assert_array_equal(getattr(a, name).cpu().numpy(), getattr(b, name).cpu().numpy(), err_msg=name)
    for name in floats:
        x, y = getattr(a, name).cpu().numpy(), getattr(b, name).cpu().numpy()
        assert np.allclose(x, y, atol=PROB_TOL, rtol=0, equal_nan=True), name


def _args(batch):
    return (batch.target_logits, batch.draft_logits, batch.parent, batch.token, batch.u_accept, batch.u_bonus)


def test_static_scratch_matches_workspace_entry_point_twice():
    # the same integer outputs are required: decisions of this size sit far from any margin
    shapes = [Workload("na1", 6, 32000, "bf16", 4, 1, 3, 1.0), Workload("na2", 3, 128256, "bf16", 3, 2, 2, 0.8)]
    for call, w in enumerate(shapes):
        batch = make_batch(w, seed=20 + call, device="cuda")
        ref = binding.verify_specinfer(*_args(batch), temperature=w.temperature)
        out = binding.alloc_outputs(w.B, w.N, w.V, "cuda")          # the caller's buffers
        got = binding.verify_specinfer_static(*_args(batch), outputs=out, temperature=w.temperature)
        torch.cuda.synchronize()
        assert (ref.status.cpu().numpy() == 0).all()
        _outputs_equal(got, ref)
        _, oref = run_oracle(batch, "specinfer")
        assert compare_decisions(oref, got, None).near_margin_mismatches == 0


@pytest.mark.parametrize("trunc", [dict(), dict(top_k=40), dict(top_p=0.9)], ids=["plain", "top_k", "top_p"])
def test_static_scratch_every_node_path_twice_and_allocates_nothing(trunc):
    """Diagnostic outputs send the call through the every-node kernel, whose published-weight slots and
    arrival counters live in the shared array; the second, smaller call must not see the first one's."""
    shapes = [Workload("nb1", 8, 32000, "bf16", 4, 1, 3, 1.0, temperature=0.7, **trunc),
              Workload("nb2", 3, 8192, "bf16", 2, 1, 2, 0.8, temperature=0.7, **trunc)]
    opts = dict(residual=True, node_thr=True, margin=True)
    batches = [make_batch(w, seed=30 + i, device="cuda") for i, w in enumerate(shapes)]
    refs = [binding.verify_specinfer(*_args(b), temperature=b.workload.temperature, top_k=b.workload.top_k,
                                     top_p=b.workload.top_p, **opts) for b in batches]
    outs = [binding.alloc_outputs(w.B, w.N, w.V, "cuda", **opts) for w in shapes]
    # first call on the device: looks up the array's address; from here on nothing may be allocated
    binding.verify_specinfer_static(*_args(batches[0]), outputs=outs[0], temperature=0.7,
                                    top_k=shapes[0].top_k, top_p=shapes[0].top_p)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    torch_alloc0 = torch.cuda.memory_stats()["allocation.all.allocated"]
    for b, w, out, ref in zip(batches, shapes, outs, refs):
        got = binding.verify_specinfer_static(*_args(b), outputs=out, temperature=w.temperature, top_k=w.top_k,
                                              top_p=w.top_p)
        torch.cuda.synchronize()
        assert (got.status.cpu().numpy() == 0).all()
        _outputs_equal(got, ref, floats=("residual", "node_thr", "margin"))
    assert torch.cuda.mem_get_info()[0] == free0, "device memory was allocated or freed by the calls"
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == torch_alloc0


def test_static_scratch_rejects_shapes_beyond_its_limit():
    w = Workload("na_big", 256, 64, "f32", 1, 0, 16, 1.0)           # 256 * 17 = 4352 nodes > 4096
    batch = make_batch(w, seed=1, device="cuda")
    out = binding.alloc_outputs(w.B, w.N, w.V, "cuda")
    with pytest.raises(RuntimeError, match="SPEC_ERR_WORKSPACE"):
        binding.verify_specinfer_static(*_args(batch), outputs=out)
