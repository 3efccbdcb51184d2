"""The allocation-free SpecInfer entry point against the ordinary one.

``spec_verify_specinfer_static`` serves callers that are not allowed to allocate device memory (a
plugin inside a server that owns the memory pool, a decoding loop in which an allocation would
stall): its scratch is an array inside the library instead of a caller-supplied workspace.  It must
give what ``spec_verify_specinfer`` gives.  Two calls in a row are checked because the second one
finds the first one's records still in the array.  This file sorts last on purpose, so that a run
that stops at the first failure has already run every other test; it also passes on its own in a
fresh process.
"""
import numpy as np
import pytest
import torch

from paper_2602_16994_b200 import binding
from paper_2602_16994_b200.synth import Workload, make_batch

pytestmark = pytest.mark.gpu


def _outputs_equal(a, b):
    for name in ("accepted_node", "accept_len", "out_tokens", "bonus_token", "status"):
        np.testing.assert_array_equal(getattr(a, name).cpu().numpy(), getattr(b, name).cpu().numpy(), err_msg=name)


def test_static_scratch_matches_workspace_entry_point_twice():
    # the same integer outputs are required: decisions of this size sit far from any margin
    shapes = [Workload("na1", 6, 32000, "bf16", 4, 1, 3, 1.0), Workload("na2", 3, 128256, "bf16", 3, 2, 2, 0.8)]
    for call, w in enumerate(shapes):
        batch = make_batch(w, seed=20 + call, device="cuda")
        args = (batch.target_logits, batch.draft_logits, batch.parent, batch.token, batch.u_accept, batch.u_bonus)
        ref = binding.verify_specinfer(*args, temperature=w.temperature)
        out = binding.alloc_outputs(w.B, w.N, w.V, "cuda")          # the caller's buffers
        got = binding.verify_specinfer_static(*args, outputs=out, temperature=w.temperature)
        torch.cuda.synchronize()
        assert (ref.status.cpu().numpy() == 0).all()
        _outputs_equal(got, ref)


def test_static_scratch_rejects_shapes_beyond_its_limit():
    w = Workload("na_big", 256, 64, "f32", 1, 0, 16, 1.0)           # 256 * 17 = 4352 nodes > 4096
    batch = make_batch(w, seed=1, device="cuda")
    out = binding.alloc_outputs(w.B, w.N, w.V, "cuda")
    with pytest.raises(RuntimeError, match="SPEC_ERR_WORKSPACE"):
        binding.verify_specinfer_static(batch.target_logits, batch.draft_logits, batch.parent, batch.token,
                                        batch.u_accept, batch.u_bonus, outputs=out)
