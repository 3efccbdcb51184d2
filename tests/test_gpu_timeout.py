"""The bounded waits of the kernels, watched running out -- on the allowed form only: a flag that nothing
sets and a short limit.  One Traversal weight slot is left pending through the library's test hook and
the wait limit is cut to about a millisecond; the call must return, the sequence must report
SPEC_DEV_TIMEOUT, nothing may hang or trap, and the next ordinary call must be right again."""
import numpy as np
import pytest
import torch

from paper_2602_16994_b200 import binding
from paper_2602_16994_b200.synth import Workload, make_batch
from tests.parity import compare_decisions, run_oracle

pytestmark = pytest.mark.gpu
SPEC_DEV_TIMEOUT = 4


def test_a_wait_that_runs_out_is_reported_and_the_library_stays_usable():
    w = Workload("to", 3, 32000, "bf16", 1, 0, 4, 1.0)        # one path of four nodes under the root
    batch = make_batch(w, seed=11, device="cuda")
    args = (batch.target_logits, batch.draft_logits, batch.parent, batch.token, batch.u_accept, batch.u_bonus)
    _, ref = run_oracle(batch, "traversal")
    ok = binding.verify_traversal(*args)
    torch.cuda.synchronize()
    assert (ok.status.cpu().numpy() == 0).all()
    try:
        # node 2 of sequence 1 never gets its weight; every wait gives up after 2e6 cycles (about 1 ms)
        binding.set_test_hooks(wait_cycles=2_000_000, hold_slot=1 * w.N + 2)
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        got = binding.verify_traversal(*args)
        t1.record()
        torch.cuda.synchronize()
        assert t0.elapsed_time(t1) < 500.0                     # milliseconds: bounded, far from a hang
        st = got.status.cpu().numpy()
        assert st[1] == SPEC_DEV_TIMEOUT, st
        assert got.accept_len.cpu().numpy()[1] == -1 and got.accepted_node.cpu().numpy()[1] == -1
        # the other sequences are either finished correctly or report the timeout of the cluster that gave up
        for b in (0, 2):
            assert st[b] in (0, SPEC_DEV_TIMEOUT), st
            if st[b] == 0:
                assert got.accepted_node.cpu().numpy()[b] == ref.accepted_node[b]
    finally:
        binding.set_test_hooks(0, -1)
    again = binding.verify_traversal(*args)
    torch.cuda.synchronize()
    assert (again.status.cpu().numpy() == 0).all()
    assert compare_decisions(ref, again, None).near_margin_mismatches == 0
