"""The time-out path of the bounded device-side waits, made to run on purpose.

Every wait inside the kernels (mbarriers of the TMA / tensor-core pipelines, flags between CTAs) gives up after
a limit, records DART_ERR_TIMEOUT in the handle's status word and lets the kernel return.  Here a one-block
kernel waits, with a small limit, on a barrier nobody signals: nothing faults and nothing hangs; the status word
must report the time-out once, and the same handle must then run a step that matches the oracle -- also when the
kernel that gave up left a work counter of a projection half counted."""
import numpy as np
import pytest
import torch

import parity
from paper_2601_19278_b200 import binding, runner, synthetic as syn

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("leave_ticket", [False, True])
def test_a_wait_that_runs_out_reports_timeout_and_the_handle_recovers(leave_ticket):
    w = syn.WORKLOADS["C1"]
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    ses = runner.DraftSession(w, wt, None, want_logits=True)
    ses.load_inputs(inp)
    ses.step()
    torch.cuda.synchronize()
    assert ses.draft.device_status() == binding.DART_OK
    ses.draft.selftest_bounded_wait(200, leave_ticket=leave_ticket)
    assert ses.draft.device_status() == binding.DART_ERR_TIMEOUT       # reported once ...
    assert ses.draft.device_status() == binding.DART_OK                # ... and cleared
    ses.logits.zero_()
    ses.step(step_counter=1)
    torch.cuda.synchronize()
    assert ses.draft.device_status() == binding.DART_OK
    ref = parity.oracle_forward(w, wt, inp)
    parity.check_logits(ses.logits.cpu().numpy(), ref["logits"])
    ids, sl = ses.topk_ids.cpu().numpy(), ses.topk_slogit.cpu().numpy()
    for r in range(w.K):
        parity.check_topk_row(ids[0, r], sl[0, r], ref["logits"][0, r], w.topk, 1e-10)
    ses.close()


def test_selftest_argument_errors():
    w = syn.WORKLOADS["C1"]
    ses = runner.DraftSession(w, syn.make_weights(w), None)
    for bad in (0, -3, 100001):
        with pytest.raises(binding.DartError) as e:
            ses.draft.selftest_bounded_wait(bad)
        assert e.value.status == binding.DART_ERR_INVALID_ARG
    assert ses.draft.device_status() == binding.DART_OK
    ses.close()
