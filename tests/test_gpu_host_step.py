"""dart_draft_step_host: the whole draft step from host buffers (copy in, forward pass, tree, copy out, wait) gives
the bits that the two device-resident calls give, for a uniform batch and for per-sequence fresh-row counts."""
import numpy as np
import pytest
import torch

from paper_2601_19278_b200 import runner
from paper_2601_19278_b200 import synthetic as syn

pytestmark = pytest.mark.gpu

C1 = syn.WORKLOADS["C1"]
CASES = {
    "C1": C1,
    "hot_b4": syn.small_variant(C1, batch=4, ragged_lo=20, prefix=160, temperature=1.0),
    "dh128_k8": syn.small_variant(C1, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, mlp_inter=1376,
                                  vocab=4112, prefix=333, K=8, tree_budget=60),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_host_step_matches_the_device_resident_calls(name):
    w = CASES[name]
    wt = syn.make_weights(w)
    ng = syn.make_ngram_rows(w.vocab, min(w.ngram_rows, 20000), w.ngram_mode)
    inp = syn.make_step_inputs(w)
    ses = runner.DraftSession(w, wt, ng)
    ses.load_inputs(inp)
    ses.step(step_counter=3)
    ses.tree()
    torch.cuda.synchronize()
    want = ses.tree_outputs()
    in_host, in_dev, out_host, out_dev, views = ses.pack_io()
    # the device copies of the step's small inputs are overwritten before the call: only the host buffer counts
    keep = in_dev.clone()
    in_dev.zero_()
    out_dev.fill_(0xEE)
    out_host.fill_(0x11)
    call = ses.host_step(in_host, in_dev, out_host, out_dev)
    call(3)                                   # synchronous: no further wait before the host buffer is read
    assert ses.draft.device_status() == 0
    assert torch.equal(in_dev.cpu(), keep.cpu())
    for n in ("tokens", "parents", "depth", "mask", "n_nodes"):
        np.testing.assert_array_equal(views["out_" + n].numpy(), want[n], err_msg=n)
    call(3)
    for n in ("tokens", "parents", "depth", "mask", "n_nodes"):
        np.testing.assert_array_equal(views["out_" + n].numpy(), want[n], err_msg=n + " (second call)")
    ses.close()
