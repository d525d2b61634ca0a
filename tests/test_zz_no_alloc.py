"""The one entry point that allocates nothing, dart_topk_rows_noalloc.

Some users of the library cannot allocate device memory when they need candidates: an inference server
that gave all of HBM to its own pool at start-up, a latency-critical loop where cudaMalloc (which
synchronises the device) is off limits, a plug-in that has no dart_handle to keep a workspace in.  For
them the selection of Algorithm 1 lines 6-8 is offered on logits they already hold, with a fixed scratch
array inside the library instead of a workspace.

The check: run dart_draft_step (the existing entry point) with its optional full-logits output, hand
those logits to the new entry point through the C ABI, and compare candidates with the step's own --
twice in a row, because the scratch array keeps the previous call's contents.  This file sorts last so
that a run that stops at the first failure has already run everything else; it also passes on its own.
"""
import numpy as np
import pytest
import torch

from paper_2601_19278_b200 import binding, runner, synthetic as syn

pytestmark = pytest.mark.gpu

TOL_ABS = 2e-2      # the tolerance the other GPU tests use for top-k log-probs
TOL_REL = 1e-2


def _step_outputs(w, seed):
    wt = syn.make_weights(w, seed=seed)
    inp = syn.make_step_inputs(w, seed=seed)
    ses = runner.DraftSession(w, wt, None, want_logits=True)
    ses.load_inputs(inp)
    ses.step()
    torch.cuda.synchronize()
    out = (ses.logits.clone(), ses.topk_ids.clone(), ses.topk_slogit.clone())
    ses.close()
    return out


def _check(logits, ids_ref, sl_ref, topk):
    rows = logits.shape[0] * logits.shape[1]
    flat = logits.reshape(rows, -1).contiguous()
    ids = torch.full((rows, topk), -5, dtype=torch.int32, device=flat.device)
    sl = torch.zeros((rows, topk), dtype=torch.float32, device=flat.device)
    before = torch.cuda.memory_allocated()
    binding.topk_rows_noalloc(flat, topk, 1e-10, ids, sl)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    got_ids, ref_ids = ids.cpu().numpy(), ids_ref.reshape(rows, topk).cpu().numpy()
    got_sl, ref_sl = sl.cpu().numpy(), sl_ref.reshape(rows, topk).cpu().numpy()
    assert np.array_equal(got_ids, ref_ids)              # same fp32 logits, same total order
    assert np.abs(got_sl - ref_sl).max() <= TOL_ABS
    assert (np.linalg.norm(got_sl - ref_sl, axis=1) / np.linalg.norm(ref_sl, axis=1)).max() <= TOL_REL


def test_noalloc_topk_matches_the_draft_step_twice_in_a_row():
    small = syn.small_variant(syn.WORKLOADS["C1"], batch=3, ragged_lo=20, prefix=90, vocab=4112)
    big = syn.small_variant(syn.WORKLOADS["C1"], batch=16, K=8, ragged_lo=10, prefix=200, vocab=2048, tree_budget=60)
    a = _step_outputs(small, seed=11)       # 12 rows
    b = _step_outputs(big, seed=12)         # 128 rows: the maximum, and it overwrites every scratch entry
    _check(*a, topk=small.topk)
    _check(*b, topk=big.topk)
    _check(*a, topk=small.topk)             # after a larger call: stale scratch contents must not leak in
    _check(*a, topk=small.topk)


def test_noalloc_topk_rejects_what_does_not_fit():
    dev = torch.device("cuda:0")
    logits = torch.zeros((129, 64), dtype=torch.float32, device=dev)
    ids = torch.zeros((129, 8), dtype=torch.int32, device=dev)
    sl = torch.zeros((129, 8), dtype=torch.float32, device=dev)
    with pytest.raises(binding.DartError) as e:
        binding.topk_rows_noalloc(logits, 8, 1e-10, ids, sl)
    assert e.value.status == binding.DART_ERR_CAPACITY
    with pytest.raises(binding.DartError) as e:
        binding.topk_rows_noalloc(logits[:4].contiguous(), 33, 1e-10, ids, sl)
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    # fewer vocabulary entries than slices still works (k clipped by the caller to the vocabulary)
    tiny = torch.arange(10, dtype=torch.float32, device=dev).reshape(1, 10).contiguous()
    binding.topk_rows_noalloc(tiny, 4, 1e-10, ids, sl)
    torch.cuda.synchronize()
    assert ids[0, :4].tolist() == [9, 8, 7, 6]
