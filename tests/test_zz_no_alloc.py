"""The one entry point that allocates nothing, dart_topk_rows_noalloc.

Some users of the library cannot allocate device memory when they need candidates: an inference server
that gave all of HBM to its own pool at start-up, a latency-critical loop where cudaMalloc (which
synchronises the device) is off limits, a plug-in that has no dart_handle to keep a workspace in.  For
them the selection of Algorithm 1 lines 6-8 is offered on logits they already hold, with a fixed scratch
array inside the library instead of a workspace.

The checks, each on two calls in a row and across calls of different sizes (the scratch array keeps the previous
call's contents): (1) dart_draft_step (the existing entry point) is run with its optional full-logits output, those
logits go to the new entry point through the C ABI, and the candidates must be the step's own; (2) independently
of any CUDA code, every row is compared with the oracle's candidate selection (Algorithm 1 lines 6-8:
oracle.forward.topk_candidates on the same fp32 logits) -- ids exactly, since both sides see identical values and
break ties towards the lower id, log-probs within the tolerance of the other GPU tests -- including rows with many
repeated logit values and topk = 32; (3) the device's free memory, as the driver reports it, is the same before and
after a call.  This file sorts last so that a run that stops at the first failure has already run everything else;
it also passes on its own.
"""
import numpy as np
import pytest
import torch

import parity
from oracle import forward as ofw
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


_first_call_done = False


def _call(flat, topk):
    global _first_call_done
    rows = flat.shape[0]
    ids = torch.full((rows, topk), -5, dtype=torch.int32, device=flat.device)
    sl = torch.zeros((rows, topk), dtype=torch.float32, device=flat.device)
    if not _first_call_done:
        # the process's first call makes the CUDA runtime load the kernels' code and the static scratch array onto
        # the device (that is the set-up the header documents, not an allocation by the library): keep it out of the
        # free-memory comparison below
        binding.topk_rows_noalloc(flat, topk, 1e-10, ids, sl)
        _first_call_done = True
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]           # the driver's figure: sees any cudaMalloc, whoever makes it
    binding.topk_rows_noalloc(flat, topk, 1e-10, ids, sl)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    return ids.cpu().numpy(), sl.cpu().numpy()


def _check_against_oracle(flat, got_ids, got_sl, topk):
    lg = flat.cpu().numpy().astype(np.float64)
    for r in range(lg.shape[0]):
        c = ofw.topk_candidates(lg[r], topk, 1e-10)
        assert np.array_equal(got_ids[r], c["ids"]), f"row {r}: candidates differ from the oracle's"
        parity.check_topk_row(got_ids[r], got_sl[r], lg[r], topk, 1e-10)


def _check(logits, ids_ref, sl_ref, topk):
    rows = logits.shape[0] * logits.shape[1]
    flat = logits.reshape(rows, -1).contiguous()
    got_ids, got_sl = _call(flat, topk)
    ref_ids, ref_sl = ids_ref.reshape(rows, topk).cpu().numpy(), sl_ref.reshape(rows, topk).cpu().numpy()
    assert np.array_equal(got_ids, ref_ids)              # same fp32 logits, same total order
    assert np.abs(got_sl - ref_sl).max() <= TOL_ABS
    assert (np.linalg.norm(got_sl - ref_sl, axis=1) / np.linalg.norm(ref_sl, axis=1)).max() <= TOL_REL
    _check_against_oracle(flat, got_ids, got_sl, topk)


def test_noalloc_topk_matches_the_draft_step_twice_in_a_row():
    small = syn.small_variant(syn.WORKLOADS["C1"], batch=3, ragged_lo=20, prefix=90, vocab=4112)
    big = syn.small_variant(syn.WORKLOADS["C1"], batch=16, K=8, ragged_lo=10, prefix=200, vocab=2048, tree_budget=60)
    a = _step_outputs(small, seed=11)       # 12 rows
    b = _step_outputs(big, seed=12)         # 128 rows: the maximum, and it overwrites every scratch entry
    _check(*a, topk=small.topk)
    _check(*b, topk=big.topk)
    _check(*a, topk=small.topk)             # after a larger call: stale scratch contents must not leak in
    _check(*a, topk=small.topk)


def test_noalloc_topk_ties_and_topk32_match_the_oracle_twice_in_a_row():
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(31)
    # few distinct values: every row has long runs of equal logits, so the order is decided by the ids
    tied = torch.randint(0, 12, (7, 5000), generator=g).float().mul_(0.25).to(dev)
    wide = torch.randn((40, 3001), generator=g).mul_(3.0).to(dev)      # vocabulary not a multiple of the slice count
    wide[3, 100:140] = wide[3, 7]                                       # a tie that straddles the k-th place
    for _ in range(2):
        for flat, k in ((tied, 32), (wide, 32), (tied, 25), (wide, 1)):
            ids, sl = _call(flat, k)
            _check_against_oracle(flat, ids, sl, k)


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
