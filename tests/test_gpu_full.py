"""GPU parity at the full sizes of the benchmark configs, in the launch configuration bench.py
times (same session object, same kernels, no debug logits in the timed configuration).

At these sizes the fp64 oracle still finishes in tens of seconds, so the comparison is complete:
every logit of every row, every top-k row, the cache append, and the tree built from the GPU's
own candidates.  C3 (Qwen3-14B shape) is the headline config; C2, C4 and C5 cover the other
hidden sizes, the 32- and 128-row code paths, ragged prefixes and temperature 1."""
import numpy as np
import pytest
import torch

import parity
from oracle import forward as ofw
from oracle import tree as otree
from paper_2601_19278_b200 import runner, synthetic as syn

pytestmark = pytest.mark.gpu


def _full_case(name, ngram_rows=200_000, step_counter=3, ragged_fresh=False):
    w = syn.WORKLOADS[name]
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w, n_fresh=syn.draw_fresh_counts(w) if ragged_fresh else None)
    counts = list(np.broadcast_to(np.asarray(inp["n_fresh"]), (w.batch,)))
    rows = syn.make_ngram_rows(w.vocab, ngram_rows, w.ngram_mode)
    ses = runner.DraftSession(w, wt, rows, want_logits=True, philox_seed=parity.PHILOX_SEED)
    ses.load_inputs(inp)
    ses.step(step_counter=step_counter)
    ses.tree()
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    got_logits = ses.logits.cpu().numpy()
    ids_g, sl_g = ses.topk_ids.cpu().numpy(), ses.topk_slogit.cpu().numpy()
    tree_g = ses.tree_outputs()
    # the configuration bench.py times: no logits buffer.  Candidates and tree must not change.
    ses.logits = None
    ses.topk_ids.fill_(-3)
    ses.step(step_counter=step_counter)
    ses.tree()
    torch.cuda.synchronize()
    assert np.array_equal(ses.topk_ids.cpu().numpy(), ids_g) and np.array_equal(ses.topk_slogit.cpu().numpy(), sl_g)
    parity.assert_tree_equal(ses.tree_outputs(), tree_g)
    kc = {b: ses.inp["k_cache"][b, :, int(inp["seq_lens"][b])].float().cpu().numpy() for b in range(w.batch)}
    ses.close()
    del ses
    torch.cuda.empty_cache()

    ref = parity.oracle_forward(w, wt, inp)
    stats = parity.check_logits(got_logits, ref["logits"])
    worst = 0.0
    for b in range(w.batch):
        for r in range(w.K):
            noise = ofw.gumbel_noise(w.vocab, r, b, step_counter, parity.PHILOX_SEED) if w.temperature > 0 else None
            worst = max(worst, parity.check_topk_row(ids_g[b, r], sl_g[b, r], ref["logits"][b, r], w.topk, 1e-10, w.temperature, noise))
        np.testing.assert_allclose(kc[b], ref["k_new"][b, 0], rtol=1e-2, atol=2e-2)
    tri, bi = otree.tables_from_rows(rows)
    ctx = inp["ctx_tail"].numpy()
    for b in range(w.batch):   # every sequence's tree starts at its own last fresh row
        fr = max(int(counts[b]), 1) - 1
        t = otree.build_tree(ids_g[b, fr:], sl_g[b, fr:], (int(ctx[b, 0]), int(ctx[b, 1])), tri, bi, beam=w.beam, budget=w.tree_budget)
        for key in ("n_nodes", "tokens", "parents", "depth", "mask"):
            assert np.array_equal(tree_g[key][b], np.asarray(t[key])), (b, key)
        assert np.array_equal(tree_g["scores"][b].view(np.uint32), np.asarray(t["scores"], dtype=np.float32).view(np.uint32))
    print(f"{name}: logits max-abs {stats['max_abs']:.3e} rel-L2 {stats['rel_l2']:.3e} s_logit max-abs {worst:.3e}")
    return stats


def test_c3_qwen3_14b_shape_full_parity():
    _full_case("C3")


def test_c2_qwen3_8b_shape_full_parity():
    _full_case("C2")


def test_c4_qwen3_32b_batch4_full_parity():
    _full_case("C4")


def test_c5_ragged_batch16_temperature1_full_parity():
    _full_case("C5")


def test_c5_per_sequence_fresh_counts_full_parity():
    """The steady-state call: every sequence brings its own number of fresh rows (1..K)."""
    _full_case("C5", ragged_fresh=True)


def test_c3_four_fresh_rows_full_parity():
    _full_case("C3", ragged_fresh=True)
