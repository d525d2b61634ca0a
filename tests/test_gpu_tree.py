"""dart_build_tree on its own, against the oracle's Algorithm 1, bit for bit: generated inputs at
the paper's settings (d = 8, k = 25, w = 20, budget 60) with a table that really hits, and the
degenerate cases -- exact ties, no table, repeated ids, tiny candidate sets, one level."""
import numpy as np
import pytest
import torch

import parity
from oracle import tree as otree
from paper_2601_19278_b200 import binding, runner, synthetic as syn

pytestmark = pytest.mark.gpu

VOCAB = 2048


def _session(batch, K, topk=25, beam=20, budget=60, rows=None, **cfg_over):
    w = syn.small_variant(syn.WORKLOADS["C1"], batch=batch, K=K, vocab=VOCAB, topk=topk, beam=beam, tree_budget=budget)
    wt = syn.make_weights(w)
    return w, runner.DraftSession(w, wt, rows, **cfg_over)


def _gpu_tree(ses, ids, sl, ctx, first_row=0, n_levels=None):
    dev = ses.dev
    ses.draft.build_tree(batch=ids.shape[0], topk_ids=torch.from_numpy(ids).to(dev), topk_slogit=torch.from_numpy(sl).to(dev),
                         ctx_tail=torch.from_numpy(ctx).to(dev), tokens=ses.tokens, parents=ses.parents, depth=ses.depth,
                         mask=ses.mask, n_nodes=ses.n_nodes, scores=ses.scores, first_row=first_row, n_levels=n_levels)
    out = ses.tree_outputs()
    assert ses.draft.device_status() == 0
    return out


@pytest.mark.parametrize("seed,budget", [(0, 60), (1, 60), (2, 16), (3, 64), (4, 2)])
def test_paper_settings_bit_exact(seed, budget):
    rows = syn.make_ngram_rows(VOCAB, 80_000, "zipf_mixed", seed=seed)
    tri, bi = otree.tables_from_rows(rows)
    w, ses = _session(4, 8, budget=budget, rows=rows)
    t = syn.make_tree_inputs(VOCAB, 4, 8, 25, seed=seed)
    got = _gpu_tree(ses, t["ids"], t["slogit"], t["ctx_tail"])
    ref = parity.oracle_tree_batch(t["ids"], t["slogit"], t["ctx_tail"], tri, bi, beam=20, budget=budget)
    parity.assert_tree_equal(got, ref)
    hits = sum((int(b), int(n)) in bi for b in t["ids"][0, 0] for n in t["ids"][0, 1])
    assert hits > 0
    ses.close()


def test_bigram_only_order_ignores_trigram_rows():
    rows = syn.make_ngram_rows(VOCAB, 80_000, "zipf_mixed", seed=5)
    tri, bi = otree.tables_from_rows(rows)
    w, ses = _session(2, 8, rows=rows, ngram_order=2)
    t = syn.make_tree_inputs(VOCAB, 2, 8, 25, seed=5)
    got = _gpu_tree(ses, t["ids"], t["slogit"], t["ctx_tail"])
    parity.assert_tree_equal(got, parity.oracle_tree_batch(t["ids"], t["slogit"], t["ctx_tail"], {}, bi, beam=20, budget=60))
    ses.close()


def test_exact_ties_no_table_and_absent_context():
    w, ses = _session(3, 8, rows=None)
    t = syn.make_tree_inputs(VOCAB, 3, 8, 25, seed=6)
    sl = t["slogit"].copy()
    sl[0] = 0.0                                   # every score ties: pure generation order
    sl[1] = np.float32(-1.5)                      # ties inside each level, levels differ
    sl[2, :, 5:] = sl[2, :, 4:5]                  # a block of ties at the tail of every level
    ctx = t["ctx_tail"].copy()
    ctx[1] = (-1, -1)
    ctx[2, 0] = -1
    got = _gpu_tree(ses, t["ids"], sl, ctx)
    parity.assert_tree_equal(got, parity.oracle_tree_batch(t["ids"], sl, ctx, {}, {}, beam=20, budget=60))
    ses.close()


def test_all_hits_repeated_ids_and_positive_scores():
    rng = np.random.default_rng(7)
    ids = rng.integers(0, 6, size=(2, 8, 25)).astype(np.int32)          # heavy repetition inside S_i
    sl = (rng.random((2, 8, 25)).astype(np.float32) - 0.3) * 4           # some positive (unphysical) scores
    ctx = np.array([[1, 2], [3, 3]], dtype=np.int32)
    a, b, c = np.meshgrid(np.arange(6), np.arange(6), np.arange(6), indexing="ij")
    tri_rows = np.stack([np.full(216, 3), a.ravel(), b.ravel(), c.ravel()], 1)
    bi_rows = np.stack([np.full(36, 2), np.full(36, -1), a.ravel()[:36] * 0 + np.repeat(np.arange(6), 6), np.tile(np.arange(6), 6)], 1)
    rows = syn.make_ngram_rows(VOCAB, 10, "zipf_mixed", seed=7, extra_rows=np.concatenate([tri_rows, bi_rows]))
    tri, bi = otree.tables_from_rows(rows)
    assert all((x, y, z) in tri for x in range(6) for y in range(6) for z in range(6))
    w, ses = _session(2, 8, rows=rows)
    got = _gpu_tree(ses, ids, sl, ctx)
    parity.assert_tree_equal(got, parity.oracle_tree_batch(ids, sl, ctx, tri, bi, beam=20, budget=60))
    ses.close()


@pytest.mark.parametrize("topk,beam,budget,K,first_row,levels", [(1, 1, 16, 6, 0, 6), (3, 2, 60, 4, 0, 4), (25, 20, 60, 8, 3, 5),
                                                              (32, 32, 64, 8, 0, 8), (25, 20, 60, 8, 7, 1), (5, 32, 40, 3, 1, 2)])
def test_small_candidate_sets_and_row_windows(topk, beam, budget, K, first_row, levels):
    rows = syn.make_ngram_rows(VOCAB, 50_000, "zipf_mixed", seed=8)
    tri, bi = otree.tables_from_rows(rows)
    w, ses = _session(2, K, topk=topk, beam=beam, budget=budget, rows=rows)
    t = syn.make_tree_inputs(VOCAB, 2, K, topk, seed=8)
    got = _gpu_tree(ses, t["ids"], t["slogit"], t["ctx_tail"], first_row=first_row, n_levels=levels)
    ref = parity.oracle_tree_batch(t["ids"][:, first_row:first_row + levels], t["slogit"][:, first_row:first_row + levels],
                                   t["ctx_tail"], tri, bi, beam=beam, budget=budget)
    parity.assert_tree_equal(got, ref)
    ses.close()


def test_argument_and_capacity_errors():
    w, ses = _session(2, 8)
    dev = ses.dev
    ids = torch.zeros((2, 8, 25), dtype=torch.int32, device=dev)
    sl = torch.zeros((2, 8, 25), dtype=torch.float32, device=dev)
    ctx = torch.zeros((2, 2), dtype=torch.int32, device=dev)
    kw = dict(topk_ids=ids, topk_slogit=sl, ctx_tail=ctx, tokens=ses.tokens, parents=ses.parents, depth=ses.depth,
              mask=ses.mask, n_nodes=ses.n_nodes)
    with pytest.raises(binding.DartError) as e:
        ses.draft.build_tree(batch=3, **kw)
    assert e.value.status == binding.DART_ERR_CAPACITY
    with pytest.raises(binding.DartError) as e:
        ses.draft.build_tree(batch=2, first_row=4, n_levels=5, **kw)
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    with pytest.raises(binding.DartError) as e:
        ses.draft.build_tree(batch=2, **dict(kw, ctx_tail=None))
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    # a step whose prefix would overflow the cache is refused before anything is enqueued
    inp = syn.make_step_inputs(w)
    ses.load_inputs(inp)
    ses.inp["seq_lens_host"] = ses.inp["seq_lens_host"] + w.K
    with pytest.raises(binding.DartError) as e:
        ses.step()
    assert e.value.status == binding.DART_ERR_CAPACITY
    ses.inp["seq_lens_host"] = ses.inp["seq_lens_host"] - w.K
    ses.inp["n_fresh"] = 9
    with pytest.raises(binding.DartError) as e:
        ses.step()
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    # per-sequence counts: one out of range, one that overflows its sequence's cache
    ses.inp["n_fresh"] = [1] * (w.batch - 1) + [w.K + 1]
    with pytest.raises(binding.DartError) as e:
        ses.step()
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    ses.inp["n_fresh"] = [1] * w.batch
    ses.inp["seq_lens_host"] = ses.inp["seq_lens_host"].copy()
    ses.inp["seq_lens_host"][-1] = w.max_prefix
    with pytest.raises(binding.DartError) as e:
        ses.step()
    assert e.value.status == binding.DART_ERR_CAPACITY
    with pytest.raises(binding.DartError) as e:
        ses.draft.build_tree(batch=2, first_row=[0, w.K], **kw)
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    torch.cuda.synchronize()
    ses.close()


@pytest.mark.parametrize("topk,beam,budget,K", [(25, 20, 60, 8), (3, 2, 60, 4), (1, 1, 16, 6), (32, 32, 64, 8)])
def test_verification_inputs_match_the_oracle(topk, beam, budget, K):
    """Position ids and root-to-leaf paths of the GPU's own trees, bit for bit."""
    rows = syn.make_ngram_rows(VOCAB, 50_000, "zipf_mixed", seed=8)
    w, ses = _session(2, K, topk=topk, beam=beam, budget=budget, rows=rows)
    t = syn.make_tree_inputs(VOCAB, 2, K, topk, seed=11)
    got = _gpu_tree(ses, t["ids"], t["slogit"], t["ctx_tail"])
    dev = ses.dev
    root_pos = torch.tensor([1000, 17], dtype=torch.int32, device=dev)
    pos = torch.full((2, budget), 7, dtype=torch.int32, device=dev)
    ret = torch.full((2, budget, K + 1), 7, dtype=torch.int32, device=dev)
    nl = torch.zeros((2,), dtype=torch.int32, device=dev)
    ses.draft.verify_inputs(batch=2, max_levels=K, parents=ses.parents, depth=ses.depth, n_nodes=ses.n_nodes, root_pos=root_pos,
                            position_ids=pos, retrieve=ret, n_leaves=nl)
    torch.cuda.synchronize()
    for b in range(2):
        ref = otree.verification_inputs(got["parents"][b], got["depth"][b], int(got["n_nodes"][b]), int(root_pos[b]), K)
        assert np.array_equal(pos[b].cpu().numpy(), ref["position_ids"])
        assert np.array_equal(ret[b].cpu().numpy(), ref["retrieve"])
        assert int(nl[b]) == int(ref["n_leaves"]) and int(nl[b]) >= 1
    ses.close()
