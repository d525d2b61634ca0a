"""dart_build_tree with the N-gram held as child lists (Appendix C) instead of the hash table: the layout changes
how a row is found, never the tree -- bit for bit against the oracle's Algorithm 1 on the same rows, for short and
vocabulary-long child lists, absent contexts, per-sequence row windows and both N-gram orders."""
import numpy as np
import pytest
import torch

import parity
from oracle import tree as otree
from paper_2601_19278_b200 import binding, runner, synthetic as syn

pytestmark = pytest.mark.gpu

VOCAB = 2048
TRIE = dict(ngram_layout=binding.NGRAM_TRIE)


def _session(batch, K, topk=25, beam=20, budget=60, rows=None, vocab=VOCAB, **cfg_over):
    w = syn.small_variant(syn.WORKLOADS["C1"], batch=batch, K=K, vocab=vocab, topk=topk, beam=beam, tree_budget=budget)
    return w, runner.DraftSession(w, syn.make_weights(w), rows, **cfg_over)


def _gpu_tree(ses, ids, sl, ctx, first_row=0, n_levels=None):
    dev = ses.dev
    # a first call on other candidates, so that nothing a call leaves in the library's workspace can stand in for the next one's work
    ses.draft.build_tree(batch=ids.shape[0], topk_ids=torch.from_numpy(np.ascontiguousarray(ids[:, ::-1, ::-1])).to(dev),
                         topk_slogit=torch.from_numpy(sl).to(dev), ctx_tail=torch.from_numpy(np.ascontiguousarray(ctx[:, ::-1])).to(dev),
                         tokens=ses.tokens, parents=ses.parents, depth=ses.depth, mask=ses.mask, n_nodes=ses.n_nodes, scores=ses.scores,
                         first_row=first_row, n_levels=n_levels)
    ses.draft.build_tree(batch=ids.shape[0], topk_ids=torch.from_numpy(ids).to(dev), topk_slogit=torch.from_numpy(sl).to(dev),
                         ctx_tail=torch.from_numpy(ctx).to(dev), tokens=ses.tokens, parents=ses.parents, depth=ses.depth,
                         mask=ses.mask, n_nodes=ses.n_nodes, scores=ses.scores, first_row=first_row, n_levels=n_levels)
    out = ses.tree_outputs()
    assert ses.draft.device_status() == 0
    return out


@pytest.mark.parametrize("seed,budget,order", [(0, 60, 3), (1, 60, 3), (2, 16, 3), (3, 64, 2)])
def test_paper_settings_bit_exact_and_smaller_than_the_hash(seed, budget, order):
    rows = syn.make_ngram_rows(VOCAB, 80_000, "zipf_mixed", seed=seed)
    tri, bi = otree.tables_from_rows(rows)
    t = syn.make_tree_inputs(VOCAB, 4, 8, 25, seed=seed)
    ref = parity.oracle_tree_batch(t["ids"], t["slogit"], t["ctx_tail"], tri if order == 3 else {}, bi, beam=20, budget=budget)
    sizes = {}
    for name, over in (("trie", TRIE), ("hash", {})):
        w, ses = _session(4, 8, budget=budget, rows=rows, ngram_order=order, **over)
        parity.assert_tree_equal(_gpu_tree(ses, t["ids"], t["slogit"], t["ctx_tail"]), ref)
        sizes[name] = ses.draft.ngram_bytes()
        ses.close()
    n_kept = len(bi) + (len(tri) if order == 3 else 0)
    n_long_max = n_kept // 1017 + 1                      # lists long enough to carry a bitmap (64 bytes per 480 tokens, + filler)
    assert 8 * n_kept <= sizes["trie"] <= 16 * n_kept + 16 * (VOCAB + 2) + n_long_max * (64 * 5 + 56)
    assert sizes["hash"] >= 32 * n_kept and sizes["trie"] < sizes["hash"] / 2


@pytest.mark.parametrize("vocab", [2048, 32768])
def test_vocabulary_long_child_lists(vocab):
    """Child lists of every length class (1 entry, a few, both sides of the long-list threshold of 1016, the whole
    vocabulary), candidates on their first and last entries, between entries and on both sides of the 480-token
    blocks of a long list's bitmap, each row with a score of its own."""
    rng = np.random.default_rng(vocab)
    ctxs = [3, 9, 100, 777, vocab - 1, 11, 12]
    lens = [vocab, 300, 17, 1016, 1, 1017, 1024]
    rows = []
    for b, n in zip(ctxs, lens):                        # 2-gram lists under b
        for t in np.sort(rng.choice(vocab, n, replace=False)) if n < vocab else range(vocab):
            rows.append((2, -1, b, int(t)))
    for a, b, n in [(3, 9, vocab), (9, 3, 300), (100, 100, 17), (777, 3, 1016), (vocab - 1, 9, 1), (11, 12, 1017), (12, 11, 1500)]:   # 3-gram lists under (a, b)
        for t in np.sort(rng.choice(vocab, n, replace=False)) if n < vocab else range(vocab):
            rows.append((3, a, b, int(t)))
    for b in range(0, vocab, 2):                        # token 9 is the first token of vocab/2 context nodes
        rows.append((3, 9, b, 5))
    extra = np.array(rows, dtype=np.int64)
    base = syn.make_ngram_rows(vocab, 10, "zipf_mixed", seed=1, extra_rows=extra)
    n = base["score"].shape[0]
    base["score"] = (-1.0 - (np.arange(n) % 9973) / 997.0).astype(np.float32)      # a score per row
    tri, bi = otree.tables_from_rows(base)
    B, K, k = 3, 8, 25
    ids = np.zeros((B, K, k), dtype=np.int32)
    pool = np.array(ctxs + [0, 1, 5, vocab - 2, vocab // 2, 479, 480, 481, 959, 960, 31, 32], dtype=np.int32)
    for b in range(B):
        for i in range(K):
            rest = rng.choice(np.setdiff1d(np.arange(vocab, dtype=np.int32), pool), k - len(pool), replace=False)
            row = np.concatenate([pool, rest.astype(np.int32)])
            rng.shuffle(row)
            ids[b, i] = row
    sl = (-rng.random((B, K, k)) * 3).astype(np.float32)
    ctx = np.array([[3, 9], [11, 12], [-1, vocab - 1]], dtype=np.int32)
    ref = parity.oracle_tree_batch(ids, sl, ctx, tri, bi, beam=20, budget=60)
    for over in (TRIE, {}):
        w, ses = _session(B, K, rows=base, vocab=vocab, **over)
        parity.assert_tree_equal(_gpu_tree(ses, ids, sl, ctx), ref)
        ses.close()
    # the inputs really reach the long lists
    assert sum((3, 9, int(t)) in tri for t in ids[0, 0]) == k and sum((3, int(t)) in bi for t in ids[0, 1]) == k


def test_no_rows_absent_context_and_out_of_range_context_tokens():
    t = syn.make_tree_inputs(VOCAB, 3, 8, 25, seed=6)
    ctx = t["ctx_tail"].copy()
    ctx[1] = (-1, -1)
    ctx[2] = (VOCAB + 5, 7)                      # a context token the table cannot hold: a miss, not a read
    w, ses = _session(3, 8, rows=None, **TRIE)
    assert ses.draft.ngram_bytes() == 0
    parity.assert_tree_equal(_gpu_tree(ses, t["ids"], t["slogit"], ctx), parity.oracle_tree_batch(t["ids"], t["slogit"], ctx, {}, {}, beam=20, budget=60))
    ses.close()
    rows = syn.make_ngram_rows(VOCAB, 50_000, "zipf_mixed", seed=6)
    tri, bi = otree.tables_from_rows(rows)
    w, ses = _session(3, 8, rows=rows, **TRIE)
    parity.assert_tree_equal(_gpu_tree(ses, t["ids"], t["slogit"], ctx), parity.oracle_tree_batch(t["ids"], t["slogit"], ctx, tri, bi, beam=20, budget=60))
    ses.close()


@pytest.mark.parametrize("topk,beam,budget,K,first_row,levels", [(1, 1, 16, 6, 0, 6), (3, 2, 60, 4, 0, 4), (25, 20, 60, 8, 3, 5),
                                                              (32, 32, 64, 8, 0, 8), (25, 20, 60, 8, 7, 1), (5, 32, 40, 3, 1, 2)])
def test_small_candidate_sets_and_row_windows(topk, beam, budget, K, first_row, levels):
    rows = syn.make_ngram_rows(VOCAB, 50_000, "zipf_mixed", seed=8)
    tri, bi = otree.tables_from_rows(rows)
    w, ses = _session(2, K, topk=topk, beam=beam, budget=budget, rows=rows, **TRIE)
    t = syn.make_tree_inputs(VOCAB, 2, K, topk, seed=8)
    got = _gpu_tree(ses, t["ids"], t["slogit"], t["ctx_tail"], first_row=first_row, n_levels=levels)
    ref = parity.oracle_tree_batch(t["ids"][:, first_row:first_row + levels], t["slogit"][:, first_row:first_row + levels],
                                   t["ctx_tail"], tri, bi, beam=beam, budget=budget)
    parity.assert_tree_equal(got, ref)
    ses.close()


def test_per_sequence_first_rows():
    rows = syn.make_ngram_rows(VOCAB, 80_000, "zipf_mixed", seed=12)
    tri, bi = otree.tables_from_rows(rows)
    B, K = 4, 8
    firsts = [0, 3, 7, 6]
    w, ses = _session(B, K, rows=rows, **TRIE)
    t = syn.make_tree_inputs(VOCAB, B, K, 25, seed=12)
    got = _gpu_tree(ses, t["ids"], t["slogit"], t["ctx_tail"], first_row=firsts, n_levels=K)
    for b, fr in enumerate(firsts):
        ref = otree.build_tree(t["ids"][b, fr:], t["slogit"][b, fr:], tuple(int(x) for x in t["ctx_tail"][b]), tri, bi, beam=20, budget=60)
        parity.assert_tree_equal({kk: v[b:b + 1] for kk, v in got.items()}, {kk: np.asarray(v)[None] for kk, v in ref.items() if kk in got})
    ses.close()
