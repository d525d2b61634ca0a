"""GPU parity at sizes the oracle finishes in seconds: the tiny reference config and odd
shapes that span several tiles with ragged tails, every batch-size code path (8, 32, 128
padded token rows), all fresh-row counts, and temperature > 0.  All calls go through the C ABI."""
import numpy as np
import pytest
import torch

import parity
from oracle import forward as ofw
from oracle import tree as otree
from paper_2601_19278_b200 import runner, synthetic as syn

pytestmark = pytest.mark.gpu

C1 = syn.WORKLOADS["C1"]
CASES = {
    "C1": C1,
    "C1_two_fresh": syn.small_variant(C1, n_fresh=2),
    "C1_all_mask": syn.small_variant(C1, n_fresh=0),
    "ragged_b2": syn.small_variant(C1, batch=2, ragged_lo=40, prefix=200),
    "b3_k4_pad32": syn.small_variant(C1, batch=3, ragged_lo=1, prefix=90, vocab=2064),
    "dh128_k8": syn.small_variant(C1, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, mlp_inter=1376,
                                  vocab=4112, prefix=333, K=8, tree_budget=60),
    "gqa5_k8": syn.small_variant(C1, hidden=640, n_q_heads=5, n_kv_heads=1, head_dim=128, mlp_inter=1040,
                                 vocab=3088, prefix=150, K=8, tree_budget=60, batch=2, ragged_lo=3),
    "b16_k8_pad128": syn.small_variant(C1, batch=16, K=8, ragged_lo=10, prefix=300, vocab=2048, tree_budget=60),
    "empty_prefix": syn.small_variant(C1, prefix=0),
    # an MLP wide enough (97 rows per SM on a 148-SM GPU, 96 on its last ones; from 48 on) for the gate / up projection
    # to run with row ownership: every CTA forms its own rows of SiLU(gate) * up from two accumulators
    "wide_mlp_row_ownership": syn.small_variant(C1, mlp_inter=14224, K=8, tree_budget=60, n_fresh=2),
    # the same at 128 token rows: gate and up advance together and share each activation slice (eight k-blocks through
    # a ring of three stages)
    "wide_mlp_row_ownership_b16": syn.small_variant(C1, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, mlp_inter=14224,
                                                    vocab=2064, batch=16, K=8, ragged_lo=10, prefix=120, tree_budget=60),
    # ... and at 32 token rows with 151 rows per SM: two row halves per matrix, four accumulators
    "tall_mlp_row_ownership_b4": syn.small_variant(C1, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, mlp_inter=22208,
                                                   vocab=2064, batch=4, K=8, ragged_lo=10, prefix=120, tree_budget=60),
    # the remaining shapes of that kernel: 32 token rows with one row half, 8 token rows with two
    "wide_mlp_row_ownership_b4": syn.small_variant(C1, mlp_inter=14224, batch=4, K=8, ragged_lo=10, prefix=120, tree_budget=60),
    "tall_mlp_row_ownership_b1": syn.small_variant(C1, mlp_inter=22208, K=8, tree_budget=60, n_fresh=2),
    "hot_b4": syn.small_variant(C1, batch=4, ragged_lo=20, prefix=160, temperature=1.0),
    # enough 64-key tiles (sum over sequences x KV heads >= 512) for the tensor-core split-KV attention: ragged
    # lengths (partial last tiles, sequences with fewer chunks), 16 and 40 query rows per KV head; one long sequence
    # just above that bound, cut into many short chunks
    "attn_tiles_g2": syn.small_variant(C1, hidden=512, n_q_heads=32, n_kv_heads=16, head_dim=128, mlp_inter=1376,
                                       vocab=2064, batch=8, ragged_lo=900, prefix=2000, K=8, tree_budget=60),
    "attn_tiles_g5": syn.small_variant(C1, hidden=512, n_q_heads=40, n_kv_heads=8, head_dim=128, mlp_inter=1376,
                                       vocab=2064, batch=8, ragged_lo=2100, prefix=3000, K=8, tree_budget=60),
    "attn_tiles_b1": syn.small_variant(C1, hidden=512, n_q_heads=40, n_kv_heads=8, head_dim=128, mlp_inter=1376,
                                       vocab=2064, batch=1, prefix=4100, K=8, tree_budget=60),
}


def _run(w, want_tree=True, step_counter=5):
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    rows = syn.make_ngram_rows(w.vocab, min(w.ngram_rows, 20000), w.ngram_mode)
    ses = runner.DraftSession(w, wt, rows, want_logits=True, philox_seed=parity.PHILOX_SEED)
    ses.load_inputs(inp)
    ses.step(step_counter=step_counter)
    if want_tree:
        ses.tree()
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    return wt, inp, rows, ses


@pytest.mark.parametrize("name", list(CASES))
def test_forward_topk_and_cache_match_oracle(name):
    w = CASES[name]
    wt, inp, rows, ses = _run(w, want_tree=False)
    ref = parity.oracle_forward(w, wt, inp)
    stats = parity.check_logits(ses.logits.cpu().numpy(), ref["logits"])
    ids_g, sl_g = ses.topk_ids.cpu().numpy(), ses.topk_slogit.cpu().numpy()
    k = ses.cfg.topk
    for b in range(w.batch):
        for r in range(w.K):
            noise = ofw.gumbel_noise(w.vocab, r, b, 5, parity.PHILOX_SEED) if w.temperature > 0 else None
            parity.check_topk_row(ids_g[b, r], sl_g[b, r], ref["logits"][b, r], k, 1e-10, w.temperature, noise)
    # cache rows P_b .. P_b+F-1 hold the fresh positions' post-RoPE k, v (bf16-rounded); earlier rows untouched
    kc, vc = ses.inp["k_cache"].float().cpu().numpy(), ses.inp["v_cache"].float().cpu().numpy()
    k0, v0 = inp["k_cache"].float().numpy(), inp["v_cache"].float().numpy()
    for b in range(w.batch):
        P = int(inp["seq_lens"][b])
        assert np.array_equal(kc[b, :, :P], k0[b, :, :P]) and np.array_equal(vc[b, :, :P], v0[b, :, :P])
        for r in range(inp["n_fresh"]):
            np.testing.assert_allclose(kc[b, :, P + r], ref["k_new"][b, r], rtol=1e-2, atol=2e-2)
            np.testing.assert_allclose(vc[b, :, P + r], ref["v_new"][b, r], rtol=1e-2, atol=2e-2)
    assert stats["max_abs"] < parity.TOL_ABS
    ses.close()


@pytest.mark.parametrize("name", ["C1", "ragged_b2", "dh128_k8", "b16_k8_pad128", "hot_b4", "C1_two_fresh"])
def test_tree_from_gpu_candidates_is_bit_exact(name):
    """The oracle's Algorithm 1 on the GPU's own (ids, s_logit) must give the GPU's tree."""
    w = CASES[name]
    wt, inp, rows, ses = _run(w)
    tri, bi = otree.tables_from_rows(rows)
    fr = max(inp["n_fresh"], 1) - 1
    ids, sl = ses.topk_ids.cpu().numpy()[:, fr:], ses.topk_slogit.cpu().numpy()[:, fr:]
    ref = parity.oracle_tree_batch(ids, sl, inp["ctx_tail"].numpy(), tri, bi, beam=w.beam, budget=w.tree_budget)
    parity.assert_tree_equal(ses.tree_outputs(), ref)
    ses.close()


def test_planted_ngram_rows_change_the_tree_and_stay_bit_exact():
    """Random-init logits almost never meet random table rows, so plant rows on the oracle's own
    top-k ids: the hit path of the lookup is then exercised end to end."""
    w = C1
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    ref = parity.oracle_forward(w, wt, inp)
    top = [ofw.topk_candidates(ref["logits"][0, r], w.topk, 1e-10)["ids"] for r in range(w.K)]
    ctx = inp["ctx_tail"].numpy()[0]
    extra = [[3, int(ctx[0]), int(ctx[1]), int(top[0][5])], [2, -1, int(ctx[1]), int(top[0][7])]]
    for r in range(1, w.K):
        extra += [[3, int(top[r - 1][j]), int(top[r - 1][j + 1]), int(top[r][9 - j])] for j in range(4)]
        extra += [[2, -1, int(top[r - 1][j]), int(top[r][j + 3])] for j in range(6)]
        if r >= 2:
            extra += [[3, int(top[r - 2][j]), int(top[r - 1][2 * j]), int(top[r][j + 1])] for j in range(6)]
    rows = syn.make_ngram_rows(w.vocab, 20000, w.ngram_mode, extra_rows=np.array(extra))
    tri, bi = otree.tables_from_rows(rows)
    ses = runner.DraftSession(w, wt, rows, want_logits=False)
    ses.load_inputs(inp)
    ses.step()
    ses.tree()
    got = ses.tree_outputs()
    ids, sl = ses.topk_ids.cpu().numpy(), ses.topk_slogit.cpu().numpy()
    with_table = parity.oracle_tree_batch(ids, sl, inp["ctx_tail"].numpy(), tri, bi, beam=w.beam, budget=w.tree_budget)
    without = parity.oracle_tree_batch(ids, sl, inp["ctx_tail"].numpy(), {}, {}, beam=w.beam, budget=w.tree_budget)
    parity.assert_tree_equal(got, with_table)
    assert not np.array_equal(with_table["tokens"], without["tokens"])
    ses.close()


def test_runs_are_bitwise_repeatable():
    w = CASES["dh128_k8"]
    wt, inp, rows, ses = _run(w)
    a = (ses.logits.clone(), ses.topk_ids.clone(), ses.topk_slogit.clone(), ses.tokens.clone(), ses.mask.clone())
    for _ in range(20):
        ses.step(step_counter=5)
        ses.tree()
        torch.cuda.synchronize()
        b = (ses.logits, ses.topk_ids, ses.topk_slogit, ses.tokens, ses.mask)
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    ses.close()


def test_runs_with_128_token_rows_and_noise_are_bitwise_repeatable():
    """At 33..128 token rows the LM head's CTAs prune against a bound they share through global memory, so which
    candidates a CTA keeps depends on timing; the merged candidates, their log-probabilities and the trees must not.
    A vocabulary wide enough for every SM to hold several tiles, temperature 1 (the bound then uses a lower bound of
    the noisy keys), 12 runs."""
    w = syn.small_variant(C1, batch=16, K=8, ragged_lo=10, prefix=300, vocab=80000, tree_budget=60, temperature=1.0)
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    rows = syn.make_ngram_rows(w.vocab, 20000, w.ngram_mode)
    ses = runner.DraftSession(w, wt, rows, want_logits=True, philox_seed=parity.PHILOX_SEED)
    ses.load_inputs(inp)
    ses.step(step_counter=5)
    ses.tree()
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    ref = parity.oracle_forward(w, wt, inp)
    stats = parity.check_logits(ses.logits.cpu().numpy(), ref["logits"])
    assert stats["max_abs"] < parity.TOL_ABS
    a = (ses.topk_ids.clone(), ses.topk_slogit.clone(), ses.tokens.clone(), ses.parents.clone(), ses.mask.clone())
    for _ in range(12):
        ses.step(step_counter=5)
        ses.tree()
        torch.cuda.synchronize()
        for x, y in zip(a, (ses.topk_ids, ses.topk_slogit, ses.tokens, ses.parents, ses.mask)):
            assert torch.equal(x, y)
    ses.close()


def test_packed_io_moves_a_step_with_one_copy_each_way():
    """The end-to-end path of the benchmark: inputs in one pinned buffer, one copy in, one copy out."""
    w = CASES["ragged_b2"]
    wt, inp, rows, ses = _run(w)
    ref = {k: getattr(ses, k).clone() for k in ("tokens", "parents", "depth", "mask", "n_nodes")}
    in_host, in_dev, out_host, out_dev, hv = ses.pack_io()
    in_dev.zero_()                                    # the inputs must really come from the host mirror
    for n in ("tokens", "parents", "depth", "mask", "n_nodes"):
        getattr(ses, n).fill_(3)
    in_dev.copy_(in_host, non_blocking=True)
    ses.step(step_counter=5)
    ses.tree()
    out_host.copy_(out_dev, non_blocking=True)
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    for n, t in ref.items():
        assert torch.equal(hv["out_" + n], t.cpu()), n
    ses.close()


@pytest.mark.parametrize("name,counts", [("ragged_b2", [2, 1]), ("b3_k4_pad32", [0, 4, 3]), ("hot_b4", [1, 3, 0, 2]),
                                          ("b16_k8_pad128", [1, 8, 2, 0, 5, 1, 1, 3, 7, 2, 4, 1, 6, 0, 1, 2])])
def test_per_sequence_fresh_counts_match_oracle(name, counts):
    """The steady-state call after a verification that accepted a different number of tokens per sequence:
    packed fresh rows, per-sequence cache append, and trees that start at each sequence's own last fresh row."""
    w = CASES[name]
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w, n_fresh=counts)
    rows = syn.make_ngram_rows(w.vocab, min(w.ngram_rows, 20000), w.ngram_mode)
    ses = runner.DraftSession(w, wt, rows, want_logits=True, philox_seed=parity.PHILOX_SEED)
    ses.load_inputs(inp)
    ses.step(step_counter=5)
    ses.tree()
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    ref = parity.oracle_forward(w, wt, inp)
    parity.check_logits(ses.logits.cpu().numpy(), ref["logits"])
    ids_g, sl_g = ses.topk_ids.cpu().numpy(), ses.topk_slogit.cpu().numpy()
    for b in range(w.batch):
        for r in range(w.K):
            noise = ofw.gumbel_noise(w.vocab, r, b, 5, parity.PHILOX_SEED) if w.temperature > 0 else None
            parity.check_topk_row(ids_g[b, r], sl_g[b, r], ref["logits"][b, r], w.topk, 1e-10, w.temperature, noise)
    # the call appends exactly the fresh positions of every sequence
    kc, vc = ses.inp["k_cache"].float().cpu().numpy(), ses.inp["v_cache"].float().cpu().numpy()
    k0, v0 = inp["k_cache"].float().numpy(), inp["v_cache"].float().numpy()
    for b in range(w.batch):
        P = int(inp["seq_lens"][b])
        for r in range(counts[b]):
            np.testing.assert_allclose(kc[b, :, P + r], ref["k_new"][b, r], rtol=1e-2, atol=2e-2)
            np.testing.assert_allclose(vc[b, :, P + r], ref["v_new"][b, r], rtol=1e-2, atol=2e-2)
        keep = np.ones(kc.shape[2], dtype=bool)
        keep[P:P + counts[b]] = False
        assert np.array_equal(kc[b][:, keep], k0[b][:, keep]) and np.array_equal(vc[b][:, keep], v0[b][:, keep])
    # every sequence's tree starts at its own last fresh row and is bit-exact from the GPU's candidates
    tri, bi = otree.tables_from_rows(rows)
    got = ses.tree_outputs()
    ctx = inp["ctx_tail"].numpy()
    for b in range(w.batch):
        fr = max(counts[b], 1) - 1
        t = otree.build_tree(ids_g[b, fr:], sl_g[b, fr:], (int(ctx[b, 0]), int(ctx[b, 1])), tri, bi, beam=w.beam, budget=w.tree_budget)
        for key in ("n_nodes", "tokens", "parents", "depth", "mask"):
            assert np.array_equal(got[key][b], np.asarray(t[key])), (b, key)
    ses.close()


def test_prefused_features_skip_the_feature_fc():
    """feat_in = 0: the caller passes g itself; logits, candidates and the appended cache rows against the oracle."""
    w = syn.small_variant(C1, batch=3, ragged_lo=9, prefix=70, K=4, n_fresh=2, vocab=2064)
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    g = torch.Generator().manual_seed(21)
    inp["feats"] = torch.randn(w.batch, 2, w.hidden, generator=g).to(torch.bfloat16)     # g instead of 3h features
    ses = runner.DraftSession(w, wt, None, want_logits=True, philox_seed=parity.PHILOX_SEED, feat_in=0)
    ses.load_inputs(inp)
    ses.step(step_counter=5)
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    npw = parity.np_weights(wt)
    npw["w_fc"] = None
    ref = ofw.draft_forward(parity.oracle_cfg(w), npw, parity.np_inputs(inp))
    stats = parity.check_logits(ses.logits.cpu().numpy(), ref["logits"])
    assert stats["max_abs"] < parity.TOL_ABS
    ids_g, sl_g = ses.topk_ids.cpu().numpy(), ses.topk_slogit.cpu().numpy()
    for b in range(w.batch):
        for r in range(w.K):
            parity.check_topk_row(ids_g[b, r], sl_g[b, r], ref["logits"][b, r], ses.cfg.topk, 1e-10, 0.0, None)
    kc = ses.inp["k_cache"].float().cpu().numpy()
    for b in range(w.batch):
        P = int(inp["seq_lens"][b])
        for r in range(2):
            np.testing.assert_allclose(kc[b, :, P + r], ref["k_new"][b, r], rtol=1e-2, atol=2e-2)
    ses.close()


def test_tensor_core_attention_edge_lengths():
    """The split-KV attention on tcgen05 with sequences of 0, 63, 64 and 65 cached positions next to long ones: an
    empty cache (only the new rows), a partial single tile, an exact tile, a one-key second tile."""
    w = syn.small_variant(C1, hidden=512, n_q_heads=32, n_kv_heads=16, head_dim=128, mlp_inter=1376, vocab=2064,
                          batch=8, ragged_lo=3000, prefix=4000, K=8, tree_budget=60)
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    lens = inp["seq_lens"].clone()
    lens[:4] = torch.tensor([0, 63, 64, 65], dtype=lens.dtype)
    inp["seq_lens"] = lens
    assert sum((int(x) + 63) // 64 for x in lens) * w.n_kv_heads >= 2048     # enough key tiles for that kernel
    ses = runner.DraftSession(w, wt, None, want_logits=True, philox_seed=parity.PHILOX_SEED)
    ses.load_inputs(inp)
    ses.step(step_counter=5)
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    ref = parity.oracle_forward(w, wt, inp)
    stats = parity.check_logits(ses.logits.cpu().numpy(), ref["logits"])
    assert stats["max_abs"] < parity.TOL_ABS
    ses.close()
