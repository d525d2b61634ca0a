"""GPU parity of the draft-side prefill (dart_draft_prefill) against the oracle's prefill_kv, and of a
drafting step that runs on the cache the prefill built."""
import numpy as np
import pytest
import torch

import parity
from oracle import forward as ofw
from paper_2601_19278_b200 import runner, synthetic as syn

pytestmark = pytest.mark.gpu

C1 = syn.WORKLOADS["C1"]
CASES = {
    # workload (its prefix is the cache capacity here), rows already cached per sequence, new rows per sequence
    "one_seq_37_rows": (syn.small_variant(C1, prefix=64), [5], [37]),
    "two_seqs_ragged": (syn.small_variant(C1, batch=2, prefix=200), [40, 3], [150, 9]),
    "three_seqs_one_empty": (syn.small_variant(C1, batch=3, prefix=200, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128,
                                               mlp_inter=1376, vocab=4112, K=8, tree_budget=60), [1, 30, 60], [1, 0, 131]),
    # the path the benchmark times: 4300 packed rows = two passes (the second sequence straddles the 4096-row pass
    # boundary), 33 token tiles x 10 feature tiles = 330 jobs of the feature FC for 148 persistent CTAs (every CTA
    # takes a second and a third tile: both accumulator buffers and their hand-over), 256 jobs of the k / v projection
    "three_seqs_two_passes": (syn.small_variant(C1, batch=3, prefix=2300, hidden=2560, n_q_heads=16, n_kv_heads=8, head_dim=128,
                                                mlp_inter=1376, vocab=4112, K=8, tree_budget=60), [3, 10, 0], [2100, 2050, 150]),
}


def _new_rows(w, counts, seed=77):
    """Features and next-token ids of the new rows, packed in sequence order."""
    n = sum(counts)
    g = torch.Generator().manual_seed(seed)
    feats = torch.randn(n, 3 * w.hidden, generator=g).to(torch.bfloat16)
    tokens = torch.randint(0, w.vocab, (n,), generator=g, dtype=torch.int32)
    return feats, tokens


@pytest.mark.parametrize("name", list(CASES))
def test_prefill_appends_the_oracle_s_keys_and_values(name):
    w, cached, counts = CASES[name]
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    inp["seq_lens"] = torch.tensor(cached, dtype=torch.int32)   # what lies beyond in the cache is overwritten or ignored
    ses = runner.DraftSession(w, wt, None, want_logits=True)
    ses.load_inputs(inp)
    feats, tokens = _new_rows(w, counts)
    k0, v0 = inp["k_cache"].float().numpy(), inp["v_cache"].float().numpy()
    ses.prefill(feats, tokens, counts)
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    kc, vc = ses.inp["k_cache"].float().cpu().numpy(), ses.inp["v_cache"].float().cpu().numpy()
    cfg, npw = parity.oracle_cfg(w), parity.np_weights(wt)
    off = 0
    for b, n in enumerate(counts):
        P = int(inp["seq_lens"][b])
        if n:
            k, v = ofw.prefill_kv(cfg, npw, syn.bf16_bits(feats[off:off + n]), tokens[off:off + n].numpy(), P + np.arange(n))
            np.testing.assert_allclose(kc[b, :, P:P + n], k.transpose(1, 0, 2), rtol=1e-2, atol=2e-2)
            np.testing.assert_allclose(vc[b, :, P:P + n], v.transpose(1, 0, 2), rtol=1e-2, atol=2e-2)
            assert np.abs(k).max() > 0.05
        keep = np.ones(kc.shape[2], dtype=bool)
        keep[P:P + n] = False                                      # nothing else is written
        assert np.array_equal(kc[b][:, keep], k0[b][:, keep]) and np.array_equal(vc[b][:, keep], v0[b][:, keep])
        off += n
    # a drafting step on the prefilled cache equals the oracle's step on the same (GPU-built, bf16) cache
    lens = inp["seq_lens"].numpy() + np.asarray(counts, dtype=np.int32)
    inp2 = dict(inp)
    inp2["seq_lens"] = torch.from_numpy(lens.astype(np.int32))
    inp2["k_cache"], inp2["v_cache"] = ses.inp["k_cache"].cpu(), ses.inp["v_cache"].cpu()
    ses.load_inputs(inp2)
    ses.step(step_counter=1)
    torch.cuda.synchronize()
    assert ses.draft.device_status() == 0
    ref = parity.oracle_forward(w, wt, inp2)
    parity.check_logits(ses.logits.cpu().numpy(), ref["logits"])
    ses.close()
