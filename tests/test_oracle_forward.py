"""Pins for the forward oracle: every function is checked against something other than
itself -- a torch fp64 library routine stating the same textbook math, a closed form, an
invariant, or a special case (Section 3.1 causal rule, Section 3.2 forward, Appendix B)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import forward as ofw
from oracle import mask as omask
from oracle import philox as ophilox
from paper_2601_19278_b200 import synthetic as syn

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cfg(w):
    return dict(hidden=w.hidden, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                K=w.K, rope_theta=1e6, rms_eps=1e-6)


def _np_weights(wt):
    return {k: syn.bf16_bits(v) for k, v in wt.items()}


def _np_inputs(inp):
    return {"feats": syn.bf16_bits(inp["feats"]), "tokens": inp["tokens"].numpy(),
            "seq_lens": inp["seq_lens"].numpy(), "k_cache": syn.bf16_bits(inp["k_cache"]),
            "v_cache": syn.bf16_bits(inp["v_cache"]), "n_fresh": inp["n_fresh"]}


TINY = syn.small_variant(syn.WORKLOADS["C1"], vocab=512, prefix=37)


def test_bf16_widening_and_rounding_match_torch():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(4096, generator=g, dtype=torch.float32) * 3
    xb = x.to(torch.bfloat16)
    assert np.array_equal(ofw.bf16_to_f64(syn.bf16_bits(xb)), xb.to(torch.float64).numpy())
    assert np.array_equal(ofw.f64_to_bf16_bits(x.to(torch.float64).numpy()), syn.bf16_bits(xb))


def test_rmsnorm_matches_torch_rms_norm():
    g = torch.Generator().manual_seed(2)
    x = torch.randn(5, 96, generator=g, dtype=torch.float64)
    gam = 1 + 0.1 * torch.randn(96, generator=g, dtype=torch.float64)
    ref = torch.nn.functional.rms_norm(x, (96,), gam, eps=1e-6).numpy()
    np.testing.assert_allclose(ofw.rmsnorm(x.numpy(), gam.numpy(), 1e-6), ref, rtol=1e-13, atol=1e-14)


def test_rope_identity_norm_relative_and_complex_form():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((2, 5, 64))
    y = rng.standard_normal((2, 5, 64))
    pos = np.array([0, 1, 7, 100, 5000])
    rx = ofw.rope(x, pos, 1e6)
    # position 0 is the identity; rotation preserves the norm
    np.testing.assert_allclose(rx[:, 0], x[:, 0], rtol=0, atol=0)
    np.testing.assert_allclose(np.linalg.norm(rx, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    # the score q.k depends only on the position difference
    d1 = np.einsum("hrd,hrd->hr", ofw.rope(x, pos, 1e6), ofw.rope(y, pos + 3, 1e6))
    d2 = np.einsum("hrd,hrd->hr", ofw.rope(x, pos + 1234, 1e6), ofw.rope(y, pos + 1237, 1e6))
    np.testing.assert_allclose(d1, d2, rtol=1e-9, atol=1e-9)
    # independent statement: pairs (x_i, x_{i+32}) as complex numbers times exp(i*pos*theta^(-2i/64))
    zc = x[..., :32] + 1j * x[..., 32:]
    freq = 1e6 ** (-np.arange(32) / 32.0)
    rot = zc * np.exp(1j * pos[:, None] * freq[None, :])
    np.testing.assert_allclose(rx, np.concatenate([rot.real, rot.imag], -1), rtol=1e-12, atol=1e-12)


def test_attention_matches_torch_sdpa_with_explicit_mask():
    rng = np.random.default_rng(4)
    K, Hq, Hkv, dh, P = 5, 6, 2, 16, 11
    q = rng.standard_normal((K, Hq, dh))
    k_all = rng.standard_normal((Hkv, P + K, dh))
    v_all = rng.standard_normal((Hkv, P + K, dh))
    got = ofw.attention_rows(q, k_all, v_all, P)
    mask = torch.tensor([[s <= P + r for s in range(P + K)] for r in range(K)])
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]                           # [1,Hq,K,dh]
    tk = torch.from_numpy(k_all).repeat_interleave(Hq // Hkv, dim=0)[None]
    tv = torch.from_numpy(v_all).repeat_interleave(Hq // Hkv, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)[0].permute(1, 0, 2)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-12, atol=1e-13)


def test_attention_special_cases():
    rng = np.random.default_rng(5)
    # all keys equal -> output is the mean of the visible values
    K, Hq, Hkv, dh, P = 3, 2, 1, 8, 6
    q = rng.standard_normal((K, Hq, dh))
    k_all = np.tile(rng.standard_normal((1, 1, dh)), (Hkv, P + K, 1))
    v_all = rng.standard_normal((Hkv, P + K, dh))
    out = ofw.attention_rows(q, k_all, v_all, P)
    for r in range(K):
        np.testing.assert_allclose(out[r, 0], v_all[0, :P + r + 1].mean(0), rtol=1e-12)
    # empty prefix, one row -> the row's own value
    out = ofw.attention_rows(q[:1], k_all[:, :1], v_all[:, :1], 0)
    np.testing.assert_allclose(out[0, 1], v_all[0, 0], rtol=1e-13)
    assert ofw.visible(4, 0, 4) and not ofw.visible(4, 0, 5) and ofw.visible(4, 2, 6)


def test_inference_mask_is_one_block_of_the_training_mask():
    """Appendix B's prefix-shared training mask, restricted to the block of prompt position n,
    is the causal rule the inference step applies to [prefix 0..n, masks]."""
    prompt_len, draft_len = 9, 7
    for n in (0, 3, 8):
        P = n                                   # cached positions 0..n-1; the fresh row is position n
        # query slots of this block in the packed row, preceded by the clean row at position n
        q_slots = [n] + [prompt_len + n * draft_len + i for i in range(draft_len)]
        kv_slots = list(range(n + 1)) + [prompt_len + n * draft_len + i for i in range(draft_len)]
        for r, qs in enumerate(q_slots):
            for s, ks in enumerate(kv_slots):
                assert omask.training_visible(qs, ks, prompt_len, draft_len, prompt_len) == ofw.visible(P, r, s), (n, r, s)
        # and it never reads another block
        other = prompt_len + ((n + 1) % prompt_len) * draft_len
        assert not omask.training_visible(q_slots[-1], other, prompt_len, draft_len, prompt_len)


def _torch_layer(w, wt, inp):
    """Second statement of the whole layer with torch fp64 library ops, batched differently."""
    f64 = lambda t: t.to(torch.float64)
    h, Hq, Hkv, dh, K = w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.K
    F, B = inp["n_fresh"], w.batch
    rn = lambda x, g: torch.nn.functional.rms_norm(x, (x.shape[-1],), f64(g), eps=1e-6)
    g = f64(wt["mask_vec"])[:h].expand(B, K, h).clone()
    e = f64(wt["mask_vec"])[h:].expand(B, K, h).clone()
    if F:
        g[:, :F] = f64(inp["feats"]) @ f64(wt["w_fc"]).T
        e[:, :F] = f64(wt["embed"])[inp["tokens"].long()]
    z = torch.cat([rn(g, wt["norm_g"]), rn(e, wt["norm_e"])], -1)
    q = (z @ f64(wt["w_q"]).T).view(B, K, Hq, dh).transpose(1, 2)
    k = (z @ f64(wt["w_k"]).T).view(B, K, Hkv, dh).transpose(1, 2)
    v = (z @ f64(wt["w_v"]).T).view(B, K, Hkv, dh).transpose(1, 2)
    outs = []
    for b in range(B):
        P = int(inp["seq_lens"][b])
        pos = torch.arange(P, P + K, dtype=torch.float64)
        inv = 1e6 ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
        ang = torch.outer(pos, inv)
        cos, sin = torch.cat([ang.cos(), ang.cos()], -1), torch.cat([ang.sin(), ang.sin()], -1)
        rot = lambda x: torch.cat([-x[..., dh // 2:], x[..., :dh // 2]], -1)
        qb, kb = q[b] * cos + rot(q[b]) * sin, k[b] * cos + rot(k[b]) * sin
        kk = torch.cat([f64(inp["k_cache"][b, :, :P]), kb], 1).repeat_interleave(Hq // Hkv, 0)
        vv = torch.cat([f64(inp["v_cache"][b, :, :P]), v[b]], 1).repeat_interleave(Hq // Hkv, 0)
        m = torch.ones(K, P + K, dtype=torch.bool).tril(diagonal=P)
        a = torch.nn.functional.scaled_dot_product_attention(qb[None], kk[None], vv[None], attn_mask=m)[0]
        outs.append(a.transpose(0, 1).reshape(K, Hq * dh))
    a = torch.stack(outs)
    x1 = g + a @ f64(wt["w_o"]).T
    n2 = rn(x1, wt["norm_post"])
    u = torch.nn.functional.silu(n2 @ f64(wt["w_gate"]).T) * (n2 @ f64(wt["w_up"]).T)
    x2 = x1 + u @ f64(wt["w_down"]).T
    return rn(x2, wt["norm_final"]) @ f64(wt["w_lm"]).T


@pytest.mark.parametrize("batch,n_fresh", [(1, 1), (2, 2), (2, 0)])
def test_whole_layer_matches_torch_restatement(batch, n_fresh):
    w = syn.small_variant(TINY, batch=batch, n_fresh=n_fresh, ragged_lo=5 if batch > 1 else 0)
    wt = syn.make_weights(w)
    inp = syn.make_step_inputs(w)
    got = ofw.draft_forward(_cfg(w), _np_weights(wt), _np_inputs(inp))["logits"]
    ref = _torch_layer(w, wt, inp).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-9, atol=1e-11)
    assert np.abs(ref).max() > 0.1            # the comparison is not between zeros


def test_causality_rows_do_not_depend_on_later_rows():
    w4 = TINY
    w6 = syn.small_variant(TINY, K=6, prefix=TINY.prefix - 2)     # same cache capacity
    wt = _np_weights(syn.make_weights(w4))
    i4 = _np_inputs(syn.make_step_inputs(w4))
    i6 = dict(i4)
    i6["seq_lens"] = i4["seq_lens"].copy()
    a = ofw.draft_forward(_cfg(w4), wt, i4)["logits"]
    b = ofw.draft_forward(_cfg(w6), wt, i6)["logits"]
    np.testing.assert_allclose(a[0], b[0, :4], rtol=1e-12, atol=1e-13)


def test_two_fresh_rows_equal_append_then_one_fresh_row():
    """A step with cache P and F=2 equals a step with cache P+1 and F=1 whose cache row P is the
    first fresh row's k, v (up to the bf16 rounding of that one cached row)."""
    w = syn.small_variant(TINY, n_fresh=2)
    wt = _np_weights(syn.make_weights(w))
    i2 = _np_inputs(syn.make_step_inputs(w))
    cfg = _cfg(w)
    o2 = ofw.draft_forward(cfg, wt, i2)
    P = int(i2["seq_lens"][0])
    i1 = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in i2.items()}
    i1["k_cache"][0, :, P] = ofw.f64_to_bf16_bits(o2["k_new"][0, 0])
    i1["v_cache"][0, :, P] = ofw.f64_to_bf16_bits(o2["v_new"][0, 0])
    i1["seq_lens"] = i2["seq_lens"] + 1
    i1["feats"], i1["tokens"], i1["n_fresh"] = i2["feats"][:, 1:], i2["tokens"][:, 1:], 1
    cfg1 = dict(cfg, K=cfg["K"] - 1)
    o1 = ofw.draft_forward(cfg1, wt, i1)
    np.testing.assert_allclose(o1["logits"][0], o2["logits"][0, 1:], rtol=0, atol=2e-3)
    assert np.abs(o1["logits"][0] - o2["logits"][0, 1:]).max() > 0   # the rounding is really there


def test_log_softmax_and_topk_against_torch():
    rng = np.random.default_rng(6)
    y = rng.standard_normal(1000) * 3
    lp = ofw.log_softmax(y)
    assert abs(np.exp(lp).sum() - 1) < 1e-12
    np.testing.assert_allclose(lp, torch.log_softmax(torch.from_numpy(y), -1).numpy(), rtol=1e-12, atol=1e-12)
    c = ofw.topk_candidates(y, 25, 1e-10)
    tv, ti = torch.topk(torch.from_numpy(y), 25)
    assert np.array_equal(c["ids"], ti.numpy())
    np.testing.assert_allclose(c["slogit"], np.log(np.exp(lp[ti.numpy()]) + 1e-10), rtol=1e-14)
    assert np.all(c["slogit"] <= math.log(1 + 1e-10) + 1e-15) and np.all(np.diff(c["slogit"]) <= 0)
    # ties go to the lower token id; k is clipped to the vocabulary
    t = np.array([1.0, 3.0, 3.0, 0.5, 3.0])
    assert ofw.topk_candidates(t, 4, 1e-10)["ids"].tolist() == [1, 2, 4, 0]
    assert len(ofw.topk_candidates(t, 9, 1e-10)["ids"]) == 5
    # eps floors s_logit for a vanishing probability
    far = np.array([0.0, -1000.0])
    assert abs(ofw.topk_candidates(far, 2, 1e-10)["slogit"][1] - math.log(1e-10)) < 1e-12


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = ophilox.philox4x32_10(np.array([v[:4]], dtype=np.uint32), (v[4], v[5]))[0]
        assert [int(x) for x in out] == v[6:]


def test_gumbel_topk_samples_from_softmax_and_limits():
    V = 16
    rng = np.random.default_rng(7)
    y = rng.standard_normal(V)
    p = np.exp(ofw.log_softmax(y))
    n = 4000
    counts = np.zeros(V)
    for step in range(n):
        noise = ofw.gumbel_noise(V, row=2, b=1, step=step, seed=99)
        assert np.all(np.isfinite(noise))
        counts[ofw.topk_candidates(y, 1, 1e-10, temperature=1.0, noise=noise)["ids"][0]] += 1
    chi2 = np.sum((counts - n * p) ** 2 / (n * p))
    assert chi2 < 45.0                      # 15 dof: P(chi2 > 45) < 1e-4
    # different (row, b, step) give different noise; the same counter gives the same noise
    a = ofw.gumbel_noise(V, 2, 1, 5, 99)
    assert np.array_equal(a, ofw.gumbel_noise(V, 2, 1, 5, 99))
    assert not np.array_equal(a, ofw.gumbel_noise(V, 3, 1, 5, 99))
    assert not np.array_equal(a, ofw.gumbel_noise(V, 2, 0, 5, 99))
    # T -> 0: the logits dominate the noise and the deterministic top-k comes back
    det = ofw.topk_candidates(y, 5, 1e-10)["ids"]
    cold = ofw.topk_candidates(y, 5, 1e-10, temperature=1e-4, noise=a)["ids"]
    assert np.array_equal(det, cold)
    # s_logit stays un-perturbed
    c = ofw.topk_candidates(y, 5, 1e-10, temperature=1.0, noise=a)
    np.testing.assert_allclose(c["slogit"], np.log(p[c["ids"]] + 1e-10), rtol=1e-12)
    # the uniform behind the noise lies strictly inside (0,1): mean of G is Euler's constant
    big = ofw.gumbel_noise(1 << 16, 0, 0, 0, 1)
    assert abs(big.mean() - 0.5772156649) < 0.02


def test_algorithmic_bytes_match_the_closed_form_per_config():
    expect = {"C1": 4_268_032, "C2": 1_789_919_232, "C3": 2_463_891_456, "C4": 2_927_362_048}
    for name, val in expect.items():
        w = syn.WORKLOADS[name]
        assert syn.algorithmic_bytes(w, syn.make_seq_lens(w)) == val


def test_per_sequence_fresh_counts_equal_each_sequence_run_alone():
    """Ragged fresh rows (the steady-state call after a verification that accepted a different number of
    tokens per sequence): every sequence of the batch must come out exactly as if it had been run alone with
    its own uniform count - which pins the packed feature/token offsets against the uniform path, itself
    pinned by the torch restatement above."""
    counts = [2, 0, 4, 1]
    w = syn.small_variant(TINY, batch=4, ragged_lo=7)
    wt = _np_weights(syn.make_weights(w))
    inp = syn.make_step_inputs(w, n_fresh=counts)
    assert inp["feats"].shape[0] == sum(counts) and list(inp["n_fresh"]) == counts
    cfg = _cfg(w)
    got = ofw.draft_forward(cfg, wt, _np_inputs(inp))
    full = syn.make_step_inputs(w, n_fresh=w.K)                   # the rows every sequence drew
    for b, F in enumerate(counts):
        solo = {"feats": full["feats"][b:b + 1, :F].contiguous(), "tokens": full["tokens"][b:b + 1, :F].contiguous(),
                "seq_lens": full["seq_lens"][b:b + 1], "k_cache": full["k_cache"][b:b + 1], "v_cache": full["v_cache"][b:b + 1],
                "n_fresh": F}
        ref = ofw.draft_forward(cfg, wt, _np_inputs(solo))
        np.testing.assert_array_equal(got["logits"][b], ref["logits"][0])
        np.testing.assert_array_equal(got["k_new"][b], ref["k_new"][0])
    # the counts matter: a fresh row and a <mask> row at the same place give different logits
    assert np.abs(got["logits"][0, 1] - got["logits"][1, 1]).max() > 1e-3


def test_prefill_keys_and_values_are_the_forward_pass_s_new_rows():
    """Draft-side prefill: the k, v it stores for a run of new rows are exactly the new rows' k, v of a forward
    pass in which all those rows are fresh (the forward pass being pinned above)."""
    w = syn.small_variant(TINY, K=6, n_fresh=6, prefix=9)
    wt = _np_weights(syn.make_weights(w))
    inp = _np_inputs(syn.make_step_inputs(w))
    cfg = _cfg(w)
    fwd = ofw.draft_forward(cfg, wt, inp)
    P = int(inp["seq_lens"][0])
    k, v = ofw.prefill_kv(cfg, wt, inp["feats"][0], inp["tokens"][0], P + np.arange(6))
    np.testing.assert_allclose(k, fwd["k_new"][0], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(v, fwd["v_new"][0], rtol=1e-12, atol=1e-13)
    # positions matter for k (RoPE) and not for v
    k2, v2 = ofw.prefill_kv(cfg, wt, inp["feats"][0], inp["tokens"][0], P + 1 + np.arange(6))
    assert np.abs(k2 - k).max() > 1e-3 and np.array_equal(v2, v)


def test_prefused_features_equal_the_layer_with_an_identity_fusion():
    """feat_in = 0: the caller hands g itself.  That is the ordinary layer whose fusion matrix is [I | 0 | 0] fed
    with [g, 0, 0] -- a product with exact zeros and ones, so the two runs agree bit for bit."""
    w = syn.small_variant(TINY, batch=2, n_fresh=2, K=4, ragged_lo=5, prefix=21)
    wt = _np_weights(syn.make_weights(w))
    inp = _np_inputs(syn.make_step_inputs(w))
    cfg = _cfg(w)
    h = w.hidden
    g_bits = inp["feats"].reshape(-1, 3 * h)[:, :h].copy()                      # any bf16 rows serve as g
    eye = np.zeros((h, 3 * h), dtype=np.float32)
    eye[np.arange(h), np.arange(h)] = 1.0
    wt_id = dict(wt, w_fc=syn.bf16_bits(torch.from_numpy(eye).to(torch.bfloat16)))
    feats3 = np.zeros((g_bits.shape[0], 3 * h), dtype=g_bits.dtype)
    feats3[:, :h] = g_bits
    ref = ofw.draft_forward(cfg, wt_id, dict(inp, feats=feats3.reshape(inp["feats"].shape)))
    got = ofw.draft_forward(cfg, dict(wt, w_fc=None), dict(inp, feats=g_bits.reshape(inp["feats"].shape[:-1] + (h,))))
    assert np.array_equal(got["logits"], ref["logits"]) and np.array_equal(got["k_new"], ref["k_new"])
    assert not np.allclose(got["logits"], ofw.draft_forward(cfg, wt, inp)["logits"])   # and it is not the random fusion
