"""Pins of the training-mask attention oracle (Section 3.3, Appendix B) against what the mask's
structure fixes: the clean part is ordinary causal attention, every masked block is the inference
step's attention over its own prefix, blocks are isolated, slots past the length are empty."""
import numpy as np
import torch

from oracle import forward as ofwd
from oracle import train_attention as ota


def _qkv(seed, Hq, Hkv, Lp, d, dh):
    rng = np.random.default_rng(seed)
    L = Lp * (1 + d)
    return rng.standard_normal((Hq, L, dh)), rng.standard_normal((Hkv, L, dh)), rng.standard_normal((Hkv, L, dh))


def test_clean_part_is_plain_causal_attention():
    Hq, Hkv, Lp, d, dh = 4, 2, 9, 3, 8
    q, k, v = _qkv(0, Hq, Hkv, Lp, d, dh)
    out = ota.training_attention(q, k, v, Lp, d, Lp)
    tq, tk, tv = (torch.from_numpy(x[:, :Lp]) for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None].repeat_interleave(Hq // Hkv, 1),
                                                           tv[None].repeat_interleave(Hq // Hkv, 1), is_causal=True)[0]
    assert np.allclose(out[:, :Lp], ref.numpy(), atol=1e-12)


def test_every_block_is_the_inference_step_over_its_own_prefix():
    Hq, Hkv, Lp, d, dh = 4, 2, 7, 4, 8
    q, k, v = _qkv(1, Hq, Hkv, Lp, d, dh)
    out = ota.training_attention(q, k, v, Lp, d, Lp)
    for n in range(Lp):
        blk = slice(Lp + n * d, Lp + (n + 1) * d)
        # the inference step with a cached prefix of n + 1 clean positions and the block's d rows as new rows
        k_all = np.concatenate([k[:, :n + 1], k[:, blk]], axis=1)
        v_all = np.concatenate([v[:, :n + 1], v[:, blk]], axis=1)
        ref = ofwd.attention_rows(np.transpose(q[:, blk], (1, 0, 2)), k_all, v_all, n + 1)      # [d, Hq, dh]
        assert np.allclose(out[:, blk], np.transpose(ref, (1, 0, 2)), atol=1e-12), n


def test_blocks_are_isolated_and_never_read_later_prompt_slots():
    Hq, Hkv, Lp, d, dh = 2, 1, 6, 3, 4
    q, k, v = _qkv(2, Hq, Hkv, Lp, d, dh)
    base = ota.training_attention(q, k, v, Lp, d, Lp)
    n = 2
    blk = slice(Lp + n * d, Lp + (n + 1) * d)
    k2, v2 = k.copy(), v.copy()
    other = np.ones(k.shape[1], dtype=bool)
    other[:n + 1] = False
    other[blk] = False                               # everything block n may not read
    k2[:, other] += 5.0
    v2[:, other] -= 3.0
    again = ota.training_attention(q, k2, v2, Lp, d, Lp)
    assert np.array_equal(again[:, blk], base[:, blk])
    assert not np.allclose(again[:, Lp + (n + 1) * d:], base[:, Lp + (n + 1) * d:])   # the others did move
    # first row of a block with a one-slot prefix reads two keys: closed form
    q0 = q[0, Lp]
    s = np.array([k[0, 0] @ q0, k[0, Lp] @ q0]) / np.sqrt(dh)
    p = np.exp(s - s.max()); p /= p.sum()
    assert np.allclose(base[0, Lp], p[0] * v[0, 0] + p[1] * v[0, Lp], atol=1e-12)


def test_slots_past_the_length_are_zero_and_unread():
    Hq, Hkv, Lp, d, dh = 2, 2, 8, 2, 4
    q, k, v = _qkv(3, Hq, Hkv, Lp, d, dh)
    S = 5
    out = ota.training_attention(q, k, v, Lp, d, S)
    assert np.all(out[:, S:Lp] == 0) and np.all(out[:, Lp + S * d:] == 0)
    assert np.all(np.abs(out[:, :S]).sum(-1) > 0) and np.all(np.abs(out[:, Lp:Lp + S * d]).sum(-1) > 0)
    # the valid part equals the same problem cut to S prompt slots
    cut = np.r_[0:S, Lp:Lp + S * d]
    small = ota.training_attention(q[:, cut], k[:, cut], v[:, cut], S, d, S)
    assert np.allclose(out[:, cut], small, atol=1e-12)
