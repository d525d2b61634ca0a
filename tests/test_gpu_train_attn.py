"""dart_train_attention_fwd against the oracle's plain statement of attention under the prefix-shared training mask
(Section 3.3, Appendix B): every output element, several query tiles per head, ragged lengths, draft lengths that do
and do not divide the 128-row tile, sharp and flat softmaxes."""
import numpy as np
import pytest
import torch

from oracle import train_attention as ota
from paper_2601_19278_b200 import binding

pytestmark = pytest.mark.gpu

ATOL, RTOL = 2e-2, 1e-2     # bf16 inputs, bf16 probabilities and bf16 output against fp64


def _run(B, Hq, Hkv, Lp, d, seq_lens, seed, q_scale=1.0):
    dh = 128
    L = Lp * (1 + d)
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn(B, Hq, L, dh, generator=g) * q_scale).to(torch.bfloat16)
    k = torch.randn(B, Hkv, L, dh, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, L, dh, generator=g).to(torch.bfloat16)
    dev = torch.device("cuda:0")
    out = torch.full((B, Hq, L, dh), float("nan"), dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.train_attention_fwd(q.to(dev), k.to(dev), v.to(dev), seq_lens, Lp, d, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = out.float().cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any(), "a row was not written"
    worst = 0.0
    for b in range(B):
        ref = ota.training_attention(q[b].double().numpy(), k[b].double().numpy(), v[b].double().numpy(), Lp, d, int(seq_lens[b]))
        err = np.abs(got[b] - ref)
        assert np.all(err <= ATOL + RTOL * np.abs(ref)), (b, float(err.max()))
        worst = max(worst, float(err.max()))
        S = int(seq_lens[b])
        assert np.all(got[b][:, S:Lp] == 0) and np.all(got[b][:, Lp + S * d:] == 0)     # slots past the length: exact zeros
    return worst


def test_several_tiles_ragged_lengths_d8():
    _run(2, 4, 2, 200, 8, [200, 137], seed=0)


def test_draft_length_that_does_not_divide_the_tile():
    _run(2, 2, 1, 150, 3, [150, 1], seed=1)


def test_d1_and_an_empty_sequence():
    _run(2, 2, 2, 130, 1, [0, 130], seed=2)


def test_odd_group_of_query_heads():
    _run(1, 6, 2, 70, 8, [66], seed=6)          # three query heads per KV head: a pair and a single per CTA row


def test_one_prompt_slot():
    _run(1, 2, 1, 1, 8, [1], seed=3)


def test_long_blocks_d16():
    _run(1, 4, 4, 40, 16, [33], seed=4)


def test_sharp_softmax_moves_the_reference_maximum():
    _run(1, 2, 1, 300, 4, [300], seed=5, q_scale=6.0)


def test_long_packed_row_on_sampled_query_slots():
    """A packed row of the size the kernel is timed on has tens of thousands of slots; the oracle (one visibility
    test per slot pair) checks a seeded sample of query slots from every region of the mask: clean slots, the first
    and last masked blocks, blocks in the middle, block boundaries, the last valid slots and slots past the length."""
    B, Hq, Hkv, Lp, d, dh = 1, 10, 2, 1100, 8, 128          # groups of five query heads, as at the 14B shape
    S = 1063                                                 # valid prompt slots: the tail of the row reads nothing
    L = Lp * (1 + d)
    g = torch.Generator().manual_seed(21)
    q = torch.randn(B, Hq, L, dh, generator=g).to(torch.bfloat16)
    k = torch.randn(B, Hkv, L, dh, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, L, dh, generator=g).to(torch.bfloat16)
    dev = torch.device("cuda:0")
    out = torch.full((B, Hq, L, dh), float("nan"), dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.train_attention_fwd(q.to(dev), k.to(dev), v.to(dev), [S], Lp, d, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = out[0].float().cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    rng = np.random.default_rng(22)
    block = lambda n: list(range(Lp + n * d, Lp + (n + 1) * d))
    slots = [0, 1, 63, 64, 127, 128, 129, S - 1, S, Lp - 1]                                   # clean part, tile edges, length cut
    slots += block(0) + block(1) + block(15) + block(16) + block(S - 1) + block(S) + block(Lp - 1)
    slots += rng.integers(0, S, 24).tolist()                                                  # random clean slots
    slots += [Lp + int(n) * d + int(r) for n, r in zip(rng.integers(0, S, 40), rng.integers(0, d, 40))]   # random block slots
    slots = sorted(set(slots))
    ref = ota.training_attention(q[0].double().numpy(), k[0].double().numpy(), v[0].double().numpy(), Lp, d, S, query_slots=slots)
    err = np.abs(got[:, slots] - ref[:, slots])
    assert np.all(err <= ATOL + RTOL * np.abs(ref[:, slots])), float(err.max())
    assert np.abs(ref[:, slots]).max() > 0.1
    assert np.all(got[:, S:Lp] == 0) and np.all(got[:, Lp + S * d:] == 0)


def test_argument_errors():
    dev = torch.device("cuda:0")
    B, Hq, Hkv, Lp, d, dh = 1, 2, 1, 16, 8, 128
    L = Lp * (1 + d)
    q = torch.zeros(B, Hq, L, dh, dtype=torch.bfloat16, device=dev)
    k = torch.zeros(B, Hkv, L, dh, dtype=torch.bfloat16, device=dev)
    out = torch.zeros_like(q)
    with pytest.raises(binding.DartError) as e:
        binding.train_attention_fwd(q, k, k, [Lp + 1], Lp, d, out)
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    with pytest.raises(binding.DartError) as e:
        binding.train_attention_fwd(q, k, k, [Lp], Lp, 17, out)
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    with pytest.raises(binding.DartError) as e:
        binding.train_attention_fwd(q[:, :, :, :64].contiguous(), k, k, [Lp], Lp, d, out)
    assert e.value.status == binding.DART_ERR_INVALID_ARG
    torch.cuda.synchronize()
