"""Seeded synthetic inputs for the DART drafting step.

This module only *draws* inputs (weights, hidden states, KV cache, token ids,
N-gram rows) with the shapes and distributions of the paper's Qwen3 workloads
(Section 5.1, Appendix B, Appendix D).  It contains none of the method's
arithmetic: both the CUDA library and the CPU oracle consume the arrays it
returns, and neither is imported here.

Tensor #n derives its generator seeds from ``seed + n`` so that a single tensor can be
regenerated without the others (large tensors use one generator per 2^24-element chunk).
"""
from __future__ import annotations

import dataclasses
import math
import os
from typing import Dict, Optional

import numpy as np
import torch

BASE_SEED = 1234

# draw order (seed offset) of every tensor
_ORDER = [
    "w_fc", "embed", "mask_vec", "norm_g", "norm_e", "w_q", "w_k", "w_v", "w_o",
    "norm_post", "w_gate", "w_up", "w_down", "norm_final", "w_lm", "feats",
    "tokens", "k_cache", "v_cache", "seq_lens", "ngram", "ctx_tail",
]
SEED_OFFSET = {name: i for i, name in enumerate(_ORDER)}


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape of one drafting workload (Appendix B: layer aligned with the target)."""

    name: str
    batch: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    mlp_inter: int
    vocab: int
    prefix: int            # fixed prefix length, or upper bound when ragged
    K: int                 # query rows per sequence = future positions d
    tree_budget: int       # nodes including the root
    ngram_rows: int
    ngram_mode: str        # "uniform_bigram" | "zipf_mixed"
    ragged_lo: int = 0     # >0: prefix lengths drawn U[ragged_lo, prefix]
    temperature: float = 0.0
    topk: int = 25         # k_i, Appendix D
    beam: int = 20         # w, Appendix D
    n_fresh: int = 1       # rows per sequence that carry fresh target features

    @property
    def max_prefix(self) -> int:
        return self.prefix + self.K

    @property
    def feat_in(self) -> int:
        return 3 * self.hidden


WORKLOADS: Dict[str, Workload] = {
    "C1": Workload("C1", 1, 256, 4, 2, 64, 688, 4096, 128, 4, 16, 20_000, "uniform_bigram"),
    "C2": Workload("C2", 1, 4096, 32, 8, 128, 12288, 151936, 2048, 8, 60, 1_000_000, "zipf_mixed"),
    "C3": Workload("C3", 1, 5120, 40, 8, 128, 17408, 151936, 4096, 8, 60, 1_000_000, "zipf_mixed"),
    "C4": Workload("C4", 4, 5120, 64, 8, 128, 25600, 151936, 8192, 8, 60, 1_000_000, "zipf_mixed"),
    "C5": Workload("C5", 16, 5120, 40, 8, 128, 17408, 151936, 8192, 8, 60, 4_000_000, "zipf_mixed",
                   ragged_lo=512, temperature=1.0),
}


def small_variant(w: Workload, **kw) -> Workload:
    """A workload with some fields replaced (used by tests for odd shapes)."""
    return dataclasses.replace(w, **kw)


def _gen(seed: int, name: str) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed + SEED_OFFSET[name])
    return g


def _randn_bf16(shape, gen, scale=1.0, shift=0.0, chunk=1 << 24) -> torch.Tensor:
    """N(shift, scale^2) rounded to bf16 (round-to-nearest-even).

    Large tensors are drawn in chunks of 2^24 elements, chunk c from its own generator seeded
    with ``gen.initial_seed() + 7919 * (c + 1)``, so that the chunks can be drawn by a few
    threads at once; the result does not depend on the number of threads.
    """
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16)
    base = gen.initial_seed()

    def draw(c: int) -> None:
        s, e = c * chunk, min(n, (c + 1) * chunk)
        g = torch.Generator(device="cpu")
        g.manual_seed(base + 7919 * (c + 1))
        t = torch.randn(e - s, generator=g, dtype=torch.float32)
        if scale != 1.0:
            t.mul_(scale)
        if shift != 0.0:
            t.add_(shift)
        out[s:e] = t.to(torch.bfloat16)

    n_chunks = (n + chunk - 1) // chunk
    if n_chunks <= 1:
        draw(0) if n else None
    else:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
            list(ex.map(draw, range(n_chunks)))
    return out.view(*shape)


class ZipfSampler:
    """Token ids with p(rank r) proportional to r^-1.1, rank r -> id r-1."""

    def __init__(self, vocab: int, a: float = 1.1):
        p = np.arange(1, vocab + 1, dtype=np.float64) ** (-a)
        self.cdf = np.cumsum(p)
        self.cdf /= self.cdf[-1]
        self.vocab = vocab

    def draw(self, n: int, gen: torch.Generator) -> np.ndarray:
        u = torch.rand(n, generator=gen, dtype=torch.float64).numpy()
        ids = np.searchsorted(self.cdf, u, side="left")
        return np.minimum(ids, self.vocab - 1).astype(np.int32)


def make_weights(w: Workload, seed: int = BASE_SEED, only: Optional[set] = None) -> Dict[str, torch.Tensor]:
    """Random-init draft weights, bf16, row-major [out, in] (Appendix B 'trainable parameters')."""
    h, dq, dkv = w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim
    shapes = {
        "w_fc": (h, 3 * h), "embed": (w.vocab, h), "mask_vec": (2 * h,),
        "norm_g": (h,), "norm_e": (h,),
        "w_q": (dq, 2 * h), "w_k": (dkv, 2 * h), "w_v": (dkv, 2 * h), "w_o": (h, dq),
        "norm_post": (h,), "w_gate": (w.mlp_inter, h), "w_up": (w.mlp_inter, h),
        "w_down": (h, w.mlp_inter), "norm_final": (h,), "w_lm": (w.vocab, h),
    }
    out = {}
    for name, shape in shapes.items():
        if only is not None and name not in only:
            continue
        g = _gen(seed, name)
        if name.startswith("norm_"):
            out[name] = _randn_bf16(shape, g, scale=0.02, shift=1.0)
        elif name == "mask_vec":
            out[name] = _randn_bf16(shape, g, scale=1.0)
        else:
            out[name] = _randn_bf16(shape, g, scale=0.02)
    return out


def make_seq_lens(w: Workload, seed: int = BASE_SEED) -> np.ndarray:
    if w.ragged_lo > 0:
        g = _gen(seed, "seq_lens")
        return torch.randint(w.ragged_lo, w.prefix + 1, (w.batch,), generator=g).numpy().astype(np.int32)
    return np.full((w.batch,), w.prefix, dtype=np.int32)


def make_step_inputs(w: Workload, seed: int = BASE_SEED, n_fresh=None) -> Dict[str, object]:
    """Per-step inputs: target features, next-token ids, prefix KV cache, lengths, context tail.
    n_fresh: one count for every sequence, or a list of per-sequence counts (see make_ragged_step_inputs)."""
    if n_fresh is not None and not isinstance(n_fresh, (int, np.integer)):
        return make_ragged_step_inputs(w, list(n_fresh), seed)
    F = w.n_fresh if n_fresh is None else n_fresh
    B = w.batch
    zipf = ZipfSampler(w.vocab)
    feats = _randn_bf16((B, max(F, 1), 3 * w.hidden), _gen(seed, "feats"))[:, :F].contiguous()
    tokens = zipf.draw(B * max(F, 1), _gen(seed, "tokens")).reshape(B, max(F, 1))[:, :F].copy()
    seq_lens = make_seq_lens(w, seed)
    P_cap = w.max_prefix
    k_cache = torch.zeros(B, w.n_kv_heads, P_cap, w.head_dim, dtype=torch.bfloat16)
    v_cache = torch.zeros_like(k_cache)
    for b in range(B):
        P = int(seq_lens[b])
        k_cache[b, :, :P] = _randn_bf16((w.n_kv_heads, P, w.head_dim), _gen(seed + 100 * b, "k_cache"))
        v_cache[b, :, :P] = _randn_bf16((w.n_kv_heads, P, w.head_dim), _gen(seed + 100 * b, "v_cache"))
    ctx_first = zipf.draw(B, _gen(seed, "ctx_tail"))
    ctx_tail = np.empty((B, 2), dtype=np.int32)
    ctx_tail[:, 0] = ctx_first
    ctx_tail[:, 1] = tokens[:, F - 1] if F > 0 else zipf.draw(B, _gen(seed + 1000, "ctx_tail"))
    return {
        "feats": feats, "tokens": torch.from_numpy(tokens.astype(np.int32)),
        "seq_lens": torch.from_numpy(seq_lens), "k_cache": k_cache, "v_cache": v_cache,
        "ctx_tail": torch.from_numpy(ctx_tail), "n_fresh": F,
    }


def draw_fresh_counts(w: Workload, seed: int = BASE_SEED, mean_accept: float = 3.5) -> list:
    """Per-sequence fresh-row counts of a steady-state call: one row for the token the target just sampled
    plus the draft tokens the last verification accepted, a geometric number with the given mean (the paper
    reports mean acceptance lengths of roughly 3 to 4 tokens per step), capped at K rows."""
    g = _gen(seed + 19, "tokens")
    u = torch.rand(w.batch, generator=g).numpy()
    q = 1.0 - 1.0 / max(mean_accept, 1.0)                      # P(accept one more)
    extra = np.floor(np.log(np.maximum(u, 1e-12)) / np.log(max(q, 1e-12))).astype(np.int64) if q > 0 else np.zeros(w.batch, np.int64)
    return [int(min(w.K, 1 + e)) for e in extra]


def make_ragged_step_inputs(w: Workload, fresh_counts, seed: int = BASE_SEED) -> Dict[str, object]:
    """The steady-state call after a verification that accepted a different number of tokens per sequence:
    sequence b has fresh_counts[b] fresh rows (0..K).  Every sequence draws K rows of features and tokens
    exactly as the uniform generator with n_fresh = K would, then keeps its first fresh_counts[b]; the kept
    rows are packed in sequence order: feats [sum F_b, 3h], tokens [sum F_b].  "n_fresh" is the list."""
    assert len(fresh_counts) == w.batch and all(0 <= f <= w.K for f in fresh_counts)
    full = make_step_inputs(w, seed, n_fresh=w.K)
    keep_f = [full["feats"][b, :f] for b, f in enumerate(fresh_counts)]
    keep_t = [full["tokens"][b, :f] for b, f in enumerate(fresh_counts)]
    out = dict(full)
    out["feats"] = torch.cat(keep_f, 0).contiguous()
    out["tokens"] = torch.cat(keep_t, 0).contiguous()
    ctx = full["ctx_tail"].clone()
    alt = ZipfSampler(w.vocab).draw(w.batch, _gen(seed + 1000, "ctx_tail"))
    for b, f in enumerate(fresh_counts):
        ctx[b, 1] = int(full["tokens"][b, f - 1]) if f > 0 else int(alt[b])
    out["ctx_tail"] = ctx
    out["n_fresh"] = [int(f) for f in fresh_counts]
    return out


def make_ngram_rows(vocab: int, n_rows: int, mode: str, seed: int = BASE_SEED,
                    eps: float = 1e-10, extra_rows: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Rows of a synthetic 2/3-gram table standing in for the Dolma 3-gram (Appendix C).

    Each row is (order, ctx0, ctx1, next) with a log-count U(0,5).  Counts are turned
    into per-context probabilities Pr and the row stores fp32(log(Pr + eps)), computed in
    fp64: the table value *is* s_ng of Appendix D for that row.  ``ctx0`` is -1 for a bigram.
    ``extra_rows`` (int array [m,4] of order,ctx0,ctx1,next) are appended before de-duplication.
    """
    g = _gen(seed, "ngram")
    if mode == "uniform_bigram":
        toks = torch.randint(0, vocab, (n_rows, 2), generator=g).numpy().astype(np.int64)
        order = np.full(n_rows, 2, dtype=np.int64)
        c0 = np.full(n_rows, -1, dtype=np.int64)
        c1, nx = toks[:, 0], toks[:, 1]
    elif mode == "zipf_mixed":
        zipf = ZipfSampler(vocab)
        toks = zipf.draw(3 * n_rows, g).reshape(n_rows, 3).astype(np.int64)
        order = np.where(np.arange(n_rows) < n_rows // 2, 2, 3).astype(np.int64)
        c0 = np.where(order == 3, toks[:, 0], -1)
        c1, nx = toks[:, 1], toks[:, 2]
    else:
        raise ValueError(mode)
    if extra_rows is not None and len(extra_rows):
        ex = np.asarray(extra_rows, dtype=np.int64)
        order = np.concatenate([order, ex[:, 0]])
        c0 = np.concatenate([c0, ex[:, 1]])
        c1 = np.concatenate([c1, ex[:, 2]])
        nx = np.concatenate([nx, ex[:, 3]])
    n = len(order)
    logcount = torch.rand(n, generator=g, dtype=torch.float64).numpy() * 5.0
    # de-duplicate (keep the first occurrence of a (order, ctx, next) row)
    V1 = vocab + 1
    ctx_key = (order - 2) * V1 * V1 + (c0 + 1) * V1 + c1
    full_key = ctx_key * vocab + nx
    _, first = np.unique(full_key, return_index=True)
    first.sort()
    order, c0, c1, nx, logcount, ctx_key = (a[first] for a in (order, c0, c1, nx, logcount, ctx_key))
    # per-context normalisation of the counts
    _, inv = np.unique(ctx_key, return_inverse=True)
    cnt = np.exp(logcount)
    tot = np.bincount(inv, weights=cnt)
    pr = cnt / tot[inv]
    score = np.log(pr + eps).astype(np.float32)
    return {
        "order": order.astype(np.uint8), "ctx0": c0.astype(np.int32), "ctx1": c1.astype(np.int32),
        "next": nx.astype(np.int32), "score": score,
    }


def make_tree_inputs(vocab: int, batch: int, levels: int, k: int, seed: int = BASE_SEED,
                     eps: float = 1e-10) -> Dict[str, np.ndarray]:
    """Stand-alone inputs for the tree builder: per level k distinct Zipf ids and the k largest
    values of a log-softmax over 4096 draws of N(0, 2^2), passed through log(exp(.)+eps)."""
    g = _gen(seed, "ctx_tail")
    g.manual_seed(seed + 7777)
    zipf = ZipfSampler(vocab)
    ids = np.empty((batch, levels, k), dtype=np.int32)
    sl = np.empty((batch, levels, k), dtype=np.float32)
    for b in range(batch):
        for i in range(levels):
            seen: list = []
            while len(seen) < k:
                for t in zipf.draw(2 * k, g):
                    if int(t) not in seen:
                        seen.append(int(t))
                        if len(seen) == k:
                            break
            ids[b, i] = np.asarray(seen, dtype=np.int32)
            x = torch.randn(4096, generator=g, dtype=torch.float64).numpy() * 2.0
            lp = x - (np.log(np.sum(np.exp(x - x.max()))) + x.max())
            top = np.sort(lp)[::-1][:k]
            sl[b, i] = np.log(np.exp(top) + eps).astype(np.float32)
    ctx = zipf.draw(2 * batch, g).reshape(batch, 2).astype(np.int32)
    return {"ids": ids, "slogit": sl, "ctx_tail": ctx}


def algorithmic_bytes(w: Workload, seq_lens: np.ndarray, with_fc: bool = True) -> int:
    """bf16 weights read once + prefix KV read once (activations, norms, outputs ignored)."""
    h, dq, dkv, I, V = w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.mlp_inter, w.vocab
    elems = 2 * h * dq + 2 * 2 * h * dkv + dq * h + 3 * h * I + V * h
    if with_fc:
        elems += 3 * h * h
    kv = int(np.sum(seq_lens.astype(np.int64))) * 2 * dkv * 2
    return 2 * elems + kv


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """View a bf16 torch tensor as a numpy uint16 array of its bit patterns (no copy)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)
