"""CPU oracle for attention under the prefix-shared training mask -- TEST INFRASTRUCTURE ONLY.

Section 3.3 ("Prefix-shared masked training") and Appendix B: one packed row holds `prompt_len`
clean positions followed by one block of `draft_len` masked positions per prefix position; a
single forward pass trains all prefixes because block n may read only prompt slots 0..n and,
causally, itself.  This file is the plain definition: for every query slot, softmax over the key
slots that `oracle.mask.training_visible` allows, in fp64, one row at a time, grouped-query heads
as in the inference step.  A query slot that may read nothing (beyond the sequence's length)
gives a zero row (reading: the paper's sparse-attention library skips fully masked rows).
"""
from __future__ import annotations

import math

import numpy as np

from .mask import training_visible


def training_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, prompt_len: int, draft_len: int, seq_len: int,
                       query_slots=None) -> np.ndarray:
    """q: [H_q, L, d_h]; k, v: [H_kv, L, d_h] with L = prompt_len * (1 + draft_len), fp64.
    Returns softmax(q k^T / sqrt(d_h) over the visible slots) v, [H_q, L, d_h].
    query_slots: compute only these query slots (the other rows of the result stay zero) -- rows are
    independent of one another, so a long packed row can be checked on a sample of its slots."""
    Hq, L, dh = q.shape
    Hkv = k.shape[0]
    assert L == prompt_len * (1 + draft_len) and Hq % Hkv == 0
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(dh)
    out = np.zeros((Hq, L, dh), dtype=np.float64)
    for qi in (range(L) if query_slots is None else query_slots):
        vis = np.array([training_visible(qi, ki, prompt_len, draft_len, seq_len) for ki in range(L)], dtype=bool)
        if not vis.any():
            continue
        for j in range(Hq):
            kk, vv = k[j // G][vis], v[j // G][vis]
            sc = (kk @ q[j, qi]) * scale
            sc = sc - sc.max()
            p = np.exp(sc)
            out[j, qi] = (p / p.sum()) @ vv
    return out
