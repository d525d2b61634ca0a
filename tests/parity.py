"""Shared helpers of the GPU parity tests: run the oracle on a workload's inputs and compare
the CUDA library's outputs with it under the stated tolerances.

Tolerances (bf16 weights, fp32 accumulate, against the fp64 oracle):
  logits and top-k log-probs: max-abs error <= 2e-2 and relative L2 error per row <= 1e-2;
  trees from identical (ids, s_logit): bit-exact.
"""
from __future__ import annotations

import os
import sys
from typing import Dict, Optional

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import forward as ofw          # noqa: E402
from oracle import tree as otree           # noqa: E402
from paper_2601_19278_b200 import synthetic as syn   # noqa: E402

TOL_ABS = 2e-2
TOL_REL = 1e-2
PHILOX_SEED = 1234


def oracle_cfg(w: syn.Workload) -> Dict:
    return dict(hidden=w.hidden, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim, K=w.K,
                rope_theta=1e6, rms_eps=1e-6)


def np_weights(wt) -> Dict[str, np.ndarray]:
    return {k: syn.bf16_bits(v) for k, v in wt.items()}


def np_inputs(inp) -> Dict[str, object]:
    return {"feats": syn.bf16_bits(inp["feats"]), "tokens": inp["tokens"].numpy(), "seq_lens": inp["seq_lens"].numpy(),
            "k_cache": syn.bf16_bits(inp["k_cache"]), "v_cache": syn.bf16_bits(inp["v_cache"]), "n_fresh": inp["n_fresh"]}


def oracle_forward(w: syn.Workload, wt, inp) -> Dict[str, np.ndarray]:
    return ofw.draft_forward(oracle_cfg(w), np_weights(wt), np_inputs(inp))


def check_logits(got: np.ndarray, ref: np.ndarray) -> Dict[str, float]:
    """got fp32 [B,K,V] from the GPU, ref fp64 from the oracle."""
    got = got.astype(np.float64)
    err = np.abs(got - ref)
    max_abs = float(err.max())
    rel = np.linalg.norm((got - ref).reshape(-1, ref.shape[-1]), axis=1) / np.linalg.norm(ref.reshape(-1, ref.shape[-1]), axis=1)
    assert np.isfinite(got).all()
    assert max_abs <= TOL_ABS, f"logits max-abs error {max_abs}"
    assert float(rel.max()) <= TOL_REL, f"logits relative L2 error {rel.max()}"
    return {"max_abs": max_abs, "rel_l2": float(rel.max())}


def check_topk_row(ids_g: np.ndarray, sl_g: np.ndarray, logits_ref_row: np.ndarray, k: int, eps: float,
                   temperature: float = 0.0, noise: Optional[np.ndarray] = None) -> float:
    """Near-tie-tolerant comparison of one row's candidates (several answers are correct when two
    selection values differ by less than the tolerance)."""
    c = ofw.topk_candidates(logits_ref_row, k, eps, temperature, noise)
    sel, lp = c["sel"], c["lp"]
    kk = len(c["ids"])
    assert len(set(ids_g.tolist())) == kk and ids_g.min() >= 0, "candidate ids must be distinct and valid"
    s_ref = np.log(np.exp(lp[ids_g]) + eps)
    err = float(np.abs(sl_g.astype(np.float64) - s_ref).max())
    assert err <= TOL_ABS, f"s_logit error {err}"
    assert np.linalg.norm(sl_g - s_ref) / np.linalg.norm(s_ref) <= TOL_REL
    kth = sel[c["ids"][-1]]
    assert np.all(sel[ids_g] >= kth - TOL_ABS), "a picked token is not within tolerance of the top-k"
    must = np.nonzero(sel > kth + TOL_ABS)[0]
    assert set(must.tolist()) <= set(ids_g.tolist()), "a clearly-top token is missing"
    assert np.all(np.diff(sel[ids_g]) <= TOL_ABS), "candidates are not in descending order"
    return err


def oracle_tree_batch(ids: np.ndarray, sl: np.ndarray, ctx: np.ndarray, tri, bi, *, beam: int, budget: int,
                      **kw) -> Dict[str, np.ndarray]:
    outs = [otree.build_tree(ids[b], sl[b], (int(ctx[b, 0]), int(ctx[b, 1])), tri, bi, beam=beam, budget=budget, **kw)
            for b in range(ids.shape[0])]
    return {k: np.stack([np.asarray(o[k]) for o in outs]) for k in ("tokens", "parents", "depth", "mask", "n_nodes", "scores")}


def assert_tree_equal(got: Dict[str, np.ndarray], ref: Dict[str, np.ndarray]) -> None:
    for key in ("n_nodes", "tokens", "parents", "depth", "mask"):
        assert np.array_equal(got[key], ref[key]), f"tree field {key} differs"
    assert np.array_equal(got["scores"].view(np.uint32), ref["scores"].astype(np.float32).view(np.uint32)), "scores differ bitwise"
