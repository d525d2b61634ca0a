"""CPU oracle for continuity-aware tree pruning -- TEST INFRASTRUCTURE ONLY.

Algorithm 1 taken step by step in the paper's order and notation, with the scores of
Appendix D.  Tree pruning is a heuristic (beam search), so the oracle *is* the algorithm:
all score arithmetic is IEEE fp32, one rounded operation at a time (numpy float32
scalars), so that a correct GPU implementation can match it bit for bit.

Readings where the paper is silent (all deterministic total orders, so that the
"in parallel" expansion of Algorithm 1 cannot change the result):
  * level is 0-based: the first drafted token has w_logit = 1 and w_level = 1;
  * g_n: the trigram row (a, b, t) if the table has it, else the bigram row (b, t),
    else log(eps_ng);
  * top-w: score descending, ties to the earlier generated candidate;
  * final top-theta: theta = budget - 1 (the budget counts the root); a node's score is
    clamped by its ancestors' (min along the path) so the selection is a tree for any
    input; ties to the shallower, then the earlier generated node.
"""
from __future__ import annotations

import math
from typing import Dict, Tuple

import numpy as np

f32 = np.float32


def level_constants(d: int, logit_decay, level_exp, eps_ng) -> Tuple[np.ndarray, np.ndarray, np.float32]:
    """w_logit = decay^level, w_level = (level+1)^-exp, log(eps): fp64 from the fp32 settings, then fp32."""
    dec, ex, ep = float(f32(logit_decay)), float(f32(level_exp)), float(f32(eps_ng))
    wl = np.array([f32(math.pow(dec, i)) for i in range(d)], dtype=f32)
    wv = np.array([f32(math.pow(float(i + 1), -ex)) for i in range(d)], dtype=f32)
    return wl, wv, f32(math.log(ep))


def ngram_score(tri: Dict, bi: Dict, a: int, b: int, t: int, miss: np.float32) -> np.float32:
    """s_ng = log(Pr(t | context) + eps) read from the table, backing off 3-gram -> 2-gram -> miss."""
    if a >= 0 and b >= 0 and (a, b, t) in tri:
        return f32(tri[(a, b, t)])
    if b >= 0 and (b, t) in bi:
        return f32(bi[(b, t)])
    return miss


def tables_from_rows(rows: Dict[str, np.ndarray]) -> Tuple[Dict, Dict]:
    """Row arrays (order, ctx0, ctx1, next, score) -> lookup dicts; the first duplicate wins."""
    tri: Dict = {}
    bi: Dict = {}
    for o, c0, c1, nx, s in zip(rows["order"].tolist(), rows["ctx0"].tolist(), rows["ctx1"].tolist(),
                                rows["next"].tolist(), rows["score"].tolist()):
        if o == 3:
            tri.setdefault((c0, c1, nx), s)
        else:
            bi.setdefault((c1, nx), s)
    return tri, bi


def build_tree(ids: np.ndarray, slogit: np.ndarray, ctx: Tuple[int, int], tri: Dict, bi: Dict, *,
               beam: int, budget: int, w_ng=0.5, logit_decay=0.9, level_exp=0.7,
               eps_ng=1e-10) -> Dict[str, np.ndarray]:
    """Algorithm 1 for one sequence.

    ids, slogit: [d, k] candidate tokens S_i and their s_logit in the order the top-k step
    emitted them.  ctx = (c_-2, c_-1), the last two known tokens (-1 = absent).
    Returns tokens/parents/depth [budget], mask [budget, budget] (ancestor-or-self), n_nodes,
    plus 'scores' (clamped, fp32) for inspection.
    """
    d, k = ids.shape
    wl, wv, miss = level_constants(d, logit_decay, level_exp, eps_ng)
    wn = f32(w_ng)
    # node arrays; node 0 is the root (the last known token, score 0, level -1)
    tok = [int(ctx[1])]
    par = [-1]
    lvl = [-1]
    score = [f32(0.0)]
    prev = [int(ctx[0])]          # token before this node on its path
    C = [0]                       # active candidate set: node indices, in beam-rank order
    for i in range(d):            # Algorithm 1 line 3
        Cp = []
        for node in C:            # line 5 (sequential here; the order only fixes 'gen')
            a, b, sc = prev[node], tok[node], score[node]
            for j in range(k):    # lines 6-7
                t = int(ids[i, j])
                s_logit = f32(slogit[i, j])                               # line 8
                s_ng = ngram_score(tri, bi, a, b, t, miss)                 # line 9
                inc = f32(f32(f32(wl[i] * s_logit) + f32(wn * s_ng)) * wv[i])   # Combine, Appendix D
                s_new = f32(sc + inc)                                      # line 10
                tok.append(t); par.append(node); lvl.append(i); score.append(s_new); prev.append(b)
                Cp.append(len(tok) - 1)                                    # lines 11-12 (node index = gen)
        Cp.sort(key=lambda n: (-float(score[n]), n))                      # line 15
        C = Cp[:beam]
    n_all = len(tok)
    clamped = [f32(np.inf)] * n_all
    for n in range(1, n_all):     # parents always precede children
        clamped[n] = score[n] if score[n] < clamped[par[n]] else clamped[par[n]]
    theta = budget - 1
    order = sorted(range(1, n_all), key=lambda n: (-float(clamped[n]), lvl[n], n))[:theta]   # line 18
    out_index = {0: 0}
    for x, n in enumerate(order):
        out_index[n] = x + 1
    tokens = np.full(budget, -1, dtype=np.int32)
    parents = np.full(budget, -1, dtype=np.int32)
    depth = np.full(budget, -1, dtype=np.int32)
    mask = np.zeros((budget, budget), dtype=np.uint8)
    scores = np.full(budget, -np.inf, dtype=np.float32)
    tokens[0], depth[0], mask[0, 0], scores[0] = tok[0], 0, 1, 0.0
    for n in order:
        x = out_index[n]
        tokens[x], parents[x], depth[x], scores[x] = tok[n], out_index[par[n]], lvl[n] + 1, clamped[n]
        mask[x, x] = 1
        p = par[n]
        while p >= 0:
            mask[x, out_index[p]] = 1
            p = par[p]
    return {"tokens": tokens, "parents": parents, "depth": depth, "mask": mask,
            "n_nodes": np.int32(1 + len(order)), "scores": scores, "n_scored": n_all - 1}


def verification_inputs(parents: np.ndarray, depth: np.ndarray, n_nodes: int, root_pos: int, max_levels: int) -> Dict[str, np.ndarray]:
    """What the target model needs to verify a draft tree in one forward pass with tree attention (Section 3,
    Figure 2: the draft tree is verified "with Tree Attention"; the tree-attention mask itself is build_tree's
    `mask`).  Reading (the paper names the step, not its encoding): node x sits at absolute position
    root_pos + depth[x], root_pos being the position of the root token c_-1; a candidate continuation is a
    root-to-leaf path, listed as the slots of its nodes.
      position_ids [budget]           root_pos + depth[x] for the n_nodes used slots, -1 elsewhere
      retrieve     [budget, L+1]      row j = the slots of the j-th leaf's path, root first, padded with -1;
                                      leaves in ascending slot order; unused rows all -1
      n_leaves                        number of leaves (used slots that are nobody's parent)"""
    budget = parents.shape[0]
    pos = np.full((budget,), -1, dtype=np.int32)
    pos[:n_nodes] = root_pos + depth[:n_nodes]
    is_parent = np.zeros((budget,), dtype=bool)
    for x in range(1, n_nodes):
        is_parent[parents[x]] = True
    retrieve = np.full((budget, max_levels + 1), -1, dtype=np.int32)
    n_leaves = 0
    for x in range(n_nodes):
        if is_parent[x]:
            continue
        path = []
        y = x
        while y >= 0:
            path.append(y)
            y = int(parents[y])
        path.reverse()
        retrieve[n_leaves, :len(path)] = path
        n_leaves += 1
    return {"position_ids": pos, "retrieve": retrieve, "n_leaves": np.int32(n_leaves)}
