"""Pins for the tree-pruning oracle (Algorithm 1, Appendix D): brute-force enumeration on tiny
inputs, degenerate settings with an obvious answer, hand-worked score values, and the
structural invariants any draft tree must satisfy."""
import itertools
import math

import numpy as np
import pytest

from oracle import tree as otree
from paper_2601_19278_b200 import synthetic as syn

f32 = np.float32


def _rand_case(rng, V, d, k, n_tri=40, n_bi=20):
    ids = np.stack([rng.permutation(V)[:k] for _ in range(d)]).astype(np.int32)
    sl = -np.sort(rng.random((d, k)).astype(np.float32) * 6, axis=1)
    tri = {tuple(rng.integers(0, V, 3).tolist()): float(f32(-rng.random() * 4)) for _ in range(n_tri)}
    bi = {tuple(rng.integers(0, V, 2).tolist()): float(f32(-rng.random() * 4)) for _ in range(n_bi)}
    ctx = tuple(rng.integers(0, V, 2).tolist())
    return ids, sl, ctx, tri, bi


def _brute_force(ids, sl, ctx, tri, bi, budget):
    """Every path of the full d-level tree, scored by the same sequential fp32 sums, clamped
    along the path, globally sorted.  No beam, no generation order: valid when scores are distinct."""
    d, k = ids.shape
    nodes = []                                   # (clamped score, path tokens)
    miss = f32(math.log(float(f32(1e-10))))
    for depth in range(1, d + 1):
        for js in itertools.product(range(k), repeat=depth):
            seq = [ctx[0], ctx[1]]
            s = f32(0.0)
            clamp = f32(np.inf)
            for i, j in enumerate(js):
                t = int(ids[i, j])
                a, b = seq[-2], seq[-1]
                if (a, b, t) in tri:
                    ng = f32(tri[(a, b, t)])
                elif (b, t) in bi:
                    ng = f32(bi[(b, t)])
                else:
                    ng = miss
                w_logit = f32(math.pow(float(f32(0.9)), i))
                w_level = f32(math.pow(i + 1.0, -float(f32(0.7))))
                s = f32(s + f32(f32(f32(w_logit * f32(sl[i, j])) + f32(f32(0.5) * ng)) * w_level))
                clamp = min(clamp, s)
                seq.append(t)
            nodes.append((float(clamp), tuple(seq[2:])))
    nodes.sort(key=lambda n: -n[0])
    top = nodes[:budget - 1]
    scores = [n[0] for n in nodes[:budget]]
    assert len(set(scores)) == len(scores), "brute force needs distinct scores"
    return top


def _paths(out):
    res = []
    for x in range(1, int(out["n_nodes"])):
        p, path = x, []
        while p > 0:
            path.append(int(out["tokens"][p]))
            p = int(out["parents"][p])
        res.append(tuple(reversed(path)))
    return res


@pytest.mark.parametrize("seed,V,d,k,budget", [(0, 5, 3, 5, 12), (1, 4, 4, 4, 20), (2, 6, 3, 4, 9), (3, 5, 4, 3, 200)])
def test_tree_equals_brute_force_when_the_beam_never_prunes(seed, V, d, k, budget):
    rng = np.random.default_rng(seed)
    ids, sl, ctx, tri, bi = _rand_case(rng, V, d, k)
    out = otree.build_tree(ids, sl, ctx, tri, bi, beam=k ** d, budget=budget)
    top = _brute_force(ids, sl, ctx, tri, bi, budget)
    assert _paths(out) == [p for _, p in top]
    np.testing.assert_array_equal(out["scores"][1:1 + len(top)], np.array([s for s, _ in top], dtype=np.float32))
    assert int(out["n_nodes"]) == 1 + len(top)


def test_greedy_chain_when_beam_and_k_are_one():
    rng = np.random.default_rng(5)
    ids, sl, ctx, tri, bi = _rand_case(rng, 50, 6, 1)
    out = otree.build_tree(ids, sl, ctx, tri, bi, beam=1, budget=16)
    assert int(out["n_nodes"]) == 7
    assert out["tokens"][1:7].tolist() == ids[:, 0].tolist()
    assert out["parents"][:7].tolist() == [-1, 0, 1, 2, 3, 4, 5]
    assert out["depth"][:7].tolist() == list(range(7))
    assert np.array_equal(out["mask"][:7, :7], np.tril(np.ones((7, 7), dtype=np.uint8)))
    assert np.all(out["tokens"][7:] == -1) and np.all(out["mask"][7:] == 0)


def test_empty_table_and_zero_ngram_weight():
    rng = np.random.default_rng(6)
    ids, sl, ctx, tri, bi = _rand_case(rng, 30, 3, 6)
    # empty table: every candidate gets the same miss score, so each level is ordered by s_logit alone
    out = otree.build_tree(ids, sl, ctx, {}, {}, beam=4, budget=7)
    lvl1 = [int(out["tokens"][x]) for x in range(1, 7) if out["depth"][x] == 1]
    assert lvl1 == [int(t) for t in ids[0, :len(lvl1)]]
    # w_ng = 0 makes the table irrelevant
    a = otree.build_tree(ids, sl, ctx, tri, bi, beam=4, budget=12, w_ng=0.0)
    b = otree.build_tree(ids, sl, ctx, {}, {}, beam=4, budget=12, w_ng=0.0)
    for key in ("tokens", "parents", "depth", "mask"):
        assert np.array_equal(a[key], b[key])


def test_hand_worked_scores_and_backoff():
    """Two levels, two candidates, worked by hand with Appendix D's Combine:
    level 0: inc = (1*s_logit + 0.5*s_ng) * 1;  level 1: inc = (0.9*s_logit + 0.5*s_ng) * 2^-0.7."""
    ids = np.array([[7, 8], [9, 10]], dtype=np.int32)
    sl = np.array([[-0.5, -1.0], [-0.25, -2.0]], dtype=np.float32)
    ctx = (3, 4)
    tri = {(3, 4, 8): -0.125, (4, 7, 9): -1.0}       # trigram hits
    bi = {(7, 10): -0.5, (4, 7): -3.0, (4, 8): -9.0}  # (4,8) is shadowed by the trigram; (4,7) backs off
    out = otree.build_tree(ids, sl, ctx, tri, bi, beam=2, budget=7)
    miss = f32(math.log(float(f32(1e-10))))
    wl1, wv1 = f32(math.pow(float(f32(0.9)), 1)), f32(math.pow(2.0, -float(f32(0.7))))
    s7 = f32(f32(-0.5) + f32(f32(0.5) * f32(-3.0)))              # bigram back-off: -2.0
    s8 = f32(f32(-1.0) + f32(f32(0.5) * f32(-0.125)))            # trigram: -1.0625
    assert float(s7) == -2.0 and float(s8) == -1.0625
    s8_9 = f32(s8 + f32(f32(f32(wl1 * f32(-0.25)) + f32(f32(0.5) * miss)) * wv1))
    s7_9 = f32(s7 + f32(f32(f32(wl1 * f32(-0.25)) + f32(f32(0.5) * f32(-1.0))) * wv1))
    s7_10 = f32(s7 + f32(f32(f32(wl1 * f32(-2.0)) + f32(f32(0.5) * f32(-0.5))) * wv1))
    s8_10 = f32(s8 + f32(f32(f32(wl1 * f32(-2.0)) + f32(f32(0.5) * miss)) * wv1))
    expect = sorted([(s8, (8,)), (s7, (7,)), (s8_9, (8, 9)), (s7_9, (7, 9)), (s7_10, (7, 10)), (s8_10, (8, 10))],
                    key=lambda x: -float(x[0]))
    assert _paths(out) == [p for _, p in expect]
    assert [float(s) for s in out["scores"][1:7]] == [float(s) for s, _ in expect]
    assert abs(float(wv1) - 2 ** -0.7) < 1e-7 and abs(float(wl1) - 0.9) < 1e-7


def test_level_constants():
    wl, wv, miss = otree.level_constants(8, 0.9, 0.7, 1e-10)
    assert wl[0] == 1.0 and wv[0] == 1.0
    np.testing.assert_allclose(wl, 0.9 ** np.arange(8), rtol=1e-6)
    np.testing.assert_allclose(wv, (np.arange(8) + 1.0) ** -0.7, rtol=1e-6)
    assert abs(float(miss) - math.log(1e-10)) < 1e-5


def test_ties_go_to_the_earlier_generated_then_shallower_node():
    # all scores identical (zero logit scores, w_ng = 0): the order is purely generation order
    ids = np.array([[5, 6, 7], [1, 2, 3]], dtype=np.int32)
    sl = np.zeros((2, 3), dtype=np.float32)
    out = otree.build_tree(ids, sl, (0, 0), {}, {}, beam=2, budget=6, w_ng=0.0)
    # beam after level 0 = first two candidates (5, 6); final order: level 0 nodes first, then by generation
    assert out["tokens"][:6].tolist() == [0, 5, 6, 7, 1, 2]
    assert out["parents"][:6].tolist() == [-1, 0, 0, 0, 1, 1]
    # an under-full candidate set keeps everything
    out = otree.build_tree(ids[:1], sl[:1], (0, 0), {}, {}, beam=20, budget=60, w_ng=0.0)
    assert int(out["n_nodes"]) == 4


def test_positive_increments_cannot_orphan_a_node():
    """With (unphysical) positive scores a child can outscore its parent; clamping keeps the
    selection ancestor-closed."""
    ids = np.array([[1, 2], [3, 4], [5, 6]], dtype=np.int32)
    sl = np.array([[1.0, 0.5], [4.0, 0.1], [9.0, 0.2]], dtype=np.float32)
    out = otree.build_tree(ids, sl, (0, 0), {}, {}, beam=2, budget=5, w_ng=0.0)
    _check_invariants(out, ids, budget=5, beam=2)


def _check_invariants(out, ids, budget, beam):
    n = int(out["n_nodes"])
    d, k = ids.shape
    assert 1 <= n <= budget
    tok, par, dep, mask = out["tokens"], out["parents"], out["depth"], out["mask"]
    assert par[0] == -1 and dep[0] == 0
    for x in range(1, n):
        assert 0 <= par[x] < x                                  # parents precede children
        assert dep[x] == dep[par[x]] + 1
        assert tok[x] in ids[dep[x] - 1]                        # token at depth m comes from S_m
        assert out["scores"][x] <= out["scores"][par[x]] or par[x] == 0
        anc = {x}
        p = par[x]
        while p >= 0:
            anc.add(int(p)); p = par[p]
        assert set(np.nonzero(mask[x])[0].tolist()) == anc        # mask = ancestor-or-self
    for p in range(n):
        kids = [int(tok[x]) for x in range(1, n) if par[x] == p]
        assert len(kids) == len(set(kids))                        # siblings are distinct
    assert np.all(np.diff(out["scores"][1:n]) <= 0)
    assert np.all(tok[n:] == -1) and np.all(par[n:] == -1) and np.all(dep[n:] == -1) and np.all(mask[n:] == 0)


@pytest.mark.parametrize("seed", [0, 1])
def test_invariants_at_paper_settings(seed):
    """d = 8, k = 25, w = 20, budget 60 (Appendix D) on Zipf ids with a table that really hits."""
    rows = syn.make_ngram_rows(2000, 60_000, "zipf_mixed", seed=seed)
    tri, bi = otree.tables_from_rows(rows)
    t = syn.make_tree_inputs(2000, 2, 8, 25, seed=seed)
    hits = 0
    for b in range(2):
        out = otree.build_tree(t["ids"][b], t["slogit"][b], tuple(t["ctx_tail"][b]), tri, bi, beam=20, budget=60)
        _check_invariants(out, t["ids"][b], 60, 20)
        assert int(out["n_nodes"]) == 60
        assert out["n_scored"] == 25 + 7 * 20 * 25                 # |T| = k * sum_i |Beam_i|
        hits += sum((int(bb), int(tt)) in bi for bb in t["ids"][b, 0] for tt in t["ids"][b, 1])
    assert hits > 0


def test_ngram_rows_are_normalised_log_probabilities():
    rows = syn.make_ngram_rows(300, 5000, "zipf_mixed", seed=3)
    assert np.all(rows["score"] <= 1e-6)
    key = rows["order"].astype(np.int64) * 10 ** 8 + (rows["ctx0"].astype(np.int64) + 1) * 10 ** 4 + rows["ctx1"]
    for c in np.unique(key)[:50]:
        assert abs(np.exp(rows["score"][key == c].astype(np.float64)).sum() - 1.0) < 1e-5
    full = key * 1000 + rows["next"]
    assert len(np.unique(full)) == len(full)


def test_verification_inputs_cover_the_tree_with_root_to_leaf_paths():
    """Pins of the verification glue: every path is a parent chain from the root, depths count up by one along
    it, the paths' union is the whole tree, a slot is a leaf iff nobody names it as parent, and the number of
    ancestors-or-self in build_tree's attention mask is the position offset plus one."""
    rng = np.random.default_rng(3)
    V, d, k = 50, 5, 6
    ids = np.stack([rng.choice(V, size=k, replace=False) for _ in range(d)]).astype(np.int32)
    sl = np.sort(rng.normal(-3, 1.5, size=(d, k)).astype(np.float32))[:, ::-1].copy()
    t = otree.build_tree(ids, sl, (3, 7), {}, {}, beam=4, budget=24)
    n = int(t["n_nodes"])
    g = otree.verification_inputs(np.asarray(t["parents"]), np.asarray(t["depth"]), n, root_pos=100, max_levels=d)
    par, dep, mask = np.asarray(t["parents"]), np.asarray(t["depth"]), np.asarray(t["mask"])
    assert np.array_equal(g["position_ids"][:n], 100 + dep[:n]) and np.all(g["position_ids"][n:] == -1)
    assert np.array_equal(mask[:n].sum(axis=1) - 1, dep[:n])                      # ancestors-or-self = depth + 1
    leaves = sorted(set(range(n)) - set(int(p) for p in par[1:n]))
    assert int(g["n_leaves"]) == len(leaves) and n > 5 and len(leaves) > 1
    seen = set()
    for j, leaf in enumerate(leaves):
        path = [int(x) for x in g["retrieve"][j] if x >= 0]
        assert path[0] == 0 and path[-1] == leaf
        for a, b in zip(path[:-1], path[1:]):
            assert par[b] == a and dep[b] == dep[a] + 1
        assert np.all(g["retrieve"][j, len(path):] == -1)
        seen.update(path)
    assert seen == set(range(n))
    assert np.all(g["retrieve"][len(leaves):] == -1)
    # a chain (beam 1, one candidate per level) has exactly one leaf and one path through every node
    t1 = otree.build_tree(ids[:, :1], sl[:, :1], (3, 7), {}, {}, beam=1, budget=24)
    g1 = otree.verification_inputs(np.asarray(t1["parents"]), np.asarray(t1["depth"]), int(t1["n_nodes"]), root_pos=0, max_levels=d)
    assert int(g1["n_leaves"]) == 1 and [int(x) for x in g1["retrieve"][0]] == list(range(d + 1))
