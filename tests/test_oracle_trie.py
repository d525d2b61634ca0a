"""Pins of the N-gram trie oracle (Appendix C) against what the row table fixes by definition."""
import numpy as np

from oracle import tree as otree
from oracle import trie as otrie
from paper_2601_19278_b200 import synthetic

MISS = np.float32(-23.0)


def _rows(lst):
    o, c0, c1, nx, s = zip(*lst)
    return {"order": np.array(o), "ctx0": np.array(c0), "ctx1": np.array(c1), "next": np.array(nx),
            "score": np.array(s, dtype=np.float32)}


def test_worked_example_by_hand():
    # rows written out by hand; expected values follow from the back-off rule alone
    rows = _rows([(3, 1, 2, 5, -0.5), (3, 1, 2, 6, -1.5), (2, -1, 2, 5, -2.0), (2, -1, 2, 7, -3.0),
                  (3, 1, 2, 5, -9.0)])            # a repeated row: the first one stays
    tri, bi = otrie.tries_from_rows(rows)
    assert otrie.candidate_scores(tri, bi, 1, 2, [5, 6, 7, 8], MISS) == [-0.5, -1.5, -3.0, MISS]
    assert otrie.candidate_scores(tri, bi, 9, 2, [5, 6, 7, 8], MISS) == [-2.0, MISS, -3.0, MISS]
    assert otrie.candidate_scores(tri, bi, -1, 2, [5, 6], MISS) == [-2.0, MISS]
    assert otrie.candidate_scores(tri, bi, 1, -1, [5, 6], MISS) == [MISS, MISS]
    assert otrie.candidate_scores(tri, bi, 2, 1, [2, 5], MISS) == [MISS, MISS]   # context order matters
    # 3-gram trie: 1 -> 2 -> {5, 6} = 4 nodes; 2-gram trie: 2 -> {5, 7} = 3 nodes
    assert otrie.count_nodes(tri) == 4 and otrie.count_nodes(bi) == 3
    # an inner node is not a row: (1, 2) is a path of the 3-gram trie, not a 2-gram row
    assert otrie.candidate_scores(tri, bi, 0, 1, [2], MISS) == [MISS]


def test_brute_force_against_a_linear_scan_of_the_rows():
    rng = np.random.default_rng(5)
    V, n = 5, 90
    order = rng.integers(2, 4, n)
    rows = {"order": order, "ctx0": np.where(order == 3, rng.integers(0, V, n), -1), "ctx1": rng.integers(0, V, n),
            "next": rng.integers(0, V, n), "score": -rng.random(n).astype(np.float32) - 0.01}
    tri, bi = otrie.tries_from_rows(rows)

    def scan(a, b, t):
        for want in (3, 2):
            for i in range(n):
                if rows["order"][i] != want or rows["ctx1"][i] != b or rows["next"][i] != t:
                    continue
                if want == 3 and (a < 0 or rows["ctx0"][i] != a):
                    continue
                return np.float32(rows["score"][i])
        return MISS

    S = list(range(V))
    for a in range(-1, V):
        for b in range(0, V):
            got = otrie.candidate_scores(tri, bi, a, b, S, MISS)
            assert got == [scan(a, b, t) for t in S], (a, b)


def test_same_scores_as_the_row_table_on_the_workload_generator():
    vocab = 512
    rows = synthetic.make_ngram_rows(vocab, 20000, "zipf_mixed", seed=77)
    tri_d, bi_d = otree.tables_from_rows(rows)
    tri, bi = otrie.tries_from_rows(rows)
    rng = np.random.default_rng(9)
    hits = 0
    for _ in range(300):
        i = int(rng.integers(0, rows["order"].shape[0]))
        a = int(rows["ctx0"][i]) if rng.random() < 0.7 else int(rng.integers(-1, vocab))
        b = int(rows["ctx1"][i])
        S = [int(rows["next"][i])] + rng.integers(0, vocab, 24).tolist()
        got = otrie.candidate_scores(tri, bi, a, b, S, MISS)
        want = [otree.ngram_score(tri_d, bi_d, a, b, t, MISS) for t in S]
        assert got == want
        hits += sum(1 for g in got if g != MISS)
    assert hits > 300      # the sample exercises hits, not only misses
    assert otrie.count_nodes(tri) >= len(tri_d) and otrie.count_nodes(bi) >= len(bi_d)
