"""CPU oracle for the N-gram trie -- TEST INFRASTRUCTURE ONLY.

Appendix C: the N-gram is a trie; to score the k_i candidates S_i that share one preceding
context, the context's node is located once and its child nodes, one per continuation
token, are then read.  This file is that structure written plainly: a node is a dict from
token to child node, a node that ends a stored row carries the row's score.  The scores
it returns are by definition those of the row table (oracle.tree.ngram_score): the trie
changes how a row is found, never which row or which value.

Stored orientation (reading; the paper does not print its node layout): a 3-gram row
(a, b, t) hangs under root -> a -> b -> t, a 2-gram row (b, t) under root -> b -> t, in
two separate tries, so that the 3-gram -> 2-gram back-off of the scoring rule is a second
context lookup.  Where rows repeat, the first one wins.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np

f32 = np.float32


class Node:
    __slots__ = ("children", "score")

    def __init__(self) -> None:
        self.children: Dict[int, "Node"] = {}
        self.score: Optional[float] = None


def insert(root: Node, path: Sequence[int], score: float) -> None:
    """Add one row; a row already present keeps its score."""
    node = root
    for t in path:
        nxt = node.children.get(int(t))
        if nxt is None:
            nxt = Node()
            node.children[int(t)] = nxt
        node = nxt
    if node.score is None:
        node.score = score


def locate(root: Node, context: Sequence[int]) -> Optional[Node]:
    """The node of a preceding context, or None if no stored row starts with it."""
    node = root
    for t in context:
        node = node.children.get(int(t))
        if node is None:
            return None
    return node


def tries_from_rows(rows: Dict[str, np.ndarray]):
    """Row arrays (order, ctx0, ctx1, next, score) -> (3-gram trie, 2-gram trie)."""
    tri, bi = Node(), Node()
    for o, c0, c1, nx, s in zip(rows["order"].tolist(), rows["ctx0"].tolist(), rows["ctx1"].tolist(),
                                rows["next"].tolist(), rows["score"].tolist()):
        if o == 3:
            insert(tri, (c0, c1, nx), s)
        else:
            insert(bi, (c1, nx), s)
    return tri, bi


def candidate_scores(tri: Node, bi: Node, a: int, b: int, S_i: Sequence[int], miss) -> List[np.float32]:
    """s_ng of every candidate t in S_i after the context (a, b): one traversal to the node of (a, b) and one
    to the node of (b), then each candidate is looked up among those nodes' children; 3-gram first, 2-gram
    next, else the miss score.  a < 0 or b < 0 marks an absent context token."""
    n3 = locate(tri, (a, b)) if (a >= 0 and b >= 0) else None
    n2 = locate(bi, (b,)) if b >= 0 else None
    out: List[np.float32] = []
    for t in S_i:
        c = n3.children.get(int(t)) if n3 is not None else None
        if c is not None and c.score is not None:
            out.append(f32(c.score))
            continue
        c = n2.children.get(int(t)) if n2 is not None else None
        if c is not None and c.score is not None:
            out.append(f32(c.score))
            continue
        out.append(f32(miss))
    return out


def count_nodes(root: Node) -> int:
    """Nodes below the root (the paper's size measure: about 1.3 billion for its 3-gram)."""
    n, stack = 0, [root]
    while stack:
        node = stack.pop()
        n += len(node.children)
        stack.extend(node.children.values())
    return n
