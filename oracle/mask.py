"""Attention-visibility rules of DART -- oracle side, TEST INFRASTRUCTURE ONLY.

``training_visible`` restates, as one boolean formula, the prefix-shared training mask that
Appendix B ("Training with Flex Attention") describes in words and code: a packed row of
`prompt_len` clean positions followed by one block of `draft_len` masked positions per
prefix position.  Its restriction to a single block must be the plain causal rule that the
inference step uses (Section 3.1, "Causal attention mask"); the tests check exactly that.
"""
from __future__ import annotations


def training_visible(q_idx: int, kv_idx: int, prompt_len: int, draft_len: int, seq_len: int) -> bool:
    """True iff query slot q_idx may read key slot kv_idx in the packed training row.

    Three regions (Figure 4): clean causal attention inside the prompt; a masked block
    reading its own prefix (block n belongs to prompt position n and reads prompt slots
    0..n); causal attention inside one masked block.  Blocks never read each other.
    """
    q_clean, kv_clean = q_idx < prompt_len, kv_idx < prompt_len
    if q_clean:
        return kv_clean and kv_idx <= q_idx and q_idx < seq_len and kv_idx < seq_len
    block = (q_idx - prompt_len) // draft_len
    if block >= seq_len:
        return False
    if kv_clean:
        return kv_idx <= block
    return (kv_idx - prompt_len) // draft_len == block and kv_idx <= q_idx
