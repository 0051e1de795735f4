"""Integer side of the oracle: page allocator and per-step batch metadata.

TEST INFRASTRUCTURE ONLY.  Written independently of the library's C++ host
code; the tests require the two to agree bit for bit.

The paper keeps its runtime's KV-cache management unchanged (Sec. 5) and gives
no allocation rule, so the rule is the library's documented one: the free list
is a stack whose pops yield page 0, 1, 2, ... on a fresh pool; a sequence that
grows gets ceil(total / page_size) - owned further pops; freeing a sequence
pushes its pages back in reverse order of acquisition; an allocation that does
not fit changes nothing.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import numpy as np


class OutOfPages(Exception):
    pass


class PageAllocator:
    def __init__(self, num_pages: int, page_size: int):
        self.page_size = page_size
        # top of the stack is the end of the list; the first pop must give page 0
        self.free: List[int] = list(range(num_pages - 1, -1, -1))
        self.owned: Dict[int, List[int]] = {}

    def alloc(self, seq_id: int, total_tokens: int) -> List[int]:
        """Grow seq_id to hold total_tokens; returns its whole block table."""
        have = self.owned.get(seq_id, [])
        need = -(-total_tokens // self.page_size) - len(have)
        if need > len(self.free):
            raise OutOfPages()
        pages = list(have)
        for _ in range(max(need, 0)):
            pages.append(self.free.pop())
        self.owned[seq_id] = pages
        return list(pages)

    def release(self, seq_id: int) -> None:
        for page in reversed(self.owned.pop(seq_id)):
            self.free.append(page)


def block_table_array(tables: Sequence[Sequence[int]], max_pages_per_seq: int) -> np.ndarray:
    """Pads per-sequence page lists with -1 into an int32 [n_seqs, max_pages_per_seq] array."""
    out = np.full((len(tables), max_pages_per_seq), -1, dtype=np.int32)
    for s, pages in enumerate(tables):
        out[s, : len(pages)] = pages
    return out


def plan_tokens(q_len: Sequence[int], ctx_len: Sequence[int], block_tables: np.ndarray,
                page_size: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Per-token metadata of a step: owning sequence, absolute position and
    cache slot (physical page * page_size + position within the page)."""
    tok_seq, tok_pos, tok_slot = [], [], []
    for s, (n, c) in enumerate(zip(q_len, ctx_len)):
        for j in range(int(n)):
            p = int(c) + j
            tok_seq.append(s)
            tok_pos.append(p)
            tok_slot.append(int(block_tables[s][p // page_size]) * page_size + p % page_size)
    return (np.asarray(tok_seq, dtype=np.int32), np.asarray(tok_pos, dtype=np.int32),
            np.asarray(tok_slot, dtype=np.int32))
