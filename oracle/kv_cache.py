"""Reference for the paged cache's write path (TEST INFRASTRUCTURE ONLY): appending one
token per sequence.  Plain Python loops over numpy arrays of bf16 bit patterns; the
definition is the layout itself -- token j of sequence b lives in slot j % P of page
block_table[b][j // P] of a pool [pages][Hkv][P][D].  The paper (arXiv 2510.07356, Sec. 3.3)
only implies this step (one new token per sequence per decode step)."""
from __future__ import annotations

import numpy as np


def kv_append(k_pages, v_pages, block_table, seq_lens, k_new, v_new, advance=True):
    """In place: stores k_new[b], v_new[b] ([Hkv][D]) at position seq_lens[b] and advances
    seq_lens[b].  A sequence whose position does not fit its table row, or whose page id is
    outside the pool, is left untouched.  advance=False is the write of a further layer of the
    same step: the rows go to the slot the step's first append opened, position seq_lens[b] - 1,
    and the lengths stay."""
    num_pages, hkv, P, _ = k_pages.shape
    for b in range(len(seq_lens)):
        pos = int(seq_lens[b]) - (0 if advance else 1)
        if pos < 0 or pos >= block_table.shape[1] * P:
            continue
        page = int(block_table[b, pos // P])
        if page < 0 or page >= num_pages:
            continue
        for g in range(hkv):
            k_pages[page, g, pos % P, :] = k_new[b, g, :]
            v_pages[page, g, pos % P, :] = v_new[b, g, :]
        if advance:
            seq_lens[b] = pos + 1


def gather_tokens(pool, block_table, b, n):
    """De-paged rows [n][Hkv][D] of the first n tokens of sequence b."""
    P = pool.shape[2]
    return np.stack([pool[int(block_table[b, j // P]), :, j % P, :] for j in range(n)]) if n else \
        np.zeros((0,) + pool.shape[1:2] + pool.shape[3:], dtype=pool.dtype)
