"""Second, separately written routine for tiny inputs (TEST INFRASTRUCTURE ONLY).

Pure-Python loops, the softmax written in its naive form (no maximum subtracted),
sums taken with ``math.fsum`` (exactly rounded).  Valid only while
``exp(score)`` neither overflows nor underflows, i.e. for the small scores of
the brute-force pin.  It deliberately shares nothing with ``attn_oracle.c``: the
page lookup, the bf16 widening and the softmax are all restated here, so that
an index or sign slip in either one shows up as a disagreement.
"""
from __future__ import annotations

import math
import struct


def bf16_bits_to_float(bits: int) -> float:
    return struct.unpack("<f", struct.pack("<I", (int(bits) & 0xFFFF) << 16))[0]


def decode_attn_naive(q, k_pages, v_pages, block_table, seq_lens, scale,
                      num_q_heads, num_kv_heads, head_dim, page_size):
    """All arguments are nested Python lists / numpy arrays of bf16 bit patterns
    (q [B][Hq][D]; pools [pages][Hkv][P][D]) and ints.  Returns (out, lse) as
    nested lists of Python floats."""
    group = num_q_heads // num_kv_heads
    scale = struct.unpack("<f", struct.pack("<f", scale))[0]  # the caller's fp32 value
    out, lse = [], []
    for b, n in enumerate(seq_lens):
        out_b, lse_b = [], []
        for h in range(num_q_heads):
            g = h // group
            e = []
            rows = []
            for j in range(int(n)):
                page = int(block_table[b][j // page_size])
                slot = j % page_size
                dot = math.fsum(
                    bf16_bits_to_float(q[b][h][c]) * bf16_bits_to_float(k_pages[page][g][slot][c])
                    for c in range(head_dim))
                e.append(math.exp(scale * dot))
                rows.append([bf16_bits_to_float(v_pages[page][g][slot][c]) for c in range(head_dim)])
            if not e:
                out_b.append([0.0] * head_dim)
                lse_b.append(-math.inf)
                continue
            z = math.fsum(e)
            out_b.append([math.fsum(e[j] * rows[j][c] for j in range(len(e))) / z
                          for c in range(head_dim)])
            lse_b.append(math.log(z))
        out.append(out_b)
        lse.append(lse_b)
    return out, lse
