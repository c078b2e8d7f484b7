"""A handle holder for torch tensors: allocation of outputs and stream lookup only."""
from __future__ import annotations

import torch

from . import binding as B


class DecodeAttention:
    """Owns one concur_attn handle.  `__call__` enqueues one decode-attention step on
    torch's current stream and returns (out bf16 [B][Hq][D], lse fp32 [B][Hq])."""

    def __init__(self, page_size: int, max_batch: int, max_pages_per_seq: int, device: int = 0,
                 num_q_heads: int = 64, kv_layout: int = 0, num_kv_heads: int = 8):
        if not torch.cuda.is_available():
            raise RuntimeError("concur_attn needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", device)
        self.cfg = B.make_config(page_size, max_batch, max_pages_per_seq, device, num_q_heads=num_q_heads,
                                 num_kv_heads=num_kv_heads, kv_layout=kv_layout)
        self.handle = B.concur_attn_create(self.cfg)

    def set_option(self, key: int, value: int):
        B.concur_attn_set_option(self.handle, key, value)

    def __call__(self, q, k_pages, v_pages, block_table, seq_lens, scale, out=None, lse=None):
        batch = q.shape[0]
        if out is None:
            out = torch.empty_like(q)
        if lse is None:
            lse = torch.empty((batch, q.shape[1]), dtype=torch.float32, device=q.device)
        stream = torch.cuda.current_stream(self.device).cuda_stream
        B.concur_decode_attn(self.handle, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse,
                             batch, k_pages.shape[0], block_table.shape[1], stream)
        return out, lse

    def status(self) -> int:
        return B.concur_attn_status(self.handle, torch.cuda.current_stream(self.device).cuda_stream)

    def last_plan(self):
        return B.concur_attn_last_plan(self.handle, torch.cuda.current_stream(self.device).cuda_stream)

    def close(self):
        if self.handle:
            B.concur_attn_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
