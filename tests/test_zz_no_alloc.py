"""The handle-free entry point for callers that cannot allocate device memory
(concur_decode_attn_static): the oracle's results, the regular entry point's results, on
calls in a row that share its built-in workspace, and no change in the device's free memory.

Collected last on purpose: should this addition ever fail, a run that stops at the first
failure has already executed every other test.
"""
import pytest
import torch

import synth
from helpers import assert_parity, oracle_sequences

pytestmark = pytest.mark.gpu

# the two entry points may split sequences differently, so their bf16 outputs agree to the
# tolerance every parity test uses, not bit for bit
OUT_ATOL, OUT_RTOL, LSE_ATOL = 4e-3, 1.6e-2, 1e-3


def test_static_entry_matches_oracle_and_handle_entry_twice_in_a_row():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as P

    stream = torch.cuda.current_stream().cuda_stream
    # different batches one after the other, so that anything an earlier call left in the shared
    # array would be noticed; the fourth has more sequences than the kernel's shared-memory plan
    # tables hold (511), so its plan is read from the built-in array itself
    many = [1 + (37 * i) % 150 for i in range(600)]
    specs = [synth.tiny_spec("na0", (3000, 1, 0, 64, 777, 12000), 64, 501),
             synth.tiny_spec("na1", (9000, 20000, 130, 64, 5, 0, 4100, 2500), 64, 502),
             synth.tiny_spec("na2", (700, 17, 0, 3000, 33), 16, 503),
             synth.tiny_spec("na3", many, 16, 504)]
    for spec in specs:
        w = synth.make_workload(spec, "cuda:0")
        B = spec.batch
        ref = P.DecodeAttention(spec.page_size, B, w.block_table.shape[1], 0)
        out_ref, lse_ref = ref(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
        out = torch.full_like(w.q, 7.0)
        lse = torch.full((B, 64), 7.0, dtype=torch.float32, device="cuda:0")

        def call():
            P.concur_decode_attn_static(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale,
                                        out, lse, B, w.num_pages, w.block_table.shape[1], spec.page_size, stream)

        call()                                   # (the very first call also resolves the array's address)
        torch.cuda.synchronize()
        # the promise in the entry point's name: a call takes no device memory and gives none back
        free_before = torch.cuda.mem_get_info(0)[0]
        out.fill_(7.0); lse.fill_(7.0)
        call()
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(0)[0] == free_before
        # against the CPU oracle, element by element ...
        ref_o, ref_l = oracle_sequences(synth.gather_sequences(w, range(B)))
        assert_parity(out, lse, ref_o, ref_l, f"static entry, {spec.name}")
        # ... and against the entry point that owns a workspace
        a, b = out.float(), out_ref.float()
        assert ((a - b).abs() <= OUT_ATOL + OUT_RTOL * b.abs()).all()
        empty = torch.isneginf(lse_ref)
        assert torch.equal(torch.isneginf(lse), empty)
        assert ((lse - lse_ref)[~empty].abs() <= LSE_ATOL).all()
        ref.close()

    # beyond the built-in workspace's batch limit: a clear error, nothing launched
    rc = P.concur_decode_attn_static(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale,
                                     out, lse, P.binding.CONCUR_STATIC_MAX_BATCH + 1, w.num_pages,
                                     w.block_table.shape[1], 64, stream, check=False)
    assert rc == P.binding.CONCUR_ERR_TOO_LARGE
    rc = P.concur_decode_attn_static(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale,
                                     out, lse, B, w.num_pages, w.block_table.shape[1], 48, stream, check=False)
    assert rc == P.binding.CONCUR_ERR_UNSUPPORTED
