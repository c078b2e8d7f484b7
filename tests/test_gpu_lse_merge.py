"""concur_lse_merge and context sharding: the decode step run on each token range of every sequence (one
call after the other on one GPU: the calls do not depend on one another), the (out, lse) pairs put side by
side as an all-gather would, merged by the kernel -- against the oracle on the unsharded inputs; and the
kernel alone against the oracle's merge on made-up parts."""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import assert_parity, oracle_sequences

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("page_size", [16, 64])
def test_context_shards_merged_equal_the_unsharded_oracle(P, world, page_size):
    lens = (0, 1, 15, 64, 65, 300, 1000, 4099, 20000)
    w = synth.make_workload(synth.tiny_spec(f"ctx_p{page_size}", lens, page_size, 9200 + page_size), "cuda:0")
    B = w.spec.batch
    ref_out, ref_lse = oracle_sequences(synth.gather_sequences(w, range(B)))
    gath_out = torch.empty((world, B, 64, 128), dtype=torch.bfloat16, device="cuda:0")
    gath_lse = torch.empty((world, B, 64), dtype=torch.float32, device="cuda:0")
    for rank in range(world):
        ws = synth.shard_context(w, rank, world)
        attn = P.DecodeAttention(page_size, B, ws.block_table.shape[1], 0)
        o, l = attn(ws.q, ws.k_pages, ws.v_pages, ws.block_table, ws.seq_lens, ws.scale)
        torch.cuda.synchronize()
        assert attn.status() == 0
        gath_out[rank] = o; gath_lse[rank] = l
        attn.close()
    out = torch.full((B, 64, 128), 7.0, dtype=torch.bfloat16, device="cuda:0")
    lse = torch.full((B, 64), 7.0, dtype=torch.float32, device="cuda:0")
    P.concur_lse_merge(gath_out, gath_lse, world, B * 64, out, lse, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert_parity(out, lse, ref_out, ref_lse, f"context sharding x{world}, page {page_size}")


def test_merge_kernel_against_the_oracle_merge(P):
    g = torch.Generator(device="cuda:0").manual_seed(9300)
    parts, rows = 5, 1003                                          # (a ragged last block)
    outs = torch.randn((parts, rows, 128), generator=g, device="cuda:0").to(torch.bfloat16)
    lses = (torch.randn((parts, rows), generator=g, device="cuda:0") * 6).float()
    lses[1, ::7] = float("-inf")                                   # parts without keys
    lses[:, 5] = float("-inf")                                     # a row nobody has keys for
    lses[3, 11] = 80.0                                             # one part dominates
    out = torch.empty((rows, 128), dtype=torch.bfloat16, device="cuda:0")
    lse = torch.empty((rows,), dtype=torch.float32, device="cuda:0")
    P.concur_lse_merge(outs, lses, parts, rows, out, lse, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    po = outs.float().cpu().numpy().astype(np.float64); pl = lses.cpu().numpy().astype(np.float64)
    ref_o = np.empty((rows, 128)); ref_l = np.empty(rows)
    for r in range(rows):
        ref_o[r], ref_l[r] = oracle.lse_merge(po[:, r], pl[:, r])
    got_o = out.float().cpu().numpy().astype(np.float64); got_l = lse.cpu().numpy().astype(np.float64)
    assert np.array_equal(np.isneginf(got_l), np.isneginf(ref_l)) and np.isneginf(got_l[5]) and (got_o[5] == 0).all()
    fin = np.isfinite(ref_l)
    assert np.abs(got_l[fin] - ref_l[fin]).max() <= 1e-4
    assert (np.abs(got_o - ref_o) <= 4e-3 + 8e-3 * np.abs(ref_o)).all()    # one bf16 rounding of the result


def test_merge_argument_errors(P):
    B_ = P.binding
    t = torch.zeros((2, 8, 128), dtype=torch.bfloat16, device="cuda:0")
    l = torch.zeros((2, 8), dtype=torch.float32, device="cuda:0")
    o = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda:0"); ol = torch.zeros(8, dtype=torch.float32, device="cuda:0")
    assert B_.concur_lse_merge(t, l, 0, 8, o, ol, check=False) == B_.CONCUR_ERR_INVALID_ARG
    assert B_.concur_lse_merge(t, l, 2, -1, o, ol, check=False) == B_.CONCUR_ERR_INVALID_ARG
    assert B_.concur_lse_merge(None, l, 2, 8, o, ol, check=False) == B_.CONCUR_ERR_INVALID_ARG
    assert B_.concur_lse_merge(t.data_ptr() + 2, l, 2, 8, o, ol, check=False) == B_.CONCUR_ERR_INVALID_ARG
    assert B_.concur_lse_merge(t, l, 2, 0, o, ol, check=False) == B_.CONCUR_OK
    assert B_.concur_lse_merge(t, l, 2, 8, o, ol, check=False) == B_.CONCUR_OK
    torch.cuda.synchronize()
