"""Group sizes other than 8 (Hq = 8, 16, 24, 40 query heads over 8 KV heads): the CUDA path against
the CPU oracle, element by element, for the plain step (both partial kernels, the host-buffer
entry point) and the shared-prefix step (both prefix kernels)."""
import numpy as np
import pytest
import torch

import synth
from helpers import assert_parity, oracle_sequences

pytestmark = pytest.mark.gpu

LENS = (0, 1, 63, 64, 65, 200, 517, 1000, 2049, 4099)


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def host(w):
    return synth.gather_sequences(w, range(w.spec.batch))


@pytest.mark.parametrize("hq", [8, 16, 24, 40, 56])
@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("page_size,ranges", [(16, 0), (64, 0), (64, 7), (32, 300), (128, 0), (128, 9)])
def test_plain_step_with_smaller_groups(P, hq, kernel, page_size, ranges):
    spec = synth.tiny_spec(f"g{hq}", LENS, page_size, 7000 + hq, num_q_heads=hq)
    w = synth.make_workload(spec, "cuda:0")
    assert w.q.shape == (len(LENS), hq, 128)
    attn = P.DecodeAttention(page_size, spec.batch, w.block_table.shape[1], 0, num_q_heads=hq)
    attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    # canaries behind out and lse: a kernel that still assumed 64 heads would write past them
    out_buf = torch.full((spec.batch * hq * 128 + 4096,), 7.0, dtype=torch.bfloat16, device="cuda:0")
    lse_buf = torch.full((spec.batch * hq + 512,), 7.0, dtype=torch.float32, device="cuda:0")
    out = out_buf[:spec.batch * hq * 128].view(spec.batch, hq, 128)
    lse = lse_buf[:spec.batch * hq].view(spec.batch, hq)
    attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out=out, lse=lse)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert (out_buf[spec.batch * hq * 128:] == 7.0).all() and (lse_buf[spec.batch * hq:] == 7.0).all()
    ref_out, ref_lse = oracle_sequences(host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"hq {hq} kernel {kernel} p{page_size} R{ranges}")
    attn.close()


def test_host_entry_point_with_40_heads(P):
    spec = synth.tiny_spec("g40h", (300, 0, 4099, 64), 64, 7100, num_q_heads=40)
    w = synth.make_workload(spec, "cpu")
    attn = P.DecodeAttention(64, spec.batch, w.block_table.shape[1], 0, num_q_heads=40)
    out = torch.empty_like(w.q)
    lse = torch.empty((spec.batch, 40), dtype=torch.float32)
    P.concur_decode_attn_host(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out, lse,
                              spec.batch, w.num_pages, w.block_table.shape[1], 0)
    ref_out, ref_lse = oracle_sequences(w)
    assert_parity(out, lse, ref_out, ref_lse, "host entry, 40 heads")
    attn.close()


GROUPS = [(1024, [100, 1, 64, 700, 333]), (0, [500]), (2048, [5, 900]),
          (512, [0, 130, 64, 1, 2000, 77, 640, 63, 65, 300]), (256, [10 * j + 1 for j in range(13)])]


@pytest.mark.parametrize("hq", [16, 40])
@pytest.mark.parametrize("prefix_kernel", [0, 1])
@pytest.mark.parametrize("page_size", [16, 64])
def test_cascade_with_smaller_groups(P, hq, prefix_kernel, page_size):
    cw = synth.make_cascade_workload(f"cg{hq}", GROUPS, page_size, 7200 + hq, "cuda:0", num_q_heads=hq)
    w = cw.w
    attn = P.DecodeAttention(page_size, w.spec.batch, w.block_table.shape[1], 0, num_q_heads=hq)
    attn.set_option(P.CONCUR_OPT_PREFIX_KERNEL, prefix_kernel)
    out = torch.full_like(w.q, 7.0)
    lse = torch.full((w.spec.batch, hq), 7.0, dtype=torch.float32, device="cuda:0")
    P.concur_decode_attn_cascade(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens,
                                 cw.group_start, cw.prefix_lens, w.scale, out, lse, w.spec.batch,
                                 len(cw.prefix_lens_host), w.num_pages, w.block_table.shape[1],
                                 torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"cascade hq {hq} prefix kernel {prefix_kernel} p{page_size}")
    attn.close()


def test_unsupported_head_counts_are_rejected(P):
    B = P.binding
    for hq in (0, 4, 12, 72, 128):
        cfg = B.make_config(64, 4, 8, 0, num_q_heads=hq)
        assert B.concur_attn_workspace_bytes(cfg) == 0
