"""Token-major pools ([page][slot][KV head][D], kv_layout = CONCUR_KV_TOKEN_MAJOR): every entry
point that reads or writes the cache, against the CPU oracle.  The inputs are the usual
head-major workloads with the two pools transposed on the device; the oracle still reads the
head-major originals, so a wrong stride or plane shows as a parity failure."""
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


def token_major(t):
    return t.permute(0, 2, 1, 3).contiguous()          # [pages][Hkv][P][D] -> [pages][P][Hkv][D]


def host(w):
    return synth.gather_sequences(w, range(w.spec.batch))


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("page_size,ranges,hq", [(16, 0, 64), (32, 5, 64), (64, 0, 64), (64, 300, 40), (128, 0, 64)])
def test_plain_step(P, kernel, page_size, ranges, hq):
    spec = synth.tiny_spec(f"tm_p{page_size}", LENS, page_size, 8000 + page_size, num_q_heads=hq)
    w = synth.make_workload(spec, "cuda:0")
    k, v = token_major(w.k_pages), token_major(w.v_pages)
    attn = P.DecodeAttention(page_size, spec.batch, w.block_table.shape[1], 0, num_q_heads=hq,
                             kv_layout=P.CONCUR_KV_TOKEN_MAJOR)
    attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    out = torch.empty_like(w.q)
    lse = torch.empty((spec.batch, hq), dtype=torch.float32, device="cuda:0")
    P.concur_decode_attn(attn.handle, w.q, k, v, w.block_table, w.seq_lens, w.scale, out, lse, spec.batch,
                         w.num_pages, w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"token-major p{page_size} kernel {kernel}")
    attn.close()


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("page_size,ranges,hq", [(16, 0, 64), (16, 9, 40), (32, 0, 64), (32, 300, 24)])
def test_small_pages_through_tma_boxes(P, layout, page_size, ranges, hq):
    """With 16- and 32-token pages the tensor-core kernel's producer copies tiles lane by lane by
    default; the alternative (one TMA box per page and head) must give the same results."""
    spec = synth.tiny_spec(f"box_p{page_size}", LENS, page_size, 8200 + page_size, num_q_heads=hq)
    w = synth.make_workload(spec, "cuda:0")
    k, v = (token_major(w.k_pages), token_major(w.v_pages)) if layout else (w.k_pages, w.v_pages)
    ref_out, ref_lse = oracle_sequences(host(w))
    outs = []
    for mode in (0, 1):
        attn = P.DecodeAttention(page_size, spec.batch, w.block_table.shape[1], 0, num_q_heads=hq, kv_layout=layout)
        attn.set_option(P.CONCUR_OPT_SMALL_PAGE_COPY, mode)
        attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
        out = torch.empty_like(w.q)
        lse = torch.empty((spec.batch, hq), dtype=torch.float32, device="cuda:0")
        P.concur_decode_attn(attn.handle, w.q, k, v, w.block_table, w.seq_lens, w.scale, out, lse, spec.batch,
                             w.num_pages, w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert attn.status() == 0
        assert_parity(out, lse, ref_out, ref_lse, f"p{page_size} layout {layout} copy mode {mode}")
        outs.append((out, lse))
        attn.close()
    # the two modes fill shared memory with the same bytes, so the arithmetic that follows is the same
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


GROUPS = [(1024, [100, 1, 64, 700, 333]), (0, [500]), (2048, [5, 900]),
          (512, [0, 130, 64, 1, 2000, 77, 640, 63, 65, 300])]


@pytest.mark.parametrize("prefix_kernel", [0, 1])
@pytest.mark.parametrize("page_size", [16, 64, 128])
def test_cascade(P, prefix_kernel, page_size):
    cw = synth.make_cascade_workload(f"tm_casc{page_size}", GROUPS, page_size, 8100 + page_size, "cuda:0")
    w = cw.w
    k, v = token_major(w.k_pages), token_major(w.v_pages)
    attn = P.DecodeAttention(page_size, w.spec.batch, w.block_table.shape[1], 0, kv_layout=P.CONCUR_KV_TOKEN_MAJOR)
    attn.set_option(P.CONCUR_OPT_PREFIX_KERNEL, prefix_kernel)
    out = torch.empty_like(w.q)
    lse = torch.empty((w.spec.batch, 64), dtype=torch.float32, device="cuda:0")
    P.concur_decode_attn_cascade(attn.handle, w.q, k, v, w.block_table, w.seq_lens, cw.group_start, cw.prefix_lens,
                                 w.scale, out, lse, w.spec.batch, len(cw.prefix_lens_host), w.num_pages,
                                 w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"token-major cascade p{page_size} prefix kernel {prefix_kernel}")
    attn.close()


@pytest.mark.parametrize("page_size", [16, 64, 128])
def test_prefill(P, page_size):
    lens = (1, 17, 64, 65, 129, 333, 700)
    q_lens = (1, 17, 64, 30, 129, 333, 100)
    pw = synth.make_prefill_workload(f"tm_pf{page_size}", lens, q_lens, page_size, 8200 + page_size, "cuda:0")
    w = pw.w
    k, v = token_major(w.k_pages), token_major(w.v_pages)
    attn = P.DecodeAttention(page_size, w.spec.batch, w.block_table.shape[1], 0, kv_layout=P.CONCUR_KV_TOKEN_MAJOR)
    out = torch.empty_like(w.q)
    lse = torch.empty((pw.total_q, 64), dtype=torch.float32, device="cuda:0")
    P.concur_prefill_attn(attn.handle, w.q, k, v, w.block_table, w.seq_lens, pw.q_start, w.scale, out, lse,
                          w.spec.batch, pw.total_q, w.num_pages, w.block_table.shape[1],
                          torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(synth.prefill_as_decode(pw, range(pw.total_q)))
    assert_parity(out, lse, ref_out, ref_lse, f"token-major prefill p{page_size}")
    attn.close()


@pytest.mark.parametrize("page_size", [16, 128])
def test_append_writes_the_same_cache(P, page_size):
    # append the same rows into a head-major and a token-major copy of one cache: the two pools must
    # stay transposes of each other, byte for byte
    spec = synth.tiny_spec("tm_app", (5, 31, 16, 127, 128), page_size, 8300 + page_size)
    w = synth.make_workload(spec, "cuda:0", spare_tokens=3)
    B = spec.batch
    k_h, v_h = w.k_pages.clone(), w.v_pages.clone()
    k_t, v_t = token_major(w.k_pages), token_major(w.v_pages)
    a_h = P.DecodeAttention(page_size, B, w.block_table.shape[1], 0)
    a_t = P.DecodeAttention(page_size, B, w.block_table.shape[1], 0, kv_layout=P.CONCUR_KV_TOKEN_MAJOR)
    lens_h, lens_t = w.seq_lens.clone(), w.seq_lens.clone()
    g = torch.Generator(device="cuda:0"); g.manual_seed(5)
    for _ in range(3):
        kn = torch.randn((B, 8, 128), generator=g, device="cuda:0").to(torch.bfloat16)
        vn = torch.randn((B, 8, 128), generator=g, device="cuda:0").to(torch.bfloat16)
        P.concur_kv_append(a_h.handle, kn, vn, k_h, v_h, w.block_table, lens_h, B, w.num_pages, w.block_table.shape[1], 0)
        P.concur_kv_append(a_t.handle, kn, vn, k_t, v_t, w.block_table, lens_t, B, w.num_pages, w.block_table.shape[1], 0)
    torch.cuda.synchronize()
    assert a_h.status() == 0 and a_t.status() == 0 and torch.equal(lens_h, lens_t)
    same = lambda a, b: torch.equal(token_major(a).view(torch.int16), b.view(torch.int16))
    assert same(k_h, k_t) and same(v_h, v_t)
    assert not torch.equal(k_h.view(torch.int16), w.k_pages.view(torch.int16))        # something was written
    a_h.close(); a_t.close()


def test_unknown_layout_is_rejected(P):
    B = P.binding
    assert B.concur_attn_workspace_bytes(B.make_config(64, 4, 8, 0, kv_layout=2)) == 0
