"""Fewer than 8 KV heads per call -- what one rank of a model that is tensor-parallel over its KV
heads passes (8 query heads over 1 KV head at 8 ranks of the 64 / 8 geometry): every entry point
against the CPU oracle, element by element, and the ranks' head slices put together against the
oracle's result on the unsharded inputs."""
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


def handle_for(P, w, kv_layout=0):
    s = w.spec
    return P.DecodeAttention(s.page_size, max(1, s.batch), w.block_table.shape[1], 0, num_q_heads=s.num_q_heads,
                             num_kv_heads=s.num_kv_heads, kv_layout=kv_layout)


@pytest.mark.parametrize("hkv,hq", [(1, 8), (2, 16), (4, 32), (1, 5), (3, 24), (6, 12), (1, 1)])
@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("page_size,ranges", [(16, 0), (64, 0), (64, 7), (32, 300), (128, 9)])
def test_plain_step(P, hkv, hq, kernel, page_size, ranges):
    spec = synth.tiny_spec(f"kv{hkv}q{hq}", LENS, page_size, 8000 + 10 * hkv + hq, num_q_heads=hq, num_kv_heads=hkv)
    w = synth.make_workload(spec, "cuda:0")
    assert w.k_pages.shape[1] == hkv and w.q.shape[1] == hq
    attn = handle_for(P, w)
    attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    # canaries behind out and lse: a kernel that still assumed 8 KV heads would write past them
    n_out = spec.batch * hq * 128
    out_buf = torch.full((n_out + 4096,), 7.0, dtype=torch.bfloat16, device="cuda:0")
    lse_buf = torch.full((spec.batch * hq + 512,), 7.0, dtype=torch.float32, device="cuda:0")
    out = out_buf[:n_out].view(spec.batch, hq, 128)
    lse = lse_buf[:spec.batch * hq].view(spec.batch, hq)
    attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out=out, lse=lse)
    torch.cuda.synchronize()
    assert attn.status() == 0
    R, W, _ = attn.last_plan()
    assert W == hkv * sum(-(-n // 64) for n in LENS)
    assert (out_buf[n_out:] == 7.0).all() and (lse_buf[spec.batch * hq:] == 7.0).all()
    ref_out, ref_lse = oracle_sequences(host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"hkv {hkv} hq {hq} kernel {kernel} p{page_size} R{ranges}")
    attn.close()


@pytest.mark.parametrize("world", [2, 4, 8])
def test_rank_slices_put_together_equal_the_unsharded_result(P, world):
    # the full 64 / 8 problem, cut the way tensor parallelism over KV heads cuts it; every rank's call
    # sees only its slice, and the slices side by side are the oracle's result on the whole problem
    spec = synth.tiny_spec("tp_full", (3000, 1, 64, 777, 9000, 0, 130), 64, 8100)
    w = synth.make_workload(spec, "cuda:0")
    ref_out, ref_lse = oracle_sequences(host(w))
    outs, lses = [], []
    for rank in range(world):
        ws = synth.shard_kv_heads(w, rank, world)
        attn = handle_for(P, ws)
        o, l = attn(ws.q, ws.k_pages, ws.v_pages, ws.block_table, ws.seq_lens, ws.scale)
        torch.cuda.synchronize()
        assert attn.status() == 0
        outs.append(o); lses.append(l)
        attn.close()
    assert_parity(torch.cat(outs, dim=1), torch.cat(lses, dim=1), ref_out, ref_lse, f"TP {world} over KV heads")


@pytest.mark.parametrize("hkv", [1, 2, 4])
def test_token_major_pools(P, hkv):
    hq = 8 * hkv
    for page_size in (16, 64, 128):
        spec = synth.tiny_spec(f"kvtm{hkv}", LENS, page_size, 8200 + hkv, num_q_heads=hq, num_kv_heads=hkv)
        w = synth.make_workload(spec, "cuda:0")
        ref_out, ref_lse = oracle_sequences(host(w))
        kt = w.k_pages.permute(0, 2, 1, 3).contiguous()
        vt = w.v_pages.permute(0, 2, 1, 3).contiguous()
        for kernel in (0, 1):
            attn = handle_for(P, w, kv_layout=P.CONCUR_KV_TOKEN_MAJOR)
            attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
            out, lse = attn(w.q, kt, vt, w.block_table, w.seq_lens, w.scale)
            torch.cuda.synchronize()
            assert attn.status() == 0
            assert_parity(out, lse, ref_out, ref_lse, f"token-major hkv {hkv} p{page_size} kernel {kernel}")
            attn.close()


GROUPS = [(1024, [100, 1, 64, 700, 333]), (0, [500]), (2048, [5, 900]),
          (512, [0, 130, 64, 1, 2000, 77, 640, 63, 65, 300]), (256, [10 * j + 1 for j in range(13)])]


@pytest.mark.parametrize("hkv,hq", [(1, 8), (2, 16), (4, 20)])
@pytest.mark.parametrize("prefix_kernel", [0, 1])
@pytest.mark.parametrize("page_size", [16, 64])
def test_cascade_step(P, hkv, hq, prefix_kernel, page_size):
    cw = synth.make_cascade_workload(f"ckv{hkv}", GROUPS, page_size, 8300 + hkv, "cuda:0", num_q_heads=hq,
                                     num_kv_heads=hkv)
    w = cw.w
    attn = handle_for(P, w)
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
    assert_parity(out, lse, ref_out, ref_lse, f"cascade hkv {hkv} hq {hq} prefix kernel {prefix_kernel} p{page_size}")
    attn.close()


@pytest.mark.parametrize("hkv,hq", [(1, 8), (2, 16), (4, 20)])
@pytest.mark.parametrize("page_size", [16, 64])
def test_prefill(P, hkv, hq, page_size):
    lens, q_lens = (70, 33, 300, 1, 129), (70, 20, 300, 1, 16)
    pw = synth.make_prefill_workload(f"pkv{hkv}", lens, q_lens, page_size, 8400 + hkv, "cuda:0", num_q_heads=hq,
                                     num_kv_heads=hkv)
    w = pw.w
    attn = handle_for(P, w)
    out = torch.full_like(w.q, 7.0)
    lse = torch.full((pw.total_q, hq), 7.0, dtype=torch.float32, device="cuda:0")
    P.concur_prefill_attn(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, pw.q_start, w.scale,
                          out, lse, len(lens), pw.total_q, w.num_pages, w.block_table.shape[1],
                          torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    d = synth.prefill_as_decode(pw, range(pw.total_q))
    ref_out, ref_lse = oracle_sequences(d)
    assert_parity(out, lse, ref_out, ref_lse, f"prefill hkv {hkv} hq {hq} p{page_size}")
    attn.close()


@pytest.mark.parametrize("hkv", [1, 2, 4])
@pytest.mark.parametrize("token_major", [0, 1])
def test_append_then_attend(P, hkv, token_major):
    import oracle
    import oracle.kv_cache as kvc
    hq, page_size, steps = 8 * hkv, 16, 5
    spec = synth.tiny_spec(f"akv{hkv}", (15, 16, 0, 200, 31), page_size, 8500 + hkv, num_q_heads=hq, num_kv_heads=hkv)
    w = synth.make_workload(spec, "cuda:0", spare_tokens=steps)
    k_ref = w.k_pages.cpu().view(torch.int16).numpy().copy()
    v_ref = w.v_pages.cpu().view(torch.int16).numpy().copy()
    lens_ref = w.lens_host.copy()
    k_dev, v_dev = w.k_pages, w.v_pages
    if token_major:
        k_dev = k_dev.permute(0, 2, 1, 3).contiguous(); v_dev = v_dev.permute(0, 2, 1, 3).contiguous()
    attn = handle_for(P, w, kv_layout=token_major)
    lens = w.seq_lens.clone()
    g = torch.Generator(device="cuda:0"); g.manual_seed(8600 + hkv)
    stream = torch.cuda.current_stream().cuda_stream
    for step in range(steps):
        kn = torch.randn((spec.batch, hkv, 128), generator=g, device="cuda:0").to(torch.bfloat16)
        vn = torch.randn((spec.batch, hkv, 128), generator=g, device="cuda:0").to(torch.bfloat16)
        P.concur_kv_append(attn.handle, kn, vn, k_dev, v_dev, w.block_table, lens, spec.batch, w.num_pages,
                           w.block_table.shape[1], stream)
        out, lse = attn(w.q, k_dev, v_dev, w.block_table, lens, w.scale)
        torch.cuda.synchronize()
        assert attn.status() == 0
        kvc.kv_append(k_ref, v_ref, w.table_host, lens_ref, kn.cpu().view(torch.int16).numpy(),
                      vn.cpu().view(torch.int16).numpy())
        assert np.array_equal(lens.cpu().numpy(), lens_ref)
        ref_out, ref_lse = oracle.decode_attn(w.q, k_ref.view(np.uint16), v_ref.view(np.uint16), w.table_host,
                                              lens_ref, w.scale)
        assert_parity(out, lse, ref_out, ref_lse, f"append step {step} hkv {hkv} token_major {token_major}")
    k_back = (k_dev.permute(0, 2, 1, 3) if token_major else k_dev).contiguous().cpu().view(torch.int16).numpy()
    assert np.array_equal(k_back, k_ref)
    attn.close()


def test_host_entry_point_with_one_kv_head(P):
    spec = synth.tiny_spec("kv1host", (300, 0, 4099, 64), 64, 8700, num_q_heads=8, num_kv_heads=1)
    w = synth.make_workload(spec, "cpu")
    attn = handle_for(P, w)
    out = torch.empty_like(w.q)
    lse = torch.empty((spec.batch, 8), dtype=torch.float32)
    P.concur_decode_attn_host(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out, lse,
                              spec.batch, w.num_pages, w.block_table.shape[1], 0)
    ref_out, ref_lse = oracle_sequences(w)
    assert_parity(out, lse, ref_out, ref_lse, "host entry, 1 KV head")
    attn.close()


def test_unsupported_kv_head_counts_are_rejected(P):
    B = P.binding
    for hq, hkv in ((8, 0), (72, 9), (64, 16), (7, 2), (18, 2), (9, 1)):
        cfg = B.make_config(64, 4, 8, 0, num_q_heads=hq, num_kv_heads=hkv)
        assert B.concur_attn_workspace_bytes(cfg) == 0, (hq, hkv)
