"""A token step of a model with several layers: one set of lengths, one pair of pools per layer.
Plan once and attend once per layer (concur_attn_plan / concur_decode_attn_planned), append per
layer (concur_kv_append_layer), the whole step replayed from one CUDA graph, with calls allowed to
overlap -- every layer of every step against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import kv_cache
from helpers import assert_parity, oracle_sequences

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def layer_workloads(lens, page_size, seed, layers, spare, **kw):
    """`layers` workloads with the same lengths and block table and their own q / K / V values."""
    spec = synth.tiny_spec("layers", lens, page_size, seed, **kw)
    ws = [synth.make_workload(spec, "cuda:0", spare_tokens=spare, value_seed=seed + 7919 * i) for i in range(layers)]
    for w in ws[1:]:
        assert torch.equal(w.block_table, ws[0].block_table) and not torch.equal(w.q, ws[0].q)
    return ws


@pytest.mark.parametrize("batch,page_size", [(600, 16), (1100, 64), (513, 32)])
def test_plan_once_attend_per_layer_beyond_the_in_kernel_plan(P, batch, page_size):
    lens = [1 + (53 * i) % 300 for i in range(batch)]
    lens[7] = 0; lens[batch - 1] = 5000
    ws = layer_workloads(lens, page_size, 9300 + page_size, 3, 0)
    w0 = ws[0]
    attn = P.DecodeAttention(page_size, batch, w0.block_table.shape[1], 0)
    stream = torch.cuda.current_stream().cuda_stream
    B = P.binding
    out = torch.full_like(w0.q, 7.0)
    lse = torch.full((batch, 64), 7.0, dtype=torch.float32, device="cuda:0")

    def planned(w, check=True):
        return P.concur_decode_attn_planned(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w0.seq_lens, w.scale,
                                            out, lse, batch, w.num_pages, w.block_table.shape[1], stream, check=check)

    # without a plan call a batch this large is refused
    assert planned(w0, check=False) == B.CONCUR_ERR_INVALID_ARG
    P.concur_attn_plan(attn.handle, w0.seq_lens, batch, w0.block_table.shape[1], stream)
    for i, w in enumerate(ws):
        out.fill_(7.0); lse.fill_(7.0)
        planned(w)
        torch.cuda.synchronize()
        assert attn.status() == 0
        ref_out, ref_lse = oracle_sequences(synth.gather_sequences(w, range(batch)))
        assert_parity(out, lse, ref_out, ref_lse, f"planned call, layer {i}, batch {batch}")
    # another kind of call in between overwrites the plan: the next planned call is refused, not wrong
    attn(w0.q, w0.k_pages, w0.v_pages, w0.block_table, w0.seq_lens, w0.scale, out=out, lse=lse)
    assert planned(w0, check=False) == B.CONCUR_ERR_INVALID_ARG
    # a plan made for other lengths (another pointer) does not count either
    other = w0.seq_lens.clone()
    P.concur_attn_plan(attn.handle, other, batch, w0.block_table.shape[1], stream)
    assert planned(w0, check=False) == B.CONCUR_ERR_INVALID_ARG
    torch.cuda.synchronize()
    attn.close()


@pytest.mark.parametrize("batch,page_size,overlap", [(5, 16, 0), (5, 16, 1), (40, 64, 1), (600, 16, 1)])
def test_four_layers_three_steps_from_one_graph(P, batch, page_size, overlap):
    layers, steps = 4, 3
    base = [100, 63, 0, 1000, 15]
    lens0 = [base[i % 5] + 3 * (i // 5) for i in range(batch)]
    ws = layer_workloads(lens0, page_size, 9400 + page_size + batch, layers, steps)
    w0 = ws[0]
    stride = w0.block_table.shape[1]
    attn = P.DecodeAttention(page_size, batch, stride, 0)
    attn.set_option(P.CONCUR_OPT_OVERLAP_CALLS, overlap)
    g = torch.Generator(device="cuda:0"); g.manual_seed(9500 + batch)
    k_new = torch.randn((layers, batch, 8, 128), generator=g, device="cuda:0").to(torch.bfloat16)
    v_new = torch.randn((layers, batch, 8, 128), generator=g, device="cuda:0").to(torch.bfloat16)
    lens = w0.seq_lens.clone()
    outs = [torch.full_like(w0.q, 7.0) for _ in range(layers)]
    lses = [torch.full((batch, 64), 7.0, dtype=torch.float32, device="cuda:0") for _ in range(layers)]

    def token_step():
        s = torch.cuda.current_stream().cuda_stream
        # the first layer's append opens the slot and advances the lengths; the plan is made after it
        for i, w in enumerate(ws):
            P.concur_kv_append_layer(attn.handle, k_new[i], v_new[i], w.k_pages, w.v_pages, w.block_table, lens, batch,
                                     w.num_pages, stride, 1 if i == 0 else 0, s)
        P.concur_attn_plan(attn.handle, lens, batch, stride, s)
        for i, w in enumerate(ws):
            P.concur_decode_attn_planned(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, lens, w.scale,
                                         outs[i], lses[i], batch, w.num_pages, stride, s)

    # host-side reference state of every layer's cache
    ref = [(bits(w.k_pages), bits(w.v_pages)) for w in ws]
    table = w0.table_host
    lens_ref = np.array(lens0, dtype=np.int32)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        token_step()                                      # warm-up outside the capture (first-call set-up)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    # undo the warm-up step's effect on the lengths; its rows are rewritten identically by the first replay
    lens.copy_(w0.seq_lens)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        token_step()
    for step in range(steps):
        graph.replay()
        torch.cuda.synchronize()
        assert attn.status() == 0
        for i in range(layers):
            kv_cache.kv_append(ref[i][0], ref[i][1], table, lens_ref, bits(k_new[i]), bits(v_new[i]), advance=(i == 0))
        assert np.array_equal(lens.cpu().numpy(), lens_ref)
        for i, w in enumerate(ws):
            ref_out, ref_lse = oracle.decode_attn(w.q, ref[i][0], ref[i][1], table, lens_ref, w.scale)
            assert_parity(outs[i], lses[i], ref_out, ref_lse, f"step {step} layer {i} batch {batch} overlap {overlap}")
    for i, w in enumerate(ws):
        assert np.array_equal(bits(w.k_pages), ref[i][0]) and np.array_equal(bits(w.v_pages), ref[i][1])
    attn.close()


def test_plain_calls_back_to_back_with_overlap_allowed(P):
    # many single-launch calls in a row on different layers' pools, each allowed to start while the one
    # before drains; every one must still claim every range exactly once and find its counters at zero
    lens = [3000, 1, 64, 777, 9000, 0, 130, 2048]
    ws = layer_workloads(lens, 64, 9600, 6, 0)
    attn = P.DecodeAttention(64, len(lens), ws[0].block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_OVERLAP_CALLS, 1)
    results = []
    for rep in range(3):
        for w in ws:
            results.append(attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale))
    torch.cuda.synchronize()
    assert attn.status() == 0
    refs = [oracle_sequences(synth.gather_sequences(w, range(len(lens)))) for w in ws]
    for n, (out, lse) in enumerate(results):
        assert_parity(out, lse, *refs[n % len(ws)], f"call {n}")
    attn.close()


def test_append_layer_argument_errors(P):
    B = P.binding
    w = synth.make_workload(synth.tiny_spec("al", (5, 0), 16, 9700), "cuda:0", spare_tokens=2)
    attn = P.DecodeAttention(16, 2, w.block_table.shape[1], 0)
    kn = torch.zeros((2, 8, 128), dtype=torch.bfloat16, device="cuda:0")
    lens = w.seq_lens.clone()
    rc = B.concur_kv_append_layer(attn.handle, kn, kn, w.k_pages, w.v_pages, w.block_table, lens, 2, w.num_pages,
                                  w.block_table.shape[1], 2, 0, check=False)
    assert rc == B.CONCUR_ERR_INVALID_ARG
    # advance = 0 on a sequence without tokens: no slot to fill, flagged, nothing written, lengths untouched
    before = w.k_pages.clone()
    B.concur_kv_append_layer(attn.handle, kn, kn, w.k_pages, w.v_pages, w.block_table, lens, 2, w.num_pages,
                             w.block_table.shape[1], 0, 0)
    torch.cuda.synchronize()
    assert attn.status() & P.CONCUR_FLAG_BAD_SEQ_LEN
    assert lens.tolist() == [5, 0]
    changed = (w.k_pages.view(torch.int16) != before.view(torch.int16)).any(dim=3).sum().item()
    assert changed == 8                                   # sequence 0's slot 4, all 8 KV heads
    attn.close()


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
@pytest.mark.parametrize("token_major", [0, 1])
@pytest.mark.parametrize("hkv,hq,ranges", [(8, 64, 0), (8, 64, 37), (2, 10, 0), (1, 8, 5)])
def test_fused_append_equals_append_then_attend(P, page_size, token_major, hkv, hq, ranges):
    # lengths already count the new token: it is the only token (1), the last slot of a page / tile (64, 128),
    # the first slot of a fresh one (65, 129, 17), somewhere inside; 0 = no token at all
    lens = (0, 1, 2, 16, 17, 63, 64, 65, 128, 129, 200, 1000, 1025, 4099)
    spec = synth.tiny_spec(f"fa_p{page_size}", lens, page_size, 9800 + page_size + hkv, num_q_heads=hq, num_kv_heads=hkv)
    w = synth.make_workload(spec, "cuda:0")
    B = spec.batch
    g = torch.Generator(device="cuda:0"); g.manual_seed(9900 + page_size)
    kn = torch.randn((B, hkv, 128), generator=g, device="cuda:0").to(torch.bfloat16)
    vn = torch.randn((B, hkv, 128), generator=g, device="cuda:0").to(torch.bfloat16)
    # the slot of every sequence's newest token holds garbage until the call stores the rows there
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16, device="cuda:0")
    for b, n in enumerate(lens):
        if n:
            page = int(w.table_host[b, (n - 1) // page_size])
            w.k_pages[page, :, (n - 1) % page_size, :] = nan
            w.v_pages[page, :, (n - 1) % page_size, :] = nan
    # reference: the layer append of the write-path reference, then the attention oracle
    k_ref, v_ref = bits(w.k_pages), bits(w.v_pages)
    lens_ref = np.array(lens, dtype=np.int32)
    kv_cache.kv_append(k_ref, v_ref, w.table_host, lens_ref, bits(kn), bits(vn), advance=False)
    assert np.array_equal(lens_ref, np.array(lens, dtype=np.int32))
    ref_out, ref_lse = oracle.decode_attn(w.q, k_ref, v_ref, w.table_host, lens_ref, w.scale)
    k_dev, v_dev = w.k_pages, w.v_pages
    if token_major:
        k_dev = k_dev.permute(0, 2, 1, 3).contiguous(); v_dev = v_dev.permute(0, 2, 1, 3).contiguous()
    attn = P.DecodeAttention(page_size, B, w.block_table.shape[1], 0, num_q_heads=hq, num_kv_heads=hkv,
                             kv_layout=token_major)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    out = torch.full_like(w.q, 7.0)
    lse = torch.full((B, hq), 7.0, dtype=torch.float32, device="cuda:0")
    lens_dev = w.seq_lens.clone()
    P.concur_decode_attn_append(attn.handle, w.q, kn, vn, k_dev, v_dev, w.block_table, lens_dev, w.scale, out, lse, B,
                                w.num_pages, w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert torch.equal(lens_dev, w.seq_lens)                      # lengths are only read
    assert_parity(out, lse, ref_out, ref_lse, f"fused append p{page_size} tm{token_major} hkv{hkv} R{ranges}")
    k_back = (k_dev.permute(0, 2, 1, 3) if token_major else k_dev).contiguous()
    v_back = (v_dev.permute(0, 2, 1, 3) if token_major else v_dev).contiguous()
    assert np.array_equal(bits(k_back), k_ref) and np.array_equal(bits(v_back), v_ref)   # byte for byte
    # and the plain call on the pools as they are now gives the same again
    out2, lse2 = attn(w.q, k_dev, v_dev, w.block_table, lens_dev, w.scale)
    torch.cuda.synchronize()
    assert_parity(out2, lse2, ref_out, ref_lse, "plain call after the fused one")
    attn.close()


def test_fused_append_needs_the_fused_tensor_core_path_and_flags_bad_pages(P):
    B_ = P.binding
    spec = synth.tiny_spec("fa_err", (70, 5), 64, 9950)
    w = synth.make_workload(spec, "cuda:0")
    kn = torch.zeros((2, 8, 128), dtype=torch.bfloat16, device="cuda:0")
    out = torch.empty_like(w.q); lse = torch.empty((2, 64), dtype=torch.float32, device="cuda:0")
    attn = P.DecodeAttention(64, 2, w.block_table.shape[1], 0)

    def call(k_new=kn, table=w.block_table):
        return B_.concur_decode_attn_append(attn.handle, w.q, k_new, kn, w.k_pages, w.v_pages, table, w.seq_lens, w.scale,
                                            out, lse, 2, w.num_pages, w.block_table.shape[1], 0, check=False)
    attn.set_option(P.CONCUR_OPT_KERNEL, 1)
    assert call() == B_.CONCUR_ERR_UNSUPPORTED
    attn.set_option(P.CONCUR_OPT_KERNEL, 0)
    attn.set_option(P.CONCUR_OPT_FUSE_COMBINE, 0)
    assert call() == B_.CONCUR_ERR_UNSUPPORTED
    attn.set_option(P.CONCUR_OPT_FUSE_COMBINE, 1)
    assert call(k_new=None) == B_.CONCUR_ERR_INVALID_ARG
    # the page of sequence 1's newest token lies outside the pool: flagged, nothing stored, nothing faults
    bad = w.block_table.clone(); bad[1, 0] = w.num_pages + 7
    before = w.k_pages.clone()
    assert call(table=bad) == B_.CONCUR_OK
    torch.cuda.synchronize()
    assert attn.status() & P.CONCUR_FLAG_BAD_PAGE_ID
    changed = (w.k_pages.view(torch.int16) != before.view(torch.int16)).any(dim=3).sum().item()
    assert changed <= 8                                           # at most sequence 0's slot, all 8 KV heads
    attn.close()
