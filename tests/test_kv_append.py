"""The cache's write path: the CPU reference is pinned against the layout's definition
(appending T tokens yields the concatenation, nothing else moves); the CUDA append and a
multi-step append + attention loop (eager and replayed from a CUDA graph) are checked
against it and against the attention oracle."""
import numpy as np
import pytest
import torch

import synth
from oracle import kv_cache
from helpers import assert_parity, oracle_sequences


def bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def test_reference_append_is_concatenation():
    rng = np.random.default_rng(3)
    P, hkv, D = 4, 2, 8
    lens0 = np.array([0, 3, 4, 9], dtype=np.int32)
    steps = 6
    pages_per = -(-(lens0 + steps) // P)
    table = np.full((4, pages_per.max() + 1), -1, dtype=np.int32)
    perm = rng.permutation(int(pages_per.sum()))
    at = 0
    for b, n in enumerate(pages_per):
        table[b, :n] = perm[at:at + n]; at += n
    k = rng.integers(0, 65536, size=(at, hkv, P, D)).astype(np.uint16)
    v = rng.integers(0, 65536, size=(at, hkv, P, D)).astype(np.uint16)
    k0, v0 = k.copy(), v.copy()
    lens = lens0.copy()
    new_k = rng.integers(0, 65536, size=(steps, 4, hkv, D)).astype(np.uint16)
    new_v = rng.integers(0, 65536, size=(steps, 4, hkv, D)).astype(np.uint16)
    for s in range(steps):
        kv_cache.kv_append(k, v, table, lens, new_k[s], new_v[s])
    assert np.array_equal(lens, lens0 + steps)
    for b in range(4):
        got = kv_cache.gather_tokens(k, table, b, int(lens[b]))
        want = np.concatenate([kv_cache.gather_tokens(k0, table, b, int(lens0[b])), new_k[:, b]])
        assert np.array_equal(got, want)
        assert np.array_equal(kv_cache.gather_tokens(v, table, b, int(lens[b]))[int(lens0[b]):], new_v[:, b])
    # exactly steps * batch * hkv rows changed in each pool (random 16-bit rows differ with certainty ~1)
    changed = (k != k0).any(axis=3).sum()
    assert changed == steps * 4 * hkv
    # a full table row and a bad page id leave everything untouched
    lens_full = np.array([table.shape[1] * P, 0, 0, 0], dtype=np.int32)
    bad = table.copy(); bad[1, 0] = at + 5
    k1 = k.copy()
    kv_cache.kv_append(k, v, bad, lens_full, new_k[0], new_v[0])
    assert lens_full[0] == table.shape[1] * P and lens_full[1] == 0 and lens_full[2] == 1
    assert (k != k1).any(axis=3).sum() == 2 * hkv          # only sequences 2 and 3 were written


def test_reference_append_for_the_further_layers_of_a_step():
    # two layers, one set of lengths: the first layer's append opens the slot and advances, the second
    # layer's append (advance=False) fills the same slot of its own pools; after T steps both layers hold
    # their own concatenation and the lengths have grown by T, not 2 T
    rng = np.random.default_rng(5)
    P, hkv, D, steps, B = 4, 2, 8, 5, 3
    lens0 = np.array([0, 3, 8], dtype=np.int32)
    pages_per = -(-(lens0 + steps) // P)
    table = np.full((B, pages_per.max()), -1, dtype=np.int32)
    perm = rng.permutation(int(pages_per.sum()))
    at = 0
    for b, n in enumerate(pages_per):
        table[b, :n] = perm[at:at + n]; at += n
    pools = [[rng.integers(0, 65536, size=(at, hkv, P, D)).astype(np.uint16) for _ in range(2)] for _ in range(2)]
    before = [[x.copy() for x in layer] for layer in pools]
    new = rng.integers(0, 65536, size=(steps, 2, 2, B, hkv, D)).astype(np.uint16)      # [step][layer][k|v]
    lens = lens0.copy()
    for s in range(steps):
        kv_cache.kv_append(pools[0][0], pools[0][1], table, lens, new[s, 0, 0], new[s, 0, 1])
        kv_cache.kv_append(pools[1][0], pools[1][1], table, lens, new[s, 1, 0], new[s, 1, 1], advance=False)
        assert np.array_equal(lens, lens0 + s + 1)
    for layer in range(2):
        for kv in range(2):
            for b in range(B):
                got = kv_cache.gather_tokens(pools[layer][kv], table, b, int(lens[b]))
                want = np.concatenate([kv_cache.gather_tokens(before[layer][kv], table, b, int(lens0[b])),
                                       new[:, layer, kv, b]])
                assert np.array_equal(got, want)
            assert (pools[layer][kv] != before[layer][kv]).any(axis=3).sum() == steps * B * hkv
    # a sequence with no token yet has no slot for a further layer to fill: nothing moves
    k, v = pools[1][0].copy(), pools[1][1].copy()
    zero = np.zeros(B, dtype=np.int32)
    kv_cache.kv_append(k, v, table, zero, new[0, 1, 0], new[0, 1, 1], advance=False)
    assert np.array_equal(k, pools[1][0]) and np.array_equal(zero, np.zeros(B, dtype=np.int32))


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def _loop_case(page_size, lens0, steps, seed):
    final = synth.make_workload(synth.tiny_spec("loop", [n + steps for n in lens0], page_size, seed), "cuda:0")
    B = len(lens0)
    idx = torch.arange(B, device="cuda:0")
    k_new = torch.empty((steps, B, 8, 128), dtype=torch.bfloat16, device="cuda:0")
    v_new = torch.empty_like(k_new)
    k0, v0 = final.k_pages.clone(), final.v_pages.clone()
    table = final.block_table.long()
    for s in range(steps):
        pos = torch.tensor([n + s for n in lens0], device="cuda:0")
        page = table[idx, pos // page_size]
        k_new[s] = final.k_pages[page, :, pos % page_size, :]
        v_new[s] = final.v_pages[page, :, pos % page_size, :]
        k0[page, :, pos % page_size, :] = float("nan")       # not written yet
        v0[page, :, pos % page_size, :] = float("nan")
    g = torch.Generator(device="cuda:0"); g.manual_seed(seed)
    q_steps = torch.randn((steps, B, 64, 128), generator=g, device="cuda:0").to(torch.bfloat16)
    return final, k0, v0, k_new, v_new, q_steps


def _check_step(final, lens_now, q, out, lse, what):
    host = synth.gather_sequences(final, range(final.spec.batch))
    host.q = q.cpu()
    host.seq_lens = torch.tensor(lens_now, dtype=torch.int32)
    host.lens_host = np.array(lens_now, dtype=np.int32)
    ref_out, ref_lse = oracle_sequences(host)
    assert_parity(out, lse, ref_out, ref_lse, what)


@pytest.mark.gpu
@pytest.mark.parametrize("page_size", [16, 64, 128])
def test_append_then_attend_loop(P, page_size):
    lens0, steps = [100, 63, 0, 1000, 15], 5
    final, k, v, k_new, v_new, q_steps = _loop_case(page_size, lens0, steps, 900 + page_size)
    B = len(lens0)
    attn = P.DecodeAttention(page_size, B, final.block_table.shape[1], 0)
    lens = torch.tensor(lens0, dtype=torch.int32, device="cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    for s in range(steps):
        P.concur_kv_append(attn.handle, k_new[s], v_new[s], k, v, final.block_table, lens, B, final.num_pages,
                           final.block_table.shape[1], stream)
        out, lse = attn(q_steps[s], k, v, final.block_table, lens, final.scale)
        torch.cuda.synchronize()
        assert lens.tolist() == [n + s + 1 for n in lens0]
        _check_step(final, [n + s + 1 for n in lens0], q_steps[s], out, lse, f"step {s}")
    assert attn.status() == 0
    # byte-exact: the pools now equal the ones the rows were taken from
    assert torch.equal(k.view(torch.int16), final.k_pages.view(torch.int16))
    assert torch.equal(v.view(torch.int16), final.v_pages.view(torch.int16))
    # against the CPU reference of the write path, from the same starting state
    attn.close()


@pytest.mark.gpu
def test_append_matches_cpu_reference_and_flags_bad_rows(P):
    lens0 = [5, 31, 16]
    final, k, v, k_new, v_new, _ = _loop_case(16, lens0, 2, 77)
    B = 3
    attn = P.DecodeAttention(16, B, final.block_table.shape[1], 0)
    kb, vb = bits(k), bits(v)
    tab = final.block_table.cpu().numpy().copy()
    lens_ref = np.array(lens0, dtype=np.int32)
    lens = torch.tensor(lens0, dtype=torch.int32, device="cuda:0")
    for s in range(2):
        kv_cache.kv_append(kb, vb, tab, lens_ref, bits(k_new[s]), bits(v_new[s]))
        P.concur_kv_append(attn.handle, k_new[s], v_new[s], k, v, final.block_table, lens, B, final.num_pages,
                           final.block_table.shape[1], 0)
    torch.cuda.synchronize()
    assert np.array_equal(bits(k), kb) and np.array_equal(bits(v), vb) and lens.cpu().numpy().tolist() == lens_ref.tolist()
    # a full row and a page id outside the pool: untouched, flagged
    bad_table = final.block_table.clone(); bad_table[1, :] = final.num_pages + 3
    lens_bad = torch.tensor([final.block_table.shape[1] * 16, 7, 7], dtype=torch.int32, device="cuda:0")
    before = k.clone()
    P.concur_kv_append(attn.handle, k_new[0], v_new[0], k, v, bad_table, lens_bad, B, final.num_pages,
                       final.block_table.shape[1], 0)
    torch.cuda.synchronize()
    flags = attn.status()
    assert flags & P.CONCUR_FLAG_BAD_SEQ_LEN and flags & P.CONCUR_FLAG_BAD_PAGE_ID
    assert lens_bad.tolist() == [final.block_table.shape[1] * 16, 7, 8]
    assert (k.view(torch.int16) != before.view(torch.int16)).any(dim=3).sum().item() == 8   # sequence 2 only
    attn.close()


@pytest.mark.gpu
def test_decode_loop_replayed_from_a_cuda_graph(P):
    lens0, steps = [300, 64, 2000, 1], 6
    final, k, v, k_new, v_new, q_steps = _loop_case(64, lens0, steps, 555)
    B = len(lens0)
    attn = P.DecodeAttention(64, B, final.block_table.shape[1], 0)
    lens = torch.tensor(lens0, dtype=torch.int32, device="cuda:0")
    q_in = torch.empty_like(q_steps[0]); kn_in = torch.empty_like(k_new[0]); vn_in = torch.empty_like(v_new[0])
    out = torch.empty_like(q_in); lse = torch.empty((B, 64), dtype=torch.float32, device="cuda:0")

    def one_step():
        stream = torch.cuda.current_stream().cuda_stream
        P.concur_kv_append(attn.handle, kn_in, vn_in, k, v, final.block_table, lens, B, final.num_pages,
                           final.block_table.shape[1], stream)
        attn(q_in, k, v, final.block_table, lens, final.scale, out=out, lse=lse)

    # the first call on a device does one-time set-up: make it before the capture, on a scratch copy
    k_keep, v_keep = k.clone(), v.clone()
    q_in.copy_(q_steps[0]); kn_in.copy_(k_new[0]); vn_in.copy_(v_new[0])
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        one_step()
    torch.cuda.synchronize()
    k.copy_(k_keep); v.copy_(v_keep); lens.copy_(torch.tensor(lens0, dtype=torch.int32))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        one_step()
    k.copy_(k_keep); v.copy_(v_keep); lens.copy_(torch.tensor(lens0, dtype=torch.int32))
    for s in range(steps):
        q_in.copy_(q_steps[s]); kn_in.copy_(k_new[s]); vn_in.copy_(v_new[s])
        graph.replay()
        torch.cuda.synchronize()
        assert lens.tolist() == [n + s + 1 for n in lens0]
        _check_step(final, [n + s + 1 for n in lens0], q_steps[s], out, lse, f"graph step {s}")
    assert attn.status() == 0
    attn.close()
