"""Pins for the CPU oracle: what mathematics fixes about softmax(scale q K^T) V over a paged
cache, checked without reference to the oracle's own formula.  A dropped term, a wrong
sign or index, a transposed operand or a wrong head map in oracle/attn_oracle.c fails
at least one of these."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import brute_force
import synth


def bf16(x):
    """float array -> bf16 bit patterns (uint16), round to nearest even."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_val(bits):
    return torch.from_numpy(np.asarray(bits).view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


def simple_case(q, k, v, P=4, Hkv=1):
    """Single sequence, identity table.  q [Hq][D], k/v [n][Hkv][D] floats (bf16-exact or not)."""
    q = np.asarray(q, dtype=np.float32)
    k = np.asarray(k, dtype=np.float32)
    v = np.asarray(v, dtype=np.float32)
    n, _, D = k.shape
    pages = max(1, -(-n // P))
    kp = np.zeros((pages, Hkv, P, D), dtype=np.float32)
    vp = np.zeros_like(kp)
    for j in range(n):
        kp[j // P, :, j % P, :] = k[j]
        vp[j // P, :, j % P, :] = v[j]
    table = np.arange(pages, dtype=np.int32)[None, :]
    return bf16(q[None]), bf16(kp), bf16(vp), table, np.array([n], dtype=np.int32)


def test_single_token_returns_v_row_exactly():
    rng = np.random.default_rng(1)
    D = 128
    q = rng.standard_normal((8, D))
    k = rng.standard_normal((1, 1, D))
    v = rng.standard_normal((1, 1, D))
    qb, kb, vb, tab, lens = simple_case(q, k, v, P=16)
    scale = 0.0883883461356163
    out, lse = oracle.decode_attn(qb, kb, vb, tab, lens, scale)
    vrow = bf16_val(vb[0, 0, 0])
    for h in range(8):
        assert np.array_equal(out[0, h], vrow)           # weight is exactly 1
        dot = math.fsum(float(a) * float(b) for a, b in zip(bf16_val(qb[0, h]), bf16_val(kb[0, 0, 0])))
        assert lse[0, h] == pytest.approx(float(np.float32(scale)) * dot, rel=1e-14, abs=1e-14)


def test_constant_scores_give_mean_of_v():
    rng = np.random.default_rng(2)
    n, D = 37, 16
    v = rng.standard_normal((n, 1, D))
    # (i) q = 0
    qb, kb, vb, tab, lens = simple_case(np.zeros((2, D)), rng.standard_normal((n, 1, D)), v, P=8)
    out, lse = oracle.decode_attn(qb, kb, vb, tab, lens, 0.7)
    mean = bf16_val(vb).reshape(-1, D)[:n].mean(axis=0)
    np.testing.assert_allclose(out[0, 0], mean, rtol=1e-14, atol=1e-15)
    assert lse[0, 1] == pytest.approx(math.log(n), rel=1e-15)
    # (ii) every K row equal: score s for all tokens
    krow = rng.standard_normal(D)
    q = rng.standard_normal((1, D))
    qb, kb, vb, tab, lens = simple_case(q, np.tile(krow, (n, 1, 1)), v, P=8)
    out, lse = oracle.decode_attn(qb, kb, vb, tab, lens, 0.25)
    s = 0.25 * float(np.dot(bf16_val(qb[0, 0]), bf16_val(kb[0, 0, 0])))
    np.testing.assert_allclose(out[0, 0], mean, rtol=1e-13, atol=1e-14)
    assert lse[0, 0] == pytest.approx(s + math.log(n), rel=1e-13)


@pytest.mark.parametrize("scale", [0.03125, -0.0625, 0.5])
def test_geometric_series_closed_form(scale):
    # q = e0, k_j = j e0 (exact in bf16 for j <= 256), v_j = j * ones: s_j = scale*j, weights r^j
    n, D = 200, 8
    k = np.zeros((n, 1, D)); k[:, 0, 0] = np.arange(n)
    v = np.tile(np.arange(n, dtype=np.float64)[:, None, None], (1, 1, D))
    q = np.zeros((1, D)); q[0, 0] = 1.0
    qb, kb, vb, tab, lens = simple_case(q, k, v, P=16)
    out, lse = oracle.decode_attn(qb, kb, vb, tab, lens, scale)
    r = math.exp(scale)
    z = (r ** n - 1.0) / (r - 1.0)
    num = r * (1.0 - n * r ** (n - 1) + (n - 1) * r ** n) / (1.0 - r) ** 2
    assert lse[0, 0] == pytest.approx(math.log(z), rel=1e-12)
    np.testing.assert_allclose(out[0, 0], np.full(D, num / z), rtol=1e-11)


def test_two_tokens_quarter_three_quarters():
    D = 4
    q = np.zeros((1, D)); q[0, 1] = 1.0
    k = np.zeros((2, 1, D)); k[1, 0, 1] = 1.0                 # scores (0, scale)
    v = np.zeros((2, 1, D)); v[0, 0, :] = [1, 0, 2, -4]; v[1, 0, :] = [0, 1, 2, 4]
    qb, kb, vb, tab, lens = simple_case(q, k, v, P=2)
    out, lse = oracle.decode_attn(qb, kb, vb, tab, lens, math.log(3.0))
    np.testing.assert_allclose(out[0, 0], [0.25, 0.75, 2.0, 2.0], rtol=0, atol=2e-7)
    assert lse[0, 0] == pytest.approx(math.log(4.0), abs=2e-7)


def _tiny_workload(seed=11, lens=(5, 16, 33, 1, 0, 47), P=16):
    return synth.make_workload(synth.tiny_spec("tiny", lens, P, seed), "cpu")


def test_page_permutation_invariance_bit_exact():
    w = _tiny_workload()
    out0, lse0 = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    rng = np.random.default_rng(5)
    perm = rng.permutation(w.num_pages)              # new physical id of old page p is perm[p]
    k2 = torch.empty_like(w.k_pages); v2 = torch.empty_like(w.v_pages)
    k2[perm] = w.k_pages; v2[perm] = w.v_pages
    tab2 = w.table_host.copy()
    tab2[tab2 >= 0] = perm[tab2[tab2 >= 0]]
    out1, lse1 = oracle.decode_attn(w.q, k2, v2, tab2, w.seq_lens, w.scale)
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


def test_token_order_invariance():
    rng = np.random.default_rng(6)
    n, D = 50, 32
    q = rng.standard_normal((4, D)); k = rng.standard_normal((n, 2, D)); v = rng.standard_normal((n, 2, D))
    a = oracle.decode_attn(*simple_case(q, k, v, P=8, Hkv=2), 0.3)
    p = rng.permutation(n)
    b = oracle.decode_attn(*simple_case(q, k[p], v[p], P=8, Hkv=2), 0.3)
    np.testing.assert_allclose(a[0], b[0], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(a[1], b[1], rtol=1e-13)


def test_shift_invariance():
    # a K column that is constant over tokens, paired with q = 1 there, shifts every score
    rng = np.random.default_rng(7)
    n, D = 40, 16
    q = rng.standard_normal((2, D)); q[:, 3] = 1.0
    k = rng.standard_normal((n, 1, D)); v = rng.standard_normal((n, 1, D))
    k0 = k.copy(); k0[:, :, 3] = 0.0
    k1 = k.copy(); k1[:, :, 3] = 6.5
    a = oracle.decode_attn(*simple_case(q, k0, v, P=8), 0.5)
    b = oracle.decode_attn(*simple_case(q, k1, v, P=8), 0.5)
    np.testing.assert_allclose(a[0], b[0], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(b[1] - a[1], 0.5 * 6.5, rtol=1e-12)


def test_split_consistency_defines_the_merge():
    w = _tiny_workload(seed=12, lens=(97, 130), P=16)
    whole, lse_whole = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    for b, n in enumerate(w.lens_host):
        for h in (0, 9, 63):
            for cuts in ([0, 40, n], [0, 1, 64, 65, n], [0, n, n], [0, 0, n]):
                parts = [oracle.attn_range(w.q, w.k_pages, w.v_pages, w.block_table, w.scale, b, h, a, e)
                         for a, e in zip(cuts[:-1], cuts[1:])]
                out, lse = oracle.lse_merge(np.stack([p[0] for p in parts]), [p[1] for p in parts])
                np.testing.assert_allclose(out, whole[b, h], rtol=1e-12, atol=1e-14)
                assert lse == pytest.approx(lse_whole[b, h], rel=1e-13)
    out, lse = oracle.lse_merge(np.zeros((2, 4)), [-math.inf, -math.inf])
    assert lse == -math.inf and not out.any()


def test_output_is_a_convex_combination_and_ignores_poison():
    w = _tiny_workload(seed=13, lens=(5, 16, 33, 1, 0, 47), P=16)
    out, lse = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    assert np.isfinite(out).all()                     # the NaN-filled unused slots are never read
    v = w.v_pages.to(torch.float64).numpy()
    for b, n in enumerate(w.lens_host):
        if n == 0:
            assert not out[b].any() and np.all(lse[b] == -np.inf)
            continue
        rows = np.stack([v[w.table_host[b, j // 16], :, j % 16, :] for j in range(n)])   # [n][Hkv][D]
        for h in range(64):
            g = h // 8
            assert np.all(out[b, h] <= rows[:, g].max(axis=0) + 1e-12)
            assert np.all(out[b, h] >= rows[:, g].min(axis=0) - 1e-12)
        assert np.all(np.isfinite(lse[b]))


def test_brute_force_tiny():
    spec = synth.tiny_spec("bf", (3, 8, 1, 0, 6), 4, 21, num_q_heads=4, num_kv_heads=2, head_dim=4)
    w = synth.make_workload(spec, "cpu")
    # brute force indexes every pool slot of used tokens only; hand it plain nested lists of bits
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16).tolist()
    ref_out, ref_lse = brute_force.decode_attn_naive(
        bits(w.q), bits(w.k_pages), bits(w.v_pages), w.table_host.tolist(), w.lens_host.tolist(),
        w.scale, 4, 2, 4, 4)
    out, lse = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    np.testing.assert_allclose(out, np.array(ref_out), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(lse, np.array(ref_lse), rtol=1e-13)


def test_library_second_opinion_torch_fp64():
    # de-paged, head-expanded tensors through torch's own softmax / matmul
    w = _tiny_workload(seed=14, lens=(70, 129, 16), P=16)
    out, lse = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    scale = float(np.float32(w.scale))
    for b, n in enumerate(w.lens_host):
        pages = torch.from_numpy(w.table_host[b, : -(-n // 16)].astype(np.int64))
        k = w.k_pages[pages].permute(1, 0, 2, 3).reshape(8, -1, 128)[:, :n].double()   # [Hkv][n][D]
        v = w.v_pages[pages].permute(1, 0, 2, 3).reshape(8, -1, 128)[:, :n].double()
        k = k.repeat_interleave(8, dim=0); v = v.repeat_interleave(8, dim=0)           # [Hq][n][D]
        s = torch.einsum("hd,hnd->hn", w.q[b].double(), k) * scale
        ref = torch.einsum("hn,hnd->hd", torch.softmax(s, dim=-1), v)
        np.testing.assert_allclose(out[b], ref.numpy(), rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(lse[b], torch.logsumexp(s, dim=-1).numpy(), rtol=1e-12)


def test_subset_selection_matches_full():
    w = _tiny_workload(seed=15, lens=(20, 40, 60), P=16)
    full = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    part = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale,
                              seqs=(1, 2), heads=(8, 16))
    assert np.array_equal(part[0][1, 8:16], full[0][1, 8:16])
    assert np.isnan(part[0][0]).all() and np.isnan(part[0][1, :8]).all()
    sub = synth.gather_sequences(w, [2, 0])
    o2, l2 = oracle.decode_attn(sub.q, sub.k_pages, sub.v_pages, sub.block_table, sub.seq_lens, sub.scale)
    assert np.array_equal(o2[0], full[0][2]) and np.array_equal(o2[1], full[0][0])
    assert np.array_equal(l2[1], full[1][0])


def test_frozen_tiny_case_has_not_drifted():
    # regression fixture written by tests/golden/make_golden.py from the oracle alone
    import importlib.util
    import json
    import os
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(here, "golden", "tiny_decode_oracle.json")) as f:
        gold = json.load(f)
    w, out, lse = mod.compute()
    assert w.q.view(-1)[:8].view(dtype=torch.int16).tolist() == gold["q_first_bits"], "input generator drifted"
    np.testing.assert_allclose(lse, np.array([[float(x) for x in r] for r in gold["lse"]]), rtol=1e-13)
    got = np.array([[out[b, h, :4] for h in range(0, 64, 8)] for b in range(4)])
    want = np.array([[[float(x) for x in hrow] for hrow in brow] for brow in gold["out_first4"]])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
