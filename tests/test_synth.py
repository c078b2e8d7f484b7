"""The seeded input generators: shapes, ranges, structure and determinism."""
import numpy as np
import torch

import synth


def test_lengths_follow_their_recipes():
    l2 = synth.make_lengths(synth.SPECS["cfg2_b16_u1k_8k_p16"])
    assert l2.shape == (16,) and l2.min() >= 1024 and l2.max() <= 8192
    l3 = synth.make_lengths(synth.SPECS["cfg3_b64_ctx16384_p64"])
    assert (l3 == 16384).all() and l3.sum() == 1_048_576
    l4 = synth.make_lengths(synth.SPECS["cfg4_b256_logu2k_32k_p64"])
    assert l4.shape == (256,) and l4.min() >= 2048 and l4.max() <= 32768
    assert 2.0e6 < l4.sum() < 3.7e6          # log-uniform mean is about 11,080
    assert np.median(l4) < l4.mean()         # right-skewed, as log-uniform is
    l5 = synth.make_lengths(synth.SPECS["cfg5_b32_skew128k_p64"])
    assert l5[0] == 131072 and l5[1:].min() >= 256 and l5[1:].max() <= 4096


def test_block_table_is_a_permutation_of_the_pool():
    spec = synth.SPECS["cfg2_b16_u1k_8k_p16"]
    lens = synth.make_lengths(spec)
    table, num_pages = synth.make_block_table(spec, lens)
    used = table[table >= 0]
    assert num_pages == int(((lens + 15) // 16).sum()) == used.size
    assert np.array_equal(np.sort(used), np.arange(num_pages))
    assert not np.array_equal(used, np.arange(num_pages))           # shuffled
    for b, n in enumerate(lens):
        assert (table[b, : -(-n // 16)] >= 0).all() and (table[b, -(-n // 16):] == -1).all()
    t1, _ = synth.make_block_table(synth.SPECS["cfg1_b1_ctx512_p16"], np.array([512], np.int32))
    assert np.array_equal(t1[0], np.arange(32))


def test_workload_is_deterministic_and_poisoned():
    spec = synth.tiny_spec("t", (5, 16, 33, 0), 16, 99)
    a = synth.make_workload(spec, "cpu")
    b = synth.make_workload(spec, "cpu")
    for x, y in ((a.q, b.q), (a.k_pages, b.k_pages), (a.v_pages, b.v_pages)):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    assert a.q.dtype == torch.bfloat16 and a.k_pages.shape == (1 + 1 + 3, 8, 16, 128)
    # slots past the end of a sequence hold NaN; used slots are finite
    page = int(a.table_host[0, 0])
    assert torch.isnan(a.k_pages[page, :, 5:, :].float()).all()
    assert torch.isfinite(a.k_pages[page, :, :5, :].float()).all()
    assert torch.isfinite(a.v_pages[int(a.table_host[1, 0])].float()).all()
    assert a.kv_tokens == 54
    assert a.algorithmic_bytes() == 54 * 4096 + 4 * (2 * 64 * 128 * 2 + 64 * 4 + 4) + 5 * 4


def test_outlier_rows_hit_all_kv_heads():
    spec = synth.tiny_spec("o", (4096,), 64, 5, k_outlier_prob=0.01)
    w = synth.make_workload(spec, "cpu")
    rms = w.k_pages.float().pow(2).mean(dim=(1, 3)).sqrt()       # [pages][P]: rms over heads and dim
    hit = rms > 5.0
    frac = hit.float().mean().item()
    assert 0.003 < frac < 0.025
    per_head = w.k_pages.float().pow(2).mean(dim=3).sqrt()        # [pages][Hkv][P]
    assert (per_head.permute(0, 2, 1)[hit] > 10.0).all()          # every head of a hit slot is scaled
    assert abs(w.v_pages.float().std().item() - 1.0) < 0.02        # V untouched
