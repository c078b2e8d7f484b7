"""Shared-prefix (cascade) decode: the result is defined as that of the plain step on the same
tables, so the CUDA path is compared with the same CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import synth
from helpers import assert_parity, oracle_sequences

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def run_cascade(P, cw, prefix_lens=None, kernel=0, ranges=0, prefix_kernel=0):
    w = cw.w
    attn = P.DecodeAttention(w.spec.page_size, w.spec.batch, w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    attn.set_option(P.CONCUR_OPT_PREFIX_KERNEL, prefix_kernel)
    out = torch.full_like(w.q, 7.0)
    lse = torch.full((w.spec.batch, 64), 7.0, dtype=torch.float32, device="cuda:0")
    pl = cw.prefix_lens if prefix_lens is None else prefix_lens
    P.concur_decode_attn_cascade(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens,
                                 cw.group_start, pl, w.scale, out, lse, w.spec.batch, len(cw.prefix_lens_host),
                                 w.num_pages, w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out, lse, attn


GROUPS = [
    (1024, [100, 1, 64, 700, 333]),            # five samples of one prompt
    (0, [500]),                                # a singleton
    (2048, [5, 900]),                          # a pair
    (512, [0, 130, 64, 1, 2000, 77, 640, 63, 65, 300]),          # ten samples; one has no tokens of its own
    (256, [10 * j + 1 for j in range(13)]),    # thirteen: the last three read everything themselves
    (0, [0]),                                  # an empty sequence
    (4096, [17, 4000, 260]),
    (64, [1, 2]),
]


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("prefix_kernel", [0, 1])
def test_cascade_matches_oracle(P, page_size, kernel, prefix_kernel):
    """prefix_kernel 0: tcgen05 / TMEM prefix pass; 1: warp-level mma.sync prefix pass."""
    groups = [(shared - shared % page_size, owns) for shared, owns in GROUPS]      # only whole pages can be shared
    cw = synth.make_cascade_workload(f"casc_p{page_size}", groups, page_size, 4000 + page_size, "cuda:0")
    out, lse, attn = run_cascade(P, cw, kernel=kernel, prefix_kernel=prefix_kernel)
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(synth.gather_sequences(cw.w, range(cw.w.spec.batch)))
    assert_parity(out, lse, ref_out, ref_lse, f"cascade p{page_size} kernel {kernel} prefix kernel {prefix_kernel}")
    attn.close()


def test_cascade_equals_plain_step_and_survives_odd_prefix_lens(P):
    cw = synth.make_cascade_workload("casc_odd", GROUPS, 16, 4100, "cuda:0")
    w = cw.w
    plain = P.DecodeAttention(16, w.spec.batch, w.block_table.shape[1], 0)
    out_p, lse_p = plain(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    torch.cuda.synchronize()
    ref_out, ref_lse = oracle_sequences(synth.gather_sequences(w, range(w.spec.batch)))
    # promises weaker than the truth are always valid: fewer shared tokens, not multiples of 64 or of the page
    for delta in (0, 1, 17, 63, 64, 100):
        pl = torch.clamp(cw.prefix_lens - delta, min=0)
        out, lse, attn = run_cascade(P, cw, prefix_lens=pl)
        assert attn.status() == 0
        assert_parity(out, lse, ref_out, ref_lse, f"prefix - {delta}")
        assert (out.float() - out_p.float()).abs().max().item() <= 2e-2
        attn.close()
    # a promise longer than the shortest sibling is cut to it and reported
    pl = cw.prefix_lens.clone(); pl[0] += 64 * 40
    out, lse, attn = run_cascade(P, cw, prefix_lens=pl)
    assert attn.status() & P.CONCUR_FLAG_BAD_SEQ_LEN
    plain.close(); attn.close()


def test_long_shared_prefix_split_over_many_ctas(P):
    # two groups only: every prefix unit is cut into several ranges, so the prefix partials of a
    # sibling come from several CTAs
    groups = [(16384, [300, 5, 1000, 64, 2, 70, 4000]), (8192, [1, 1])]
    cw = synth.make_cascade_workload("casc_long", groups, 64, 4200, "cuda:0")
    out, lse, attn = run_cascade(P, cw)
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(synth.gather_sequences(cw.w, range(cw.w.spec.batch)))
    assert_parity(out, lse, ref_out, ref_lse, "long shared prefix")
    for ranges in (1, 7, 200):
        out, lse, a2 = run_cascade(P, cw, ranges=ranges)
        assert_parity(out, lse, ref_out, ref_lse, f"long shared prefix, {ranges} suffix ranges")
        a2.close()
    out, lse, a3 = run_cascade(P, cw, prefix_kernel=1)
    assert_parity(out, lse, ref_out, ref_lse, "long shared prefix, mma.sync prefix pass")
    a3.close()
    attn.close()


@pytest.mark.parametrize("prefix_kernel", [0, 1])
def test_malformed_group_tables_share_nothing_and_are_flagged(P, prefix_kernel):
    # group_start is device data: whatever it holds, the step must not fault.  A table that is not a
    # non-decreasing walk through [0, batch] switches sharing off for the call -- the result is the
    # plain step's -- and sets CONCUR_FLAG_BAD_GROUP.
    cw = synth.make_cascade_workload("casc_badgroups", GROUPS, 64, 4400, "cuda:0")
    w = cw.w
    B_ = w.spec.batch
    ref_out, ref_lse = oracle_sequences(synth.gather_sequences(w, range(B_)))
    good = cw.group_start.cpu().tolist()
    G = len(good) - 1
    bad_tables = [
        [0, 10, 1, 11, 2, 12, 3, 13, 4][:G + 1],               # overlapping, non-monotonic
        [good[0]] + [B_ + 5] * G,                              # beyond the batch
        [-3] + good[1:],                                       # negative start
        list(reversed(good)),                                  # decreasing
        [0] + [2 ** 30] * (G - 1) + [B_],                      # huge entries in the middle
    ]
    for table in bad_tables:
        assert len(table) == G + 1
        gs = torch.tensor(table, dtype=torch.int32, device="cuda:0")
        attn = P.DecodeAttention(64, B_, w.block_table.shape[1], 0)
        attn.set_option(P.CONCUR_OPT_PREFIX_KERNEL, prefix_kernel)
        out = torch.full_like(w.q, 7.0)
        lse = torch.full((B_, 64), 7.0, dtype=torch.float32, device="cuda:0")
        P.concur_decode_attn_cascade(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, gs,
                                     cw.prefix_lens, w.scale, out, lse, B_, G, w.num_pages,
                                     w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert attn.status() & P.CONCUR_FLAG_BAD_GROUP, table
        assert_parity(out, lse, ref_out, ref_lse, f"group table {table}")
        attn.close()
    # a table that stops short of the batch is a valid walk: the sequences behind it belong to no group
    short = torch.tensor(good[:-1] + [good[-1] - 1], dtype=torch.int32, device="cuda:0")
    attn = P.DecodeAttention(64, B_, w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_PREFIX_KERNEL, prefix_kernel)
    out = torch.full_like(w.q, 7.0)
    lse = torch.full((B_, 64), 7.0, dtype=torch.float32, device="cuda:0")
    P.concur_decode_attn_cascade(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, short,
                                 cw.prefix_lens, w.scale, out, lse, B_, G, w.num_pages, w.block_table.shape[1],
                                 torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert_parity(out, lse, ref_out, ref_lse, "group table one short of the batch")
    attn.close()


def test_cascade_argument_errors(P):
    B = P.binding
    cw = synth.make_cascade_workload("casc_args", [(64, [1, 2])], 16, 4300, "cuda:0")
    w = cw.w
    attn = P.DecodeAttention(16, 2, w.block_table.shape[1], 0)
    out = torch.empty_like(w.q); lse = torch.empty((2, 64), dtype=torch.float32, device="cuda:0")
    def call(gs=cw.group_start, pl=cw.prefix_lens, ng=1):
        return B.concur_decode_attn_cascade(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, gs, pl,
                                            w.scale, out, lse, 2, ng, w.num_pages, w.block_table.shape[1], 0, check=False)
    assert call() == B.CONCUR_OK
    assert call(gs=None) == B.CONCUR_ERR_INVALID_ARG
    assert call(pl=None) == B.CONCUR_ERR_INVALID_ARG
    assert call(ng=0) == B.CONCUR_ERR_INVALID_ARG
    assert call(ng=3) == B.CONCUR_ERR_INVALID_ARG
    torch.cuda.synchronize()
    attn.close()
    big = P.DecodeAttention(16, 5000, 8, 0)
    rc = B.concur_decode_attn_cascade(big.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, cw.group_start,
                                      cw.prefix_lens, w.scale, out, lse, 2, 1, w.num_pages, w.block_table.shape[1], 0,
                                      check=False)
    assert rc == B.CONCUR_ERR_UNSUPPORTED
    big.close()


@pytest.mark.parametrize("name,nseq", [("casc_24x10_pre2048_p64", 12), ("casc_16x10_pre16384_p64", 6)])
def test_bench_workloads_on_sampled_sequences(P, name, nseq):
    # the workloads bench.py times, in its launch configuration; the oracle on a seeded sample of sequences
    cw = synth.make_named_cascade(name, "cuda:0")
    out, lse, attn = run_cascade(P, cw)
    assert attn.status() == 0
    rng = np.random.default_rng(11)
    seqs = sorted(rng.choice(cw.w.spec.batch, size=nseq, replace=False).tolist())
    ref_out, ref_lse = oracle_sequences(synth.gather_sequences(cw.w, seqs))
    idx = torch.as_tensor(seqs, device="cuda:0")
    assert_parity(out[idx], lse[idx], ref_out, ref_lse, f"{name}, sampled sequences")
    attn.close()
