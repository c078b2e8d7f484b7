"""Prefill (causal attention of several query tokens per sequence) on the tcgen05 kernel against
the CPU oracle.  Per query token the definition is the decode definition for a sequence that ends
at that token, so the oracle is the same pinned routine, called on a batch in which every query
token is a sequence of its own (synth.prefill_as_decode only re-indexes)."""
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


# both kernels behind the entry point: 0 = two query tiles per CTA over 128-token steps (the default),
# 1 = one tile over 64-token tiles
KERNEL = {"value": 0}


@pytest.fixture(autouse=True, params=[0, 1], ids=["pair", "single"])
def prefill_kernel(request):
    KERNEL["value"] = request.param
    yield request.param
    KERNEL["value"] = 0


def run_prefill(P, pw, hq=64):
    w = pw.w
    attn = P.DecodeAttention(w.spec.page_size, w.spec.batch, w.block_table.shape[1], 0, num_q_heads=hq)
    attn.set_option(P.CONCUR_OPT_PREFILL_KERNEL, KERNEL["value"])
    tq = pw.total_q
    out = torch.full((tq + 8, hq, 128), 7.0, dtype=torch.bfloat16, device="cuda:0")
    lse = torch.full((tq + 8, hq), 7.0, dtype=torch.float32, device="cuda:0")
    P.concur_prefill_attn(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, pw.q_start, w.scale,
                          out, lse, w.spec.batch, tq, w.num_pages, w.block_table.shape[1],
                          torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert (out[tq:] == 7.0).all() and (lse[tq:] == 7.0).all(), "wrote past the last query token"
    return out[:tq], lse[:tq], attn


def check(P, pw, tokens=None, hq=64, what=""):
    out, lse, attn = run_prefill(P, pw, hq)
    assert attn.status() == 0
    tokens = list(range(pw.total_q)) if tokens is None else list(tokens)
    ref_out, ref_lse = oracle_sequences(synth.prefill_as_decode(pw, tokens))
    idx = torch.as_tensor(tokens, dtype=torch.long, device="cuda:0")
    assert_parity(out[idx], lse[idx], ref_out, ref_lse, what)
    attn.close()


# whole prompts (q_len = len) and chunks (q_len < len), lengths around tile and block boundaries
LENS = (1, 2, 15, 16, 17, 63, 64, 65, 100, 129, 200, 333)


@pytest.mark.parametrize("page_size", [64, 16, 32, 128])
def test_whole_prompts_every_token(P, page_size):
    pw = synth.make_prefill_workload(f"pf_p{page_size}", LENS, LENS, page_size, 9000 + page_size, "cuda:0")
    check(P, pw, what=f"whole prompts p{page_size}")


@pytest.mark.parametrize("page_size", [16, 64, 128])
def test_chunks_at_the_end_of_longer_contexts(P, page_size):
    lens = (500, 64, 1000, 129, 2049, 77, 640)
    q_lens = (1, 64, 17, 100, 48, 0, 333)           # one sequence has no query token at all
    pw = synth.make_prefill_workload(f"pfc_p{page_size}", lens, q_lens, page_size, 9100 + page_size, "cuda:0")
    check(P, pw, what=f"chunks p{page_size}")


@pytest.mark.parametrize("hq", [8, 40])
def test_smaller_groups(P, hq):
    pw = synth.make_prefill_workload(f"pf_h{hq}", (100, 65, 300), (100, 20, 300), 64, 9200 + hq, "cuda:0",
                                     num_q_heads=hq)
    check(P, pw, hq=hq, what=f"prefill, {hq} heads")


def test_long_prompt_on_sampled_tokens(P):
    # 4,096- and 2,500-token prompts: every 16-token block of every KV head is a unit with up to
    # 64 tiles; parity on a seeded sample of query tokens (first, last, block and tile edges included)
    pw = synth.make_prefill_workload("pf_long", (4096, 2500), (4096, 2500), 64, 9300, "cuda:0")
    rng = np.random.default_rng(3)
    tokens = sorted(set([0, 1, 15, 16, 63, 64, 65, 4095, 4096, 4097, 4096 + 2499] +
                        rng.integers(0, pw.total_q, 40).tolist()))
    check(P, pw, tokens=tokens, what="long prompts")


def test_decode_is_the_one_token_case(P):
    # q_len = 1 everywhere: prefill must agree with the decode step on the same cache
    lens = (300, 1, 64, 1025)
    pw = synth.make_prefill_workload("pf_dec", lens, (1, 1, 1, 1), 64, 9400, "cuda:0")
    out, lse, attn = run_prefill(P, pw)
    w = pw.w
    out_d, lse_d = attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    torch.cuda.synchronize()
    assert (out.float() - out_d.float()).abs().max().item() <= 2e-2
    assert (lse - lse_d).abs().max().item() <= 1e-3
    attn.close()


def test_too_many_query_tokens_are_cut_and_flagged(P):
    pw = synth.make_prefill_workload("pf_bad", (100, 50), (100, 50), 64, 9500, "cuda:0")
    w = pw.w
    short = w.seq_lens.clone(); short[1] = 20            # 50 query tokens, only 20 cached
    attn = P.DecodeAttention(64, 2, w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_PREFILL_KERNEL, KERNEL["value"])
    out = torch.zeros_like(w.q); lse = torch.zeros((pw.total_q, 64), dtype=torch.float32, device="cuda:0")
    P.concur_prefill_attn(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, short, pw.q_start, w.scale, out, lse,
                          2, pw.total_q, w.num_pages, w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() & P.CONCUR_FLAG_BAD_SEQ_LEN
    assert torch.isfinite(out.float()).all()
    attn.close()


def test_argument_errors(P):
    B = P.binding
    pw = synth.make_prefill_workload("pf_args", (64,), (64,), 64, 9600, "cuda:0")
    w = pw.w
    attn = P.DecodeAttention(64, 1, w.block_table.shape[1], 0)
    out = torch.empty_like(w.q); lse = torch.empty((64, 64), dtype=torch.float32, device="cuda:0")
    def call(qs=pw.q_start, tq=64):
        return B.concur_prefill_attn(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, qs, w.scale,
                                     out, lse, 1, tq, w.num_pages, w.block_table.shape[1], 0, check=False)
    assert call() == B.CONCUR_OK
    assert call(qs=None) == B.CONCUR_ERR_INVALID_ARG
    assert call(tq=-1) == B.CONCUR_ERR_INVALID_ARG
    torch.cuda.synchronize()
    attn.close()


@pytest.mark.parametrize("name", ["prefill_16x2048_p64", "prefill_chunk_8x2048_of_16384_p64"])
def test_bench_workloads_on_sampled_tokens(P, name):
    # the workloads bench.py times; the oracle on a seeded sample of query tokens
    pw = synth.make_named_prefill(name, "cuda:0")
    rng = np.random.default_rng(13)
    tokens = sorted(set([0, pw.total_q - 1] + rng.integers(0, pw.total_q, 24).tolist()))
    check(P, pw, tokens=tokens, what=name)
