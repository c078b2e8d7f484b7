"""The softmax scale is any finite number: negative (the kernels then look for the smallest raw score),
zero (every visible token weighs the same) and large (peaked rows, whose running maximum jumps by more than
the slack the tensor-core kernels allow their reference, so that the accumulators are rescaled in place).
Every entry point and kernel choice against the CPU oracle, element by element."""
import pytest
import torch

import synth
from helpers import assert_parity, oracle_sequences

pytestmark = pytest.mark.gpu

SCALES = [-0.07, 0.0, 0.6, -0.5]


def tol(scale):
    """With |scale| of 0.5 and more a row's weight sits on one or two tokens, so the rounding of the
    probabilities to bf16 (2^-9 relative, the kernels' precision for the P.V product) no longer averages out
    over many terms: the error of an output is up to 2^-9 x the |V| values it is made of (here up to ~4),
    instead of a fraction of that.  The relative part and the lse bound stay what they are everywhere."""
    return dict(out_atol=1.2e-2, rel_rms_max=1e-2) if abs(scale) >= 0.5 else {}


LENS = (0, 1, 63, 64, 65, 200, 517, 1000, 2049, 4099)


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def host(w):
    return synth.gather_sequences(w, range(w.spec.batch))


@pytest.mark.parametrize("scale", SCALES)
@pytest.mark.parametrize("kernel,page_size,ranges", [(0, 64, 0), (0, 16, 7), (0, 32, 300), (1, 64, 0)])
def test_decode_step(P, scale, kernel, page_size, ranges):
    w = synth.make_workload(synth.tiny_spec(f"sc{page_size}", LENS, page_size, 5100 + page_size), "cuda:0")
    w.scale = scale
    attn = P.DecodeAttention(page_size, len(LENS), w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    out, lse = attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"decode, scale {scale}, kernel {kernel}, p{page_size}, R{ranges}", **tol(scale))
    attn.close()


GROUPS = [(1024, [100, 1, 64, 700, 333]), (0, [500]), (2048, [5, 900]), (512, [0, 130, 64, 1, 2000, 77, 640, 63, 65, 300])]


@pytest.mark.parametrize("scale", SCALES)
@pytest.mark.parametrize("prefix_kernel", [0, 1])
def test_cascade_step(P, scale, prefix_kernel):
    cw = synth.make_cascade_workload("sc_casc", GROUPS, 64, 5200, "cuda:0")
    w = cw.w
    w.scale = scale
    attn = P.DecodeAttention(64, w.spec.batch, w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_PREFIX_KERNEL, prefix_kernel)
    out = torch.full_like(w.q, 7.0)
    lse = torch.full((w.spec.batch, 64), 7.0, dtype=torch.float32, device="cuda:0")
    P.concur_decode_attn_cascade(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, cw.group_start,
                                 cw.prefix_lens, w.scale, out, lse, w.spec.batch, len(cw.prefix_lens_host), w.num_pages,
                                 w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"cascade, scale {scale}, prefix kernel {prefix_kernel}", **tol(scale))
    attn.close()


@pytest.mark.parametrize("scale", SCALES)
@pytest.mark.parametrize("prefill_kernel", [0, 1])
@pytest.mark.parametrize("page_size", [64, 16])
def test_prefill(P, scale, prefill_kernel, page_size):
    lens, q_lens = (70, 33, 300, 1, 129, 517), (70, 20, 300, 1, 16, 200)
    pw = synth.make_prefill_workload("sc_pf", lens, q_lens, page_size, 5300 + page_size, "cuda:0")
    w = pw.w
    w.scale = scale
    attn = P.DecodeAttention(page_size, len(lens), w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_PREFILL_KERNEL, prefill_kernel)
    out = torch.full_like(w.q, 7.0)
    lse = torch.full((pw.total_q, 64), 7.0, dtype=torch.float32, device="cuda:0")
    P.concur_prefill_attn(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, pw.q_start, w.scale, out, lse,
                          len(lens), pw.total_q, w.num_pages, w.block_table.shape[1],
                          torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(synth.prefill_as_decode(pw, range(pw.total_q)))
    assert_parity(out, lse, ref_out, ref_lse, f"prefill, scale {scale}, kernel {prefill_kernel}, p{page_size}", **tol(scale))
    attn.close()
