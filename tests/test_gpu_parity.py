"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element on
the same seeded inputs; plus the device-side error handling that must never fault."""
import numpy as np
import pytest
import torch

import synth
from helpers import assert_parity, oracle_sequences

pytestmark = pytest.mark.gpu

KERNELS = {"mma": 0, "scalar": 1}


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def run(P, w, kernel=0, ranges=0, grid=0, pad=0):
    """One call on the device copy of workload `w`; returns (out, lse, attn)."""
    attn = P.DecodeAttention(w.spec.page_size, max(1, w.spec.batch), w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    attn.set_option(P.CONCUR_OPT_GRID_CTAS, grid)
    out, lse = attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    torch.cuda.synchronize()
    return out, lse, attn


def to_host(w):
    return synth.gather_sequences(w, range(w.spec.batch))


EDGE_LENS = (0, 1, 2, 15, 16, 17, 31, 33, 63, 64, 65, 127, 128, 129, 191, 200, 257, 1000, 1023, 1025, 4099)


@pytest.mark.parametrize("kernel", list(KERNELS))
@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
@pytest.mark.parametrize("ranges", [0, 1, 2, 3, 7, 61, 4736])
def test_edge_lengths_and_forced_splits(P, kernel, page_size, ranges):
    spec = synth.tiny_spec(f"edge_p{page_size}", EDGE_LENS, page_size, 1000 + page_size)
    w = synth.make_workload(spec, "cuda:0")
    out, lse, attn = run(P, w, KERNELS[kernel], ranges)
    assert attn.status() == 0
    R, W, starts = attn.last_plan()
    tiles = sum(-(-n // 64) for n in EDGE_LENS) * 8
    assert W == tiles
    if ranges:
        assert R == min(ranges, W)
    assert starts[0] == 0 and starts[-1] == W and all(a < b for a, b in zip(starts, starts[1:]))
    ref_out, ref_lse = oracle_sequences(to_host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"{kernel} p{page_size} R{ranges}")
    attn.close()


@pytest.mark.parametrize("kernel", list(KERNELS))
def test_single_sequence_split_many_ways(P, kernel):
    # one long sequence cut into many partials per KV head: pins the LSE combine
    spec = synth.tiny_spec("long1", (5000,), 16, 77)
    w = synth.make_workload(spec, "cuda:0")
    ref_out, ref_lse = oracle_sequences(to_host(w))
    for ranges in (1, 8, 9, 13, 100, 632):
        out, lse, attn = run(P, w, KERNELS[kernel], ranges)
        assert attn.status() == 0
        assert_parity(out, lse, ref_out, ref_lse, f"{kernel} R{ranges}")
        attn.close()


@pytest.mark.parametrize("kernel", list(KERNELS))
@pytest.mark.parametrize("name", ["cfg1_b1_ctx512_p16", "cfg2_b16_u1k_8k_p16", "cfg5_b32_skew128k_p64"])
def test_full_configs_elementwise(P, kernel, name):
    w = synth.make_workload(name, "cuda:0")
    out, lse, attn = run(P, w, KERNELS[kernel])
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(to_host(w))
    stats = assert_parity(out, lse, ref_out, ref_lse, f"{kernel} {name}")
    print(name, kernel, stats)
    attn.close()


@pytest.mark.parametrize("name", ["cfg3_b64_ctx16384_p64", "cfg4_b256_logu2k_32k_p64"])
def test_large_configs_every_sequence(P, name):
    # full-size launch (the configuration the benchmark times); the oracle checks every element of
    # every sequence (a second or two of the host's cores for 1 M tokens, a few for 2.8 M)
    w = synth.make_workload(name, "cuda:0")
    out, lse, attn = run(P, w, 0)
    assert attn.status() == 0
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    # in chunks of sequences, so that the host copy of their pages stays at a few GB
    worst = {"max_abs": 0.0, "rel_rms": 0.0, "lse_max_abs": 0.0}
    for b0 in range(0, w.spec.batch, 64):
        seqs = list(range(b0, min(b0 + 64, w.spec.batch)))
        ref_out, ref_lse = oracle_sequences(synth.gather_sequences(w, seqs))
        stats = assert_parity(out[seqs], lse[seqs], ref_out, ref_lse, f"{name} sequences {b0}..")
        worst = {k: max(worst[k], stats[k]) for k in worst}
    print(name, worst)
    attn.close()


@pytest.mark.parametrize("claim_ahead", [0, 1, 3, 1 << 20])
@pytest.mark.parametrize("page_size", [16, 64])
def test_claim_ahead_values(P, claim_ahead, page_size):
    # few CTAs and many ranges, so that every CTA claims range after range; whenever the claim is
    # made (0 = only once the range has been streamed to its end) each range is taken exactly once
    spec = synth.tiny_spec(f"claim_p{page_size}", EDGE_LENS, page_size, 1200 + page_size)
    w = synth.make_workload(spec, "cuda:0")
    ref_out, ref_lse = oracle_sequences(to_host(w))
    for grid, ranges in ((4, 61), (3, 0), (148, 0)):
        attn = P.DecodeAttention(page_size, spec.batch, w.block_table.shape[1], 0)
        attn.set_option(P.CONCUR_OPT_CLAIM_AHEAD, claim_ahead)
        attn.set_option(P.CONCUR_OPT_GRID_CTAS, grid)
        attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
        if ranges == 0:
            attn.set_option(P.CONCUR_OPT_RANGES_PER_CTA, 5)
        out, lse = attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
        torch.cuda.synchronize()
        assert attn.status() == 0
        assert_parity(out, lse, ref_out, ref_lse, f"claim_ahead {claim_ahead} grid {grid} ranges {ranges}")
        attn.close()


def test_scalar_and_mma_kernels_agree_on_a_large_config(P):
    w = synth.make_workload("cfg2_b16_u1k_8k_p16", "cuda:0")
    o0, l0, a0 = run(P, w, 0)
    o1, l1, a1 = run(P, w, 1)
    assert (o0.float() - o1.float()).abs().max().item() <= 8e-3
    assert (l0 - l1).abs().max().item() <= 1e-3
    a0.close(); a1.close()


def test_outputs_do_not_depend_on_unused_memory(P):
    # same workload, different garbage in the slots past each length and in the table tails
    spec = synth.tiny_spec("garbage", (5, 70, 130, 1), 64, 31)
    w = synth.make_workload(spec, "cuda:0", table_stride=9)
    o0, l0, a0 = run(P, w)
    k2, v2 = w.k_pages.clone(), w.v_pages.clone()
    for b, n in enumerate(w.lens_host):
        page = int(w.table_host[b, (n - 1) // 64])
        k2[page, :, n % 64:, :] = 3.0e38
        v2[page, :, n % 64:, :] = float("inf")
    bt2 = w.block_table.clone()
    bt2[bt2 < 0] = 2 ** 30
    attn = P.DecodeAttention(64, 4, 9, 0)
    o1, l1 = attn(w.q, k2, v2, bt2, w.seq_lens, w.scale)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert torch.equal(o0.view(torch.int16), o1.view(torch.int16)) and torch.equal(l0, l1)
    a0.close(); attn.close()


def test_writes_stay_inside_out_and_lse(P):
    spec = synth.tiny_spec("canary", (300, 0, 64, 4000), 16, 32)
    w = synth.make_workload(spec, "cuda:0")
    B = spec.batch
    for kernel in (0, 1):
        big_out = torch.full((B + 2, 64, 128), 7.0, dtype=torch.bfloat16, device="cuda:0")
        big_lse = torch.full((B + 2, 64), 7.0, dtype=torch.float32, device="cuda:0")
        attn = P.DecodeAttention(16, B, w.block_table.shape[1], 0)
        attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
        attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out=big_out[1:B + 1], lse=big_lse[1:B + 1])
        torch.cuda.synchronize()
        assert (big_out[0] == 7).all() and (big_out[B + 1] == 7).all()
        assert (big_lse[0] == 7).all() and (big_lse[B + 1] == 7).all()
        assert not (big_out[2] != 0).any() and torch.isneginf(big_lse[2]).all()      # the empty sequence
        attn.close()


def test_bad_page_ids_and_lengths_are_flagged_not_dereferenced(P):
    spec = synth.tiny_spec("bad", (100, 200, 50), 16, 33)
    w = synth.make_workload(spec, "cuda:0")
    for kernel in (0, 1):
        attn = P.DecodeAttention(16, 3, w.block_table.shape[1], 0)
        attn.set_option(P.CONCUR_OPT_KERNEL, kernel)
        bt = w.block_table.clone()
        bt[1, 3] = w.num_pages + 12345
        bt[0, 0] = -7
        out, lse = attn(w.q, w.k_pages, w.v_pages, bt, w.seq_lens, w.scale)
        torch.cuda.synchronize()
        assert attn.status() == P.CONCUR_FLAG_BAD_PAGE_ID
        assert attn.status() == 0                                  # cleared by the read
        ref_out, ref_lse = oracle_sequences(to_host(w), [2])
        assert_parity(out[2:3], lse[2:3], ref_out, ref_lse, "untouched sequence")
        lens = w.seq_lens.clone()
        lens[0] = -5
        lens[1] = 10 ** 6
        out, lse = attn(w.q, w.k_pages, w.v_pages, w.block_table, lens, w.scale)
        torch.cuda.synchronize()
        flags = attn.status()
        assert flags & P.CONCUR_FLAG_BAD_SEQ_LEN
        assert not (out[0] != 0).any() and torch.isneginf(lse[0]).all()   # clamped to empty
        attn.close()


def test_argument_errors(P):
    B = P.binding
    spec = synth.tiny_spec("args", (100, 20), 16, 34)
    w = synth.make_workload(spec, "cuda:0")
    attn = P.DecodeAttention(16, 2, 8, 0)
    out = torch.empty_like(w.q)
    lse = torch.empty((2, 64), dtype=torch.float32, device="cuda:0")
    args = [w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out, lse, 2, w.num_pages,
            w.block_table.shape[1]]

    def call(**kw):
        a = list(args)
        names = ["q", "k_pages", "v_pages", "block_table", "seq_lens", "scale", "out", "lse", "batch",
                 "num_pages", "block_table_stride"]
        for k, v in kw.items():
            a[names.index(k)] = v
        return B.concur_decode_attn(attn.handle, *a, check=False)

    assert call() == B.CONCUR_OK
    assert call(q=None) == B.CONCUR_ERR_INVALID_ARG
    assert call(lse=None) == B.CONCUR_ERR_INVALID_ARG
    assert call(q=w.q.data_ptr() + 2) == B.CONCUR_ERR_INVALID_ARG
    assert call(batch=3) == B.CONCUR_ERR_TOO_LARGE
    assert call(block_table_stride=9) == B.CONCUR_ERR_TOO_LARGE
    assert call(batch=-1) == B.CONCUR_ERR_INVALID_ARG
    assert call(num_pages=0) == B.CONCUR_ERR_INVALID_ARG
    assert call(batch=0) == B.CONCUR_OK
    assert B.concur_attn_set_option(attn.handle, 99, 1, check=False) == B.CONCUR_ERR_INVALID_ARG
    assert B.concur_attn_set_option(attn.handle, B.CONCUR_OPT_KERNEL, 5, check=False) == B.CONCUR_ERR_INVALID_ARG
    torch.cuda.synchronize()
    attn.close()


def test_caller_workspace_and_too_small_workspace(P):
    B = P.binding
    cfg = P.make_config(16, 4, 128)
    need = P.concur_attn_workspace_bytes(cfg)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda:0")
    base = (ws.data_ptr() + 255) // 256 * 256
    small = P.make_config(16, 4, 128, workspace=base, workspace_bytes=need - 1)
    with pytest.raises(B.ConcurError) as e:
        P.concur_attn_create(small)
    assert e.value.code == B.CONCUR_ERR_TOO_LARGE
    h = P.concur_attn_create(P.make_config(16, 4, 128, workspace=base, workspace_bytes=need))
    spec = synth.tiny_spec("ws", (100, 2000, 7), 16, 35)
    w = synth.make_workload(spec, "cuda:0")
    out = torch.empty_like(w.q)
    lse = torch.empty((3, 64), dtype=torch.float32, device="cuda:0")
    B.concur_decode_attn(h, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out, lse, 3,
                         w.num_pages, w.block_table.shape[1], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    ref_out, ref_lse = oracle_sequences(to_host(w))
    assert_parity(out, lse, ref_out, ref_lse, "caller workspace")
    P.concur_attn_destroy(h)


def test_host_entry_point_matches_device_entry_point(P):
    B = P.binding
    spec = synth.tiny_spec("host", (300, 1, 4000, 64), 64, 36)
    w = synth.make_workload(spec, "cuda:0")
    out_d, lse_d, attn = run(P, w)
    hw = to_host(w)        # pages renumbered in logical order; same values
    pin = lambda t: t.contiguous().pin_memory()
    q, k, v, bt, sl = pin(hw.q), pin(hw.k_pages), pin(hw.v_pages), pin(hw.block_table), pin(hw.seq_lens)
    out_h = torch.empty_like(q).pin_memory()
    lse_h = torch.empty((4, 64), dtype=torch.float32).pin_memory()
    for _ in range(2):
        B.concur_decode_attn_host(attn.handle, q, k, v, bt, sl, hw.scale, out_h, lse_h, 4, k.shape[0],
                                  bt.shape[1], torch.cuda.current_stream().cuda_stream)
    assert torch.equal(out_h.view(torch.int16), out_d.cpu().view(torch.int16))
    assert torch.equal(lse_h, lse_d.cpu())
    attn.close()


@pytest.mark.parametrize("kernel", list(KERNELS))
def test_many_short_sequences(P, kernel):
    # more sequences than the partial kernel caches plan rows for (it then reads them from
    # global memory), a third of them empty or shorter than one page
    rng = np.random.default_rng(2024)
    lens = rng.integers(0, 400, size=700)
    lens[rng.integers(0, 700, size=60)] = 0
    lens[rng.integers(0, 700, size=60)] = rng.integers(1, 16, size=60)
    spec = synth.tiny_spec("many", [int(x) for x in lens], 16, 88)
    w = synth.make_workload(spec, "cuda:0")
    out, lse, attn = run(P, w, KERNELS[kernel])
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(to_host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"{kernel} 700 sequences")
    attn.close()


@pytest.mark.parametrize("batch", [288, 289, 300, 511, 512])
@pytest.mark.parametrize("page_size,ranges", [(64, 0), (16, 37)])
def test_batch_sizes_around_the_in_kernel_plan_limits(P, batch, page_size, ranges):
    # up to 511 sequences the tensor-core kernel derives the tile prefix and the range count from
    # seq_lens itself (288 threads per scan round: one round, two rounds, the last cached batch);
    # from 512 on it reads the plan kernel's tables.  Both must cut the same ranges.
    rng = np.random.default_rng(4000 + batch)
    lens = rng.integers(0, 300, size=batch)
    lens[rng.integers(0, batch, size=20)] = 0
    lens[batch - 1] = 777                                  # the last sequence matters to the scan's tail
    spec = synth.tiny_spec(f"plan{batch}", [int(x) for x in lens], page_size, 4100 + batch)
    w = synth.make_workload(spec, "cuda:0")
    out, lse, attn = run(P, w, 0, ranges)
    assert attn.status() == 0
    R, W, starts = attn.last_plan()
    assert W == 8 * sum(-(-int(n) // 64) for n in lens)
    ref_out, ref_lse = oracle_sequences(to_host(w))
    assert_parity(out, lse, ref_out, ref_lse, f"batch {batch} p{page_size} R{ranges}")
    attn.close()


def test_repeated_calls_on_one_handle_are_identical(P):
    # the workspace is reused call after call: counters and partial slots of an earlier,
    # larger call must not leak into a later one
    big = synth.make_workload(synth.tiny_spec("rep_big", (9000, 300, 4097), 64, 41), "cuda:0")
    small = synth.make_workload(synth.tiny_spec("rep_small", (130, 64), 64, 42), "cuda:0")
    attn = P.DecodeAttention(64, 3, max(big.block_table.shape[1], small.block_table.shape[1]), 0)
    first = None
    for _ in range(3):
        ob, lb = attn(big.q, big.k_pages, big.v_pages, big.block_table, big.seq_lens, big.scale)
        os_, ls = attn(small.q, small.k_pages, small.v_pages, small.block_table, small.seq_lens, small.scale)
        torch.cuda.synchronize()
        if first is None:
            first = (ob.clone(), lb.clone(), os_.clone(), ls.clone())
        else:
            for a, b in zip(first, (ob, lb, os_, ls)):
                assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                                   b.view(torch.int16) if b.dtype == torch.bfloat16 else b)
    ref_out, ref_lse = oracle_sequences(to_host(small))
    assert_parity(first[2], first[3], ref_out, ref_lse, "small after big")
    assert attn.status() == 0
    attn.close()


@pytest.mark.parametrize("page_size,ranges,grid", [(32, 300, 0), (64, 700, 0), (16, 500, 37), (64, 0, 0)])
def test_results_are_the_same_bits_from_launch_to_launch(P, page_size, ranges, grid):
    # More ranges than CTAs: which CTA claims which range changes from launch to launch.  How a segment's
    # tiles are grouped into sums must not change with it, so every launch gives the same bits.
    lens = (4099, 0, 517, 9000, 64, 2049, 1, 12000, 333, 6000)
    w = synth.make_workload(synth.tiny_spec("bits", lens, page_size, 4300 + page_size), "cuda:0")
    attn = P.DecodeAttention(page_size, len(lens), w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, ranges)
    attn.set_option(P.CONCUR_OPT_GRID_CTAS, grid)
    first = None
    for _ in range(12):
        out, lse = attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
        torch.cuda.synchronize()
        if first is None:
            first = (out.clone(), lse.clone())
        else:
            assert torch.equal(first[0].view(torch.int16), out.view(torch.int16))
            assert torch.equal(first[1], lse)
    assert attn.status() == 0
    ref_out, ref_lse = oracle_sequences(to_host(w))
    assert_parity(first[0], first[1], ref_out, ref_lse, f"p{page_size} R{ranges} grid {grid}")
    attn.close()


def test_a_wait_that_runs_out_returns_with_the_flag_and_leaves_the_handle_usable(P):
    # One CTA streams a whole 16,384-token sequence in two ranges that cut no unit, so its combiner
    # warp has nothing to merge and waits for a job from the kernel's start to its end, hundreds of
    # microseconds.  With the roles' wait limit set to 20 microseconds that wait gives up: the
    # kernel must still end by itself, report CONCUR_FLAG_WAIT_LIMIT, and fault nothing; with the
    # default limit back, the same handle then computes the right result.
    spec = synth.tiny_spec("waitlimit", (16384,), 64, 1300)
    w = synth.make_workload(spec, "cuda:0")
    attn = P.DecodeAttention(64, 1, w.block_table.shape[1], 0)
    attn.set_option(P.CONCUR_OPT_GRID_CTAS, 1)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, 2)
    attn.set_option(P.CONCUR_OPT_WAIT_LIMIT_NS, 20_000)
    out, lse = attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    torch.cuda.synchronize()
    assert attn.status() & P.CONCUR_FLAG_WAIT_LIMIT
    assert attn.status() == 0                                   # reading the flags clears them
    attn.set_option(P.CONCUR_OPT_WAIT_LIMIT_NS, 0)              # the default again
    ref_out, ref_lse = oracle_sequences(to_host(w))
    for grid in (1, 0):
        attn.set_option(P.CONCUR_OPT_GRID_CTAS, grid)
        out, lse = attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
        torch.cuda.synchronize()
        assert attn.status() == 0
        assert_parity(out, lse, ref_out, ref_lse, f"after a wait limit, grid {grid}")
    attn.close()
