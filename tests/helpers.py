"""Test-side helpers: the oracle run over many sequences with a thread pool (the oracle
itself stays single-threaded; ctypes releases the GIL), and the parity criteria."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

import oracle

# tolerance of the bf16 output and fp32 lse against the fp64 oracle
OUT_ATOL, OUT_RTOL = 4e-3, 1.6e-2
LSE_ATOL = 1e-3
REL_RMS_MAX = 5e-3          # stricter internal gate on the whole output


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_sequences(w, seqs=None, threads=None):
    """Oracle for the given sequences of a host-resident workload.  Returns
    (out [len(seqs)][Hq][D] f64, lse [len(seqs)][Hq] f64)."""
    seqs = list(range(w.spec.batch)) if seqs is None else list(seqs)
    qb = oracle._u16(w.q); kb = oracle._u16(w.k_pages); vb = oracle._u16(w.v_pages)
    tb = oracle._i32(w.block_table); lb = oracle._i32(w.seq_lens)
    threads = threads or host_cores()
    if not seqs:
        return np.zeros((0, w.spec.num_q_heads, w.spec.head_dim)), np.zeros((0, w.spec.num_q_heads))
    # a few chunks of sequences per thread; each call gets only its chunk's rows of q, of the
    # table and of the lengths, so that its result arrays are chunk-sized (a call over the whole
    # batch allocates batch-sized results, which for thousands of short sequences is gigabytes)
    idx = np.asarray(seqs, dtype=np.int64)
    nchunks = min(len(seqs), threads * 4)
    chunks = [c for c in np.array_split(idx, nchunks) if len(c)]

    def one(c):
        return oracle.decode_attn(np.ascontiguousarray(qb[c]), kb, vb, np.ascontiguousarray(tb[c]),
                                  np.ascontiguousarray(lb[c]), w.scale)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        res = list(ex.map(one, chunks))
    return np.concatenate([r[0] for r in res]), np.concatenate([r[1] for r in res])


def assert_parity(out_gpu, lse_gpu, ref_out, ref_lse, what="", out_atol=None, rel_rms_max=None):
    """out_gpu bf16 / lse_gpu fp32 torch tensors (any device) against fp64 numpy references.
    out_atol / rel_rms_max replace the defaults where a test derives its own (peaked rows)."""
    og = out_gpu.detach().cpu().to(torch.float64).numpy()
    lg = lse_gpu.detach().cpu().to(torch.float64).numpy()
    assert og.shape == ref_out.shape and lg.shape == ref_lse.shape, what
    assert np.isfinite(og).all(), f"{what}: non-finite output"
    err = np.abs(og - ref_out)
    bound = (OUT_ATOL if out_atol is None else out_atol) + OUT_RTOL * np.abs(ref_out)
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), f"{what}: out[{worst}] = {og[worst]} vs {ref_out[worst]}"
    empty = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(lg), empty), f"{what}: lse -inf pattern"
    lerr = np.abs(lg[~empty] - ref_lse[~empty])
    assert lerr.size == 0 or lerr.max() <= LSE_ATOL, f"{what}: lse error {lerr.max()}"
    den = np.sqrt(np.mean(ref_out ** 2))
    rel_rms = float(np.sqrt(np.mean(err ** 2)) / den) if den > 0 else 0.0
    assert rel_rms <= (REL_RMS_MAX if rel_rms_max is None else rel_rms_max), f"{what}: relative RMS error {rel_rms}"
    return {"max_abs": float(err.max()) if err.size else 0.0, "rel_rms": rel_rms,
            "lse_max_abs": float(lerr.max()) if lerr.size else 0.0}
