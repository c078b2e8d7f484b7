"""The curation kernels against the CPU oracle on the same seeded records: integer and boolean
results bit-exact, float32 speedups bit-exact (both sides divide in float32), float64 sums and the
correlation within 1e-9 relative (the order of the last additions differs)."""
import numpy as np
import pytest
import torch

from oracle import curation as C
from synth import records as R

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def run(P, rec, top_k=4892, p=1.0, b=5.0, easy=4000, hard=8500):
    B = P.binding
    N, M = rec.correct.shape
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    correct, tt, tk, L, sk, task_key = t(rec.correct), t(rec.t_torch), t(rec.t_kernel), t(rec.length), t(rec.sample_key), t(rec.task_key)
    out = dict(speedup=torch.full((N, M), -1.0, device=dev), rule_a=torch.full((N,), -7, dtype=torch.int32, device=dev),
               rule_b=torch.full((N, M), 9, dtype=torch.uint8, device=dev),
               pick=torch.full((4, N), -7, dtype=torch.int32, device=dev),
               keep=torch.full((4, N), 9, dtype=torch.uint8, device=dev),
               difficulty=torch.full((N,), 9, dtype=torch.uint8, device=dev),
               stats=torch.full((B.CONCUR_CURATE_NUM_STATS,), 123.0, dtype=torch.float64, device=dev))
    prm = B.concur_curate_params_t(N, M, b, p, top_k, easy, hard, 0)
    B.concur_curate(prm, correct, tt, tk, L, sk, task_key, out["speedup"], out["rule_a"], out["rule_b"], out["pick"],
                    out["keep"], out["difficulty"], out["stats"], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def check(P, rec, top_k=4892, p=1.0):
    B = P.binding
    g = run(P, rec, top_k=top_k, p=p)
    N, M = rec.correct.shape
    sp = C.speedup(rec.correct, rec.t_torch, rec.t_kernel)
    assert np.array_equal(g["speedup"].view(np.uint32), sp.view(np.uint32)), "Eq. (1) must be bit-exact"
    assert np.array_equal(g["rule_a"], C.rule_a(rec.correct, sp, rec.length))
    assert np.array_equal(g["rule_b"].astype(bool), C.rule_b(sp))
    assert np.array_equal(g["difficulty"], C.difficulty(rec.length))
    sels = [C.select_random(rec.correct, rec.sample_key, rec.task_key, top_k), C.select_max_length(rec.correct, rec.length, top_k),
            C.select_min_length(rec.correct, rec.length, top_k), C.select_speedup(rec.correct, sp, top_k)]
    for s, (pick, keep) in enumerate(sels):
        assert np.array_equal(g["pick"][s], pick), f"pick of selection {s}"
        assert np.array_equal(g["keep"][s].astype(bool), keep), f"top-k of selection {s}"
    st = g["stats"]
    m = rec.correct.astype(bool)
    assert st[B.CONCUR_STAT_CORRECT] == m.sum() and st[B.CONCUR_STAT_TASKS_CORRECT] == m.any(axis=1).sum()
    assert st[B.CONCUR_STAT_RULE_A] == (g["rule_a"] >= 0).sum() and st[B.CONCUR_STAT_RULE_B] == C.rule_b(sp).sum()
    assert st[B.CONCUR_STAT_LENGTH_SUM] == rec.length.astype(np.int64).sum()
    assert st[B.CONCUR_STAT_ARL] == pytest.approx(C.arl(rec.length), rel=1e-12)
    assert st[B.CONCUR_STAT_FAST_FIRST] == pytest.approx(C.fast_p(sp[:, 0], p), abs=1e-15)
    assert st[B.CONCUR_STAT_FAST_BEST] == pytest.approx(C.fast_p(sp.max(axis=1), p), abs=1e-15)
    assert st[B.CONCUR_STAT_EXEC_FIRST_COUNT] == m[:, 0].sum()
    r, n = C.pearson(rec.length, sp, rec.correct)
    assert st[B.CONCUR_STAT_N] == n
    if np.isnan(r):
        assert np.isnan(st[B.CONCUR_STAT_PEARSON_R])
    else:
        assert st[B.CONCUR_STAT_PEARSON_R] == pytest.approx(r, rel=1e-9, abs=1e-12)
    assert (st[18:] == 0).all()
    return g


def test_the_synthesis_run_shape(P):
    g = check(P, R.make_records())                        # 18,162 tasks x 5 generations, top 4,892
    assert g["keep"].sum(axis=1).tolist() == [4892] * 4


def test_evaluation_shape_and_other_sizes(P):
    check(P, R.make_records(200, 10, 5), top_k=50)        # KernelBench-sized: 200 tasks x 10 generations
    check(P, R.make_records(1, 1, 6), top_k=1)
    check(P, R.make_records(257, 3, 7), top_k=10 ** 6, p=0.0)
    check(P, R.make_records(1000, 32, 8), top_k=0)


def test_ties_and_degenerate_tables(P):
    rec = R.make_records(600, 5, 9)
    rec.length[:] = 5000                                   # every length ties: first generation is "shortest"
    rec.task_key[:] = 0.5; rec.sample_key[:] = 0.25        # every random key ties
    check(P, rec, top_k=100)
    rec = R.make_records(300, 4, 10)
    rec.correct[:] = 0                                     # nothing correct anywhere
    g = check(P, rec, top_k=100)
    assert (g["pick"] == -1).all() and g["keep"].sum() == 0 and (g["speedup"] == 0).all()
    rec = R.make_records(300, 4, 11)
    rec.correct[:] = 1; rec.t_kernel[:] = rec.t_torch      # every speedup exactly 1: fast_1 is 0, rule (a) keeps all
    g = check(P, rec, top_k=100)
    assert (g["rule_a"] >= 0).all()


def test_argument_errors(P):
    B = P.binding
    rec = R.make_records(8, 2, 12)
    dev = "cuda:0"
    z = torch.zeros(64, dtype=torch.float64, device=dev)
    def call(prm, first=z):
        return B.concur_curate(prm, first, z, z, z, z, z, z, z, z, z, z, z, z, 0, check=False)
    assert call(B.concur_curate_params_t(8, 2, 5.0, 1.0, 4, 4000, 8500, 0)) == B.CONCUR_OK
    assert call(B.concur_curate_params_t(0, 2, 5.0, 1.0, 4, 4000, 8500, 0)) == B.CONCUR_ERR_INVALID_ARG
    assert call(B.concur_curate_params_t(8, 33, 5.0, 1.0, 4, 4000, 8500, 0)) == B.CONCUR_ERR_INVALID_ARG
    assert call(B.concur_curate_params_t(8, 2, 5.0, 1.0, 4, 4000, 8500, 1)) == B.CONCUR_ERR_INVALID_ARG
    assert call(B.concur_curate_params_t(8, 2, 5.0, 1.0, 4, 4000, 8500, 0), first=None) == B.CONCUR_ERR_INVALID_ARG
    torch.cuda.synchronize()
