"""Pins of the curation oracle (CPU only): the hand-worked example, closed forms, a library
special case, brute force and invariants -- each chosen so that a plausible mistake (a dropped
indicator, >= for >, the wrong tie rule, a transposed axis) fails one of them."""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import curation as C
from synth import records as R

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "curation_worked_example.json")))


def gold_arrays():
    return (np.array(GOLD["correct"], np.uint8), np.array(GOLD["t_torch"], np.float32),
            np.array(GOLD["t_kernel"], np.float32), np.array(GOLD["length"], np.int32))


def test_worked_example():
    correct, tt, tk, L = gold_arrays()
    sp = C.speedup(correct, tt, tk)
    assert sp.dtype == np.float32 and np.array_equal(sp, np.array(GOLD["speedup"], np.float32))
    assert np.array_equal(C.rule_a(correct, sp, L), GOLD["rule_a"])
    assert np.array_equal(C.rule_b(sp), np.array(GOLD["rule_b"], bool))
    assert C.arl(L) == GOLD["arl"]
    assert C.fast_p(sp[:, 0], 1.0) == GOLD["fast_1_first_generation"]
    assert C.fast_p(sp.max(axis=1), 1.0) == GOLD["fast_1_best_generation"]
    assert correct[:, 0].mean() == GOLD["exec_first_generation"]
    pick, keep = C.select_max_length(correct, L, 2)
    assert list(pick) == GOLD["pick_max_length"] and list(np.flatnonzero(keep)) == GOLD["keep_max_length_k2_tasks"]
    pick, keep = C.select_min_length(correct, L, 2)
    assert list(pick) == GOLD["pick_min_length"] and list(np.flatnonzero(keep)) == GOLD["keep_min_length_k2_tasks"]
    pick, keep = C.select_speedup(correct, sp, 2)
    assert list(pick) == GOLD["pick_speedup"] and list(np.flatnonzero(keep)) == GOLD["keep_speedup_k2_tasks"]
    lo, hi = GOLD["difficulty_bounds"]
    assert list(C.difficulty(L, lo, hi)) == GOLD["difficulty"]


def test_speedup_is_zero_exactly_where_incorrect_and_a_float32_quotient():
    rec = R.make_records(500, 5, 1)
    sp = C.speedup(rec.correct, rec.t_torch, rec.t_kernel)
    assert np.array_equal(sp == 0, rec.correct == 0)
    q64 = rec.t_torch.astype(np.float64) / rec.t_kernel.astype(np.float64)
    m = rec.correct.astype(bool)
    assert np.array_equal(sp[m], q64[m].astype(np.float32))          # correctly rounded quotient


def test_fast_p_is_strict_and_is_a_fraction_of_tasks():
    s = np.array([0.0, 1.0, 1.0000001, 5.0, 7.5], np.float32)
    assert C.fast_p(s, 1.0) == 3 / 5          # 1.0 itself does not count
    assert C.fast_p(s, 5.0) == 1 / 5
    assert C.fast_p(s, 0.0) == 4 / 5          # an incorrect kernel (speedup 0) never counts
    assert C.fast_p(s, 100.0) == 0.0


def test_arl_constant_and_arithmetic_series():
    assert C.arl(np.full((7, 3), 1234)) == 1234.0
    L = np.arange(1, 21).reshape(4, 5)
    assert C.arl(L) == 10.5
    assert C.arl(L.T) == 10.5                 # a mean over both axes


def test_pearson_closed_forms_and_library_special_case():
    x = np.arange(1, 51).reshape(10, 5)
    ones = np.ones((10, 5), np.uint8)
    r, n = C.pearson(x, (3.0 * x + 2).astype(np.float32), ones)
    assert n == 50 and abs(r - 1.0) < 1e-12
    r, _ = C.pearson(x, (100.0 - 2 * x).astype(np.float32), ones)
    assert abs(r + 1.0) < 1e-12
    rec = R.make_records(2000, 5, 2)
    sp = C.speedup(rec.correct, rec.t_torch, rec.t_kernel)
    r, n = C.pearson(rec.length, sp, rec.correct)
    m = rec.correct.astype(bool)
    assert n == m.sum()
    assert abs(r - np.corrcoef(rec.length[m].astype(np.float64), sp[m].astype(np.float64))[0, 1]) < 1e-10
    mask = np.zeros_like(rec.correct); mask[0, 0] = 1
    assert np.isnan(C.pearson(rec.length, sp, mask)[0])              # fewer than two samples
    assert np.isnan(C.pearson(np.full((10, 5), 7), sp[:10], ones)[0])    # a constant column


def brute_rule_a(correct, sp, L):
    out = []
    for i in range(L.shape[0]):
        shortest = [j for j in range(L.shape[1]) if all(L[i, j] <= L[i, k] for k in range(L.shape[1]))]
        j = min(shortest)
        ok = bool(correct[i, j]) and all(sp[i, j] >= sp[i, k] for k in range(L.shape[1]))
        out.append(j if ok else -1)
    return out


def test_rule_a_brute_force_on_all_small_cases():
    # every assignment of 3 generations with lengths in {1, 2} and speedups in {0 (incorrect), 1, 2}
    for lens in itertools.product([1, 2], repeat=3):
        for sps in itertools.product([0.0, 1.0, 2.0], repeat=3):
            L = np.array([lens]); sp = np.array([sps], np.float32); correct = (sp > 0)
            assert list(C.rule_a(correct, sp, L)) == brute_rule_a(correct, sp, L), (lens, sps)


def test_rule_a_and_b_invariants_on_synthetic_records():
    rec = R.make_records(3000, 5, 3)
    sp = C.speedup(rec.correct, rec.t_torch, rec.t_kernel)
    a = C.rule_a(rec.correct, sp, rec.length)
    kept = np.flatnonzero(a >= 0)
    rows = np.arange(len(a))
    assert (rec.correct[kept, a[kept]] == 1).all()
    assert (rec.length[kept, a[kept]] == rec.length[kept].min(axis=1)).all()
    assert (sp[kept, a[kept]] == sp[kept].max(axis=1)).all()
    # a task whose shortest generation is correct and fastest must be kept
    j0 = rec.length.argmin(axis=1)
    must = (rec.correct[rows, j0] == 1) & (sp[rows, j0] >= sp.max(axis=1))
    assert np.array_equal(must, a >= 0)
    b = C.rule_b(sp)
    assert np.array_equal(b, sp > 5) and b.sum() > 0 and not b[rec.correct == 0].any()
    assert not C.rule_b(np.array([[5.0]], np.float32)).any()          # strictly greater than 5


def test_selectors_pick_and_rank():
    rec = R.make_records(1500, 5, 4)
    sp = C.speedup(rec.correct, rec.t_torch, rec.t_kernel)
    has = rec.correct.any(axis=1)
    K = 200
    for name, (pick, keep) in {
        "random": C.select_random(rec.correct, rec.sample_key, rec.task_key, K),
        "max": C.select_max_length(rec.correct, rec.length, K),
        "min": C.select_min_length(rec.correct, rec.length, K),
        "speedup": C.select_speedup(rec.correct, sp, K),
    }.items():
        assert np.array_equal(pick >= 0, has), name
        rows = np.flatnonzero(has)
        assert (rec.correct[rows, pick[rows]] == 1).all(), name
        assert keep.sum() == min(K, has.sum()) and not keep[~has].any(), name
    pick, keep = C.select_max_length(rec.correct, rec.length, K)
    rows = np.flatnonzero(has)
    key = np.where(rec.correct[rows] == 1, rec.length[rows], -1).max(axis=1)
    assert (rec.length[rows, pick[rows]] == key).all()
    assert key[keep[rows]].min() >= key[~keep[rows]].max()            # the K longest
    pick, keep = C.select_speedup(rec.correct, sp, K)
    key = sp[rows].max(axis=1)
    assert (sp[rows, pick[rows]] == key).all() and key[keep[rows]].min() >= key[~keep[rows]].max()
    # k larger than the number of tasks with a correct kernel keeps them all
    assert C.select_min_length(rec.correct, rec.length, 10 ** 6)[1].sum() == has.sum()


def test_top_k_ties_go_to_the_lower_task_index():
    correct = np.ones((4, 1), np.uint8)
    L = np.array([[7], [9], [9], [7]])
    assert list(np.flatnonzero(C.select_max_length(correct, L, 1)[1])) == [1]
    assert list(np.flatnonzero(C.select_min_length(correct, L, 1)[1])) == [0]
    assert list(np.flatnonzero(C.select_max_length(correct, L, 3)[1])) == [0, 1, 2]


def test_difficulty_bins_use_exact_integer_comparison():
    L = np.array([[3999, 4000, 4001], [4000, 4000, 4000], [8500, 8500, 8500], [8500, 8500, 8501], [1, 1, 1]])
    assert list(C.difficulty(L)) == [1, 1, 1, 2, 0]                   # 4000 is medium, 8500 is medium
    assert list(C.difficulty(np.array([[3999, 3999, 4001]]))) == [0]  # mean 3999.67 < 4000


def test_synthetic_records_have_the_stated_shape():
    rec = R.make_records()
    assert rec.correct.shape == (18162, 5) and rec.length.max() <= 32768 and rec.length.min() >= 64
    frac_tasks = rec.correct.any(axis=1).mean()
    assert 0.35 < frac_tasks < 0.75 and 0.15 < rec.correct.mean() < 0.40
    sp = C.speedup(rec.correct, rec.t_torch, rec.t_kernel)
    r, _ = C.pearson(rec.length, sp, rec.correct)
    assert abs(r) < 0.1                                               # length says almost nothing about speedup
    short, long_ = rec.length < 5000, rec.length > 9000
    assert rec.correct[short].mean() > rec.correct[long_].mean()      # shorter traces are correct more often
