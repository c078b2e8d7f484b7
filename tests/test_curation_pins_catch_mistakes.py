"""Do the curation pins pin?  Each test of tests/test_curation_pins.py is run against copies of the
curation oracle into which one plausible mistake has been planted (on the CPU, in this file only:
a dropped indicator, >= for >, an inverted quotient, the wrong tie rule, an ignored mask, ...).
Every planted mistake must make at least one pin fail; the unmodified oracle passes them all."""
import types

import numpy as np
import pytest

from oracle import curation as REAL
import test_curation_pins as PINS

PIN_TESTS = [getattr(PINS, n) for n in dir(PINS) if n.startswith("test_")]


def _pick(correct, key, largest, need_correct=True):
    correct = np.asarray(correct).astype(bool)
    out = np.full(correct.shape[0], -1, np.int32)
    for i in range(correct.shape[0]):
        best = -1
        for j in range(correct.shape[1]):
            if need_correct and not correct[i, j]:
                continue
            if best < 0 or (key[i, j] > key[i, best] if largest else key[i, j] < key[i, best]):
                best = j
        out[i] = best
    return out


def _top_k(pick, key, k, largest, ties_high=False):
    idx = np.flatnonzero(pick >= 0)
    keys = np.asarray(key)[idx]
    if ties_high:
        idx, keys = idx[::-1], keys[::-1]
    order = np.argsort(-keys if largest else keys, kind="stable")
    keep = np.zeros(pick.shape[0], bool)
    keep[idx[order[:k]]] = True
    return keep


def _sel_len(correct, length, k, largest, need_correct=True, ties_high=False):
    L = np.asarray(length, np.int64)
    pick = _pick(correct, L, largest, need_correct)
    key = np.where(pick >= 0, L[np.arange(L.shape[0]), np.maximum(pick, 0)], 0)
    return pick, _top_k(pick, key, k, largest, ties_high)


def _rule_a(correct, sp, length, longest=False, strict=False, need_correct=True):
    correct = np.asarray(correct).astype(bool)
    out = np.full(correct.shape[0], -1, np.int32)
    for i in range(correct.shape[0]):
        j = int(np.argmax(length[i]) if longest else np.argmin(length[i]))
        others = np.delete(np.asarray(sp[i]), j)
        fastest = (sp[i, j] > others).all() if strict else sp[i, j] >= np.asarray(sp[i]).max()
        if (correct[i, j] or not need_correct) and fastest:
            out[i] = j
    return out


def _pearson(length, sp, correct, centred=True, masked=True):
    m = np.asarray(correct).astype(bool) if masked else np.ones(np.asarray(correct).shape, bool)
    x = np.asarray(length, np.float64)[m]; y = np.asarray(sp, np.float64)[m]
    n = x.size
    if n < 2:
        return float("nan"), n
    if centred:
        x = x - x.mean(); y = y - y.mean()
    d = (x * x).sum() * (y * y).sum()
    if not d > 0:
        return float("nan"), n
    return float((x * y).sum() / np.sqrt(d)), n


MISTAKES = {
    "speedup without the correctness indicator":
        dict(speedup=lambda c, tt, tk: (np.asarray(tt, np.float32) / np.asarray(tk, np.float32)).astype(np.float32)),
    "speedup inverted":
        dict(speedup=lambda c, tt, tk: np.where(np.asarray(c).astype(bool), np.asarray(tk, np.float32) / np.asarray(tt, np.float32),
                                                np.float32(0)).astype(np.float32)),
    "fast_p with >=":
        dict(fast_p=lambda s, p: float(np.count_nonzero(np.asarray(s, np.float32) >= np.float32(p))) / np.asarray(s).size),
    "fast_p over the correct kernels only":
        dict(fast_p=lambda s, p: float(np.count_nonzero(np.asarray(s, np.float32) > np.float32(p))) /
             max(1, np.count_nonzero(np.asarray(s) > 0))),
    "arl divided by the number of tasks":
        dict(arl=lambda L: float(np.asarray(L, np.int64).sum()) / np.asarray(L).shape[0]),
    "rule (a) takes the longest generation":
        dict(rule_a=lambda c, sp, L: _rule_a(c, sp, L, longest=True)),
    "rule (a) wants a strictly highest speedup":
        dict(rule_a=lambda c, sp, L: _rule_a(c, sp, L, strict=True)),
    "rule (a) keeps incorrect generations":
        dict(rule_a=lambda c, sp, L: _rule_a(c, sp, L, need_correct=False)),
    "rule (b) with >=":
        dict(rule_b=lambda sp, threshold=5.0: np.asarray(sp, np.float32) >= np.float32(threshold)),
    "correlation without centring":
        dict(pearson=lambda L, sp, c: _pearson(L, sp, c, centred=False)),
    "correlation over all samples":
        dict(pearson=lambda L, sp, c: _pearson(L, sp, c, masked=False)),
    "selection among incorrect generations too":
        dict(select_max_length=lambda c, L, k: _sel_len(c, L, k, True, need_correct=False)),
    "ranking ties go to the higher task index":
        dict(select_max_length=lambda c, L, k: _sel_len(c, L, k, True, ties_high=True),
             select_min_length=lambda c, L, k: _sel_len(c, L, k, False, ties_high=True)),
    "shortest selection returns the longest":
        dict(select_min_length=lambda c, L, k: _sel_len(c, L, k, True)),
    "difficulty compares the mean with <=":
        dict(difficulty=lambda L, easy_below=4000, hard_above=8500: np.where(
            np.asarray(L, np.float64).mean(axis=1) <= easy_below, 0,
            np.where(np.asarray(L, np.float64).mean(axis=1) >= hard_above, 2, 1)).astype(np.uint8)),
}


def failing_pins(module):
    failed = []
    saved = PINS.C
    PINS.C = module
    try:
        for t in PIN_TESTS:
            try:
                t()
            except Exception as e:                    # an assertion, or a crash the mistake provokes
                failed.append(f"{t.__name__}: {type(e).__name__}")
    finally:
        PINS.C = saved
    return failed


def test_the_oracle_passes_every_pin():
    assert failing_pins(REAL) == []


def test_the_restated_helpers_agree_with_the_oracle():
    # the helpers above, without a mistake, are the oracle's definitions: otherwise a mutant could fail for that reason
    clean = types.SimpleNamespace(**{k: getattr(REAL, k) for k in dir(REAL) if not k.startswith("_")})
    clean.rule_a = lambda c, sp, L: _rule_a(c, sp, L)
    clean.pearson = lambda L, sp, c: _pearson(L, sp, c)
    clean.select_max_length = lambda c, L, k: _sel_len(c, L, k, True)
    clean.select_min_length = lambda c, L, k: _sel_len(c, L, k, False)
    assert failing_pins(clean) == []


@pytest.mark.parametrize("name", list(MISTAKES))
def test_every_planted_mistake_fails_some_pin(name):
    mutant = types.SimpleNamespace(**{k: getattr(REAL, k) for k in dir(REAL) if not k.startswith("_")})
    for k, fn in MISTAKES[name].items():
        setattr(mutant, k, fn)
    assert failing_pins(mutant), f"no pin notices: {name}"
