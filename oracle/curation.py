"""CPU oracle of the paper's curation arithmetic (test infrastructure only: tests, smoke and the
bench's CPU baseline may import it; the product path never does).

Plain numpy, one definition per function, written from the paper's text:

  speedup            Eq. (1):  T_torch / T_kernel * 1[correct]
  fast_p             Eq. (2):  (1/N) sum_i 1[speedup_i > p]
  arl                Eq. (3):  (1/(N M)) sum_ij L[i, j]
  rule_a             Sec. 3.5 (a): per task, the generation with the shortest reasoning length is kept
                     if it also has the highest speedup of the task's generations
  rule_b             Sec. 3.5 (b): kernels with speedup > 5
  pearson            Sec. 3.4, Observation 2: correlation of reasoning length and speedup
  select_*           Sec. 5: the four ablation selections (random / longest / shortest / fastest correct
                     kernel per task, then the K tasks that rank first by that key)
  difficulty         Sec. 6.1 / Table 4: tasks binned by their average reasoning length

Precision: speedup is a float32 quotient (IEEE division of the two float32 times), because the
comparisons `speedup > p` and the rankings decide integers and both sides must take them in the
same precision; every sum is exact integer arithmetic or float64.

Readings where the text is silent: ties in "shortest" / "longest" / "highest" go to the lowest
generation index; rule (a) needs the shortest generation to be correct (an incorrect one has
speedup 0 and nothing to add to a dataset) and "highest" means >= every other generation's
speedup; tasks that tie in a ranking go by lower task index; the random selection draws no
numbers itself -- it ranks by keys that the caller passes in; the correlation coefficient of a
constant column (or of fewer than two samples) is NaN.
"""
from __future__ import annotations

import numpy as np


def speedup(correct, t_torch, t_kernel):
    """Eq. (1).  correct [N][M] bool/u8, times [N][M] float32 -> float32 [N][M]."""
    q = np.asarray(t_torch, np.float32) / np.asarray(t_kernel, np.float32)
    return np.where(np.asarray(correct).astype(bool), q, np.float32(0)).astype(np.float32)


def fast_p(speedups, p):
    """Eq. (2) over one speedup per task: fraction of tasks with speedup > p."""
    s = np.asarray(speedups, np.float32)
    return float(np.count_nonzero(s > np.float32(p))) / s.size


def arl(length):
    """Eq. (3): mean reasoning length over all N x M samples."""
    L = np.asarray(length, np.int64)
    return float(L.sum()) / L.size


def rule_a(correct, sp, length):
    """Sec. 3.5 (a).  Returns int32 [N]: the kept generation of each task, or -1."""
    correct = np.asarray(correct).astype(bool)
    N, M = correct.shape
    out = np.full(N, -1, np.int32)
    for i in range(N):
        j = int(np.argmin(length[i]))                    # first of the shortest
        if correct[i, j] and sp[i, j] >= sp[i].max():
            out[i] = j
    return out


def rule_b(sp, threshold=5.0):
    """Sec. 3.5 (b).  bool [N][M]: speedup > threshold."""
    return np.asarray(sp, np.float32) > np.float32(threshold)


def pearson(length, sp, correct):
    """Correlation coefficient of (length, speedup) over the correct samples, in float64.
    Returns (r, n)."""
    m = np.asarray(correct).astype(bool)
    x = np.asarray(length, np.float64)[m]
    y = np.asarray(sp, np.float64)[m]
    n = x.size
    if n < 2:
        return float("nan"), n
    # the textbook definition, centred on the means:
    #   r = sum (x - mx)(y - my) / sqrt( sum (x - mx)^2 * sum (y - my)^2 )
    dx, dy = x - x.mean(), y - y.mean()
    cov = (dx * dy).sum()
    vx = (dx * dx).sum()
    vy = (dy * dy).sum()
    if not vx * vy > 0:                                  # a constant column: the coefficient is undefined
        return float("nan"), n
    return float(cov / np.sqrt(vx * vy)), n


def _pick(correct, key, largest):
    """Per task the correct generation with the largest (smallest) key, lowest index on ties; -1 if
    no generation is correct."""
    correct = np.asarray(correct).astype(bool)
    N, M = correct.shape
    out = np.full(N, -1, np.int32)
    for i in range(N):
        best = -1
        for j in range(M):
            if not correct[i, j]:
                continue
            if best < 0 or (key[i, j] > key[i, best] if largest else key[i, j] < key[i, best]):
                best = j
        out[i] = best
    return out


def _top_k(pick, task_key, k, largest):
    """bool [N]: among the tasks that have a pick, the k that rank first by task_key (ties: lower
    task index first)."""
    idx = np.flatnonzero(pick >= 0)
    keys = np.asarray(task_key)[idx]
    order = np.argsort(-keys if largest else keys, kind="stable")
    keep = np.zeros(pick.shape[0], bool)
    keep[idx[order[:k]]] = True
    return keep


def select_random(correct, sample_key, task_key, k):
    """5K-random: per task the correct generation with the largest sample key; then the k tasks with
    the largest task key.  (The keys stand for the paper's random draws.)"""
    pick = _pick(correct, np.asarray(sample_key, np.float32), True)
    return pick, _top_k(pick, np.asarray(task_key, np.float32), k, True)


def select_max_length(correct, length, k):
    """5K-max: per task the correct generation with the longest reasoning; the k longest overall."""
    L = np.asarray(length, np.int64)
    pick = _pick(correct, L, True)
    key = np.where(pick >= 0, L[np.arange(L.shape[0]), np.maximum(pick, 0)], 0)
    return pick, _top_k(pick, key, k, True)


def select_min_length(correct, length, k):
    """5K-min: per task the correct generation with the shortest reasoning; the k shortest overall."""
    L = np.asarray(length, np.int64)
    pick = _pick(correct, L, False)
    key = np.where(pick >= 0, L[np.arange(L.shape[0]), np.maximum(pick, 0)], 0)
    return pick, _top_k(pick, key, k, False)


def select_speedup(correct, sp, k):
    """5K-speedup: per task the correct generation with the highest speedup; the k fastest overall."""
    S = np.asarray(sp, np.float32)
    pick = _pick(correct, S, True)
    key = np.where(pick >= 0, S[np.arange(S.shape[0]), np.maximum(pick, 0)], np.float32(0))
    return pick, _top_k(pick, key, k, True)


def difficulty(length, easy_below=4000, hard_above=8500):
    """Table 4: 0 (easy) if the task's mean reasoning length < easy_below, 2 (hard) if > hard_above,
    else 1.  Compared as integers: sum < M * bound, so no rounding is involved."""
    L = np.asarray(length, np.int64)
    M = L.shape[1]
    s = L.sum(axis=1)
    return np.where(s < M * easy_below, 0, np.where(s > M * hard_above, 2, 1)).astype(np.uint8)
