"""Seeded synthetic generation records for the curation arithmetic (no arithmetic of the method
here: only random draws).  One record per (task, generation): whether the kernel was correct,
the two run times, the reasoning length in tokens, and the random keys that stand for the
method's own random choices.

Shaped like the paper's synthesis run: 18,162 tasks x 5 generations; about half the tasks with at
least one correct kernel and about a quarter of the kernels correct; lengths of a few thousand
tokens under a 32,768 limit, longer traces less often correct; speedups log-normal around 1 with a
thin tail beyond 5 and almost uncorrelated with the length.  No record of the paper's dataset is
used or reproduced.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class Records:
    correct: np.ndarray      # [N][M] uint8
    t_torch: np.ndarray      # [N][M] float32, milliseconds
    t_kernel: np.ndarray     # [N][M] float32, milliseconds
    length: np.ndarray       # [N][M] int32, reasoning tokens
    sample_key: np.ndarray   # [N][M] float32 in [0, 1)
    task_key: np.ndarray     # [N] float32 in [0, 1)


def make_records(num_tasks=18162, gens=5, seed=73590) -> Records:
    r = np.random.Generator(np.random.Philox(key=[seed, 11]))
    N, M = num_tasks, gens
    task_difficulty = r.normal(0.0, 1.0, size=(N, 1))                      # harder tasks: longer, less often correct
    length = np.exp(8.6 + 0.35 * task_difficulty + 0.30 * r.normal(size=(N, M)))
    length = np.clip(np.rint(length), 64, 32768).astype(np.int32)
    z = (length - 6000.0) / 3000.0
    p_correct = 1.0 / (1.0 + np.exp(1.0 + 0.6 * task_difficulty + 0.5 * z))
    correct = (r.random((N, M)) < p_correct).astype(np.uint8)
    t_torch = np.exp(r.normal(-1.0, 1.0, size=(N, 1)) + np.zeros((N, M))).astype(np.float32)
    t_kernel = (t_torch / np.exp(r.normal(0.0, 0.7, size=(N, M)))).astype(np.float32)
    return Records(correct, t_torch, t_kernel, length, r.random((N, M), dtype=np.float32),
                   r.random(N, dtype=np.float32))
