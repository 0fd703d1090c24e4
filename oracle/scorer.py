"""Oracle: step scorer and running-mean trace score (fp64).

TEST INFRASTRUCTURE ONLY - never imported by the product path.

Step scorer (Sec. 3.1 "Model Architecture"; Table 5 gives the shape
Input -> 512 (ReLU) -> 1): for the hidden state h of a step-end token

    a = ReLU(W1 h + b1)          W1 : [m, D], b1 : [m]
    z = w2 . a + b2              w2 : [m],    b2 scalar
    y = 1 / (1 + exp(-z))

Only step-end rows are scored (Algorithm 1: the scorer runs when the new
token closes a step).  Trace score (Sec. 3.3): the arithmetic mean of all
step scores the trace has produced so far.
"""
from __future__ import annotations

import numpy as np


def step_score(h, W1, b1, w2, b2) -> float:
    """Score of one hidden state; every operand is taken to float64."""
    h = np.asarray(h, dtype=np.float64)
    W1 = np.asarray(W1, dtype=np.float64)
    b1 = np.asarray(b1, dtype=np.float64)
    w2 = np.asarray(w2, dtype=np.float64)
    pre = W1 @ h + b1
    a = np.where(pre > 0.0, pre, 0.0)
    z = float(w2 @ a) + float(b2)
    return 1.0 / (1.0 + np.exp(-z))


def score_steps(hidden, boundary_mask, W1, b1, w2, b2) -> np.ndarray:
    """Scores for the rows whose mask is non-zero; NaN for the others.

    hidden : [M, D], boundary_mask : [M]; returns [M] float64.
    """
    hidden = np.asarray(hidden)
    M = hidden.shape[0]
    out = np.full(M, np.nan, dtype=np.float64)
    for i in range(M):
        if boundary_mask[i]:
            out[i] = step_score(hidden[i], W1, b1, w2, b2)
    return out


class TraceScores:
    """Per-trace running mean of step scores (Sec. 3.3).

    score_t = (1/n) sum_{i<=n} y_i^t.  A trace with no scored step yet reports
    `unscored_score` (the paper leaves 0/0 undefined; see the pool's notes).
    """

    def __init__(self, max_traces: int, unscored_score: float = 1.0):
        self.sum = np.zeros(max_traces, dtype=np.float64)
        self.cnt = np.zeros(max_traces, dtype=np.int64)
        self.unscored_score = float(unscored_score)

    def update(self, step_scores, boundary_mask, row_trace=None) -> None:
        """Fold one batch of rows in, in row order."""
        M = len(step_scores)
        for i in range(M):
            if boundary_mask[i]:
                t = i if row_trace is None else int(row_trace[i])
                self.sum[t] += float(step_scores[i])
                self.cnt[t] += 1

    def score(self, t: int) -> float:
        if self.cnt[t] == 0:
            return self.unscored_score
        return self.sum[t] / self.cnt[t]

    def scores(self) -> np.ndarray:
        return np.array([self.score(t) for t in range(len(self.sum))], dtype=np.float64)

    def clear(self, t: int) -> None:
        self.sum[t] = 0.0
        self.cnt[t] = 0


def scorer_flops(m: int, d: int) -> int:
    """Cost of one scorer call as the paper's overhead appendix counts it."""
    # first layer: m rows of (d multiply-adds); second layer: m multiply-adds
    return 2 * m * d + 2 * m
