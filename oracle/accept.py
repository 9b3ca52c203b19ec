"""Acceptance oracle: greedy verification (Eq. 4), Relaxed Verification (Eq. 8).

Test infrastructure only (see the package docstring).

Row i-1 of the logits (0-based) is the distribution q_i that verifies draft
token i.  Drafts are checked in order; the first failure stops the prefix
(Section 2.1: later drafts are discarded and the failed position is corrected by
argmax q_c).  When every draft passes, the last row yields one more token.

Modes
  STRICT  (0)  x_i == argmax q_i                                   (Eq. 4)
  RELAXED (1)  x_i in TopK(q_i, k)  and  q_i(x_i) > p              (Eq. 8)
  TOPK    (2)  x_i in TopK(q_i, k)                                 (Eq. 7)
  TOPP    (3)  x_i == argmax q_i  or  q_i(x_i) > p                 (Section 4.3.2, "top-p")
  RELAXED_ARGMAX (4)  x_i == argmax q_i  or  Eq. 8                  (Eq. 8 read with the "highest probability
               or" of Section 4.3.2: the arg-max is accepted whatever its probability, so this rule accepts
               whatever STRICT or RELAXED accepts)

Ties between equal logits rank the smaller token id first.  Probabilities are
softmax at temperature 1, evaluated in fp64 from fp32 differences (l - max).
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

STRICT, RELAXED, TOPK, TOPP, RELAXED_ARGMAX = 0, 1, 2, 3, 4


def argmax_row(row: np.ndarray) -> int:
    return int(np.argmax(row))          # numpy returns the first (smallest id) maximum


def rank_of(row: np.ndarray, t: int) -> int:
    """Number of tokens ranked ahead of t (0 = top)."""
    lt = row[t]
    return int((row > lt).sum() + (row[:t] == lt).sum())


def prob_of(row: np.ndarray, t: int) -> float:
    """softmax(row)[t] in fp64; the shift (l - max) is taken in fp32."""
    row = np.asarray(row, dtype=np.float32)
    shifted = (row - row.max()).astype(np.float64)
    return float(np.exp(shifted[t]) / np.exp(shifted).sum())


def passes(row: np.ndarray, t: int, mode: int, k: int, p: float) -> bool:
    if mode == STRICT:
        return t == argmax_row(row)
    if mode == RELAXED:
        return rank_of(row, t) < k and prob_of(row, t) > p
    if mode == TOPK:
        return rank_of(row, t) < k
    if mode == TOPP:
        return t == argmax_row(row) or prob_of(row, t) > p
    if mode == RELAXED_ARGMAX:
        return t == argmax_row(row) or (rank_of(row, t) < k and prob_of(row, t) > p)
    raise ValueError("mode")


def accept_one(logits: np.ndarray, tokens: np.ndarray, n_rows: int, mode: int,
               k: int, p: float) -> Tuple[int, list]:
    """logits [>=n_rows, V]; tokens[0] = pending token, tokens[1..n_rows-1] = drafts.

    Returns (a, emitted) with a = accepted drafts and emitted = the a accepted drafts
    followed by argmax of row a (correction if a < m, bonus if a == m).
    """
    m = n_rows - 1
    a = 0
    while a < m and passes(logits[a], int(tokens[a + 1]), mode, k, p):
        a += 1
    emitted = [int(t) for t in tokens[1:1 + a]] + [argmax_row(logits[a])]
    return a, emitted


def accept_batch(logits: np.ndarray, tokens: np.ndarray, n_rows: np.ndarray, mode: int,
                 k: int = 2, p: float = 0.1) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """logits fp32 [B, K+1, V], tokens int32 [B, K+1], n_rows int32 [B].

    Returns n_accept int32[B], out_tokens int32[B, K+1] (padded -1), n_out int32[B].
    A sequence with n_rows == 0 is inactive: n_accept = n_out = 0.
    """
    B, R, _ = logits.shape
    n_acc = np.zeros(B, dtype=np.int32)
    out = np.full((B, R), -1, dtype=np.int32)
    n_out = np.zeros(B, dtype=np.int32)
    for b in range(B):
        if n_rows[b] <= 0:
            continue
        a, em = accept_one(logits[b], tokens[b], int(n_rows[b]), mode, k, p)
        n_acc[b] = a
        out[b, :len(em)] = em
        n_out[b] = len(em)
    return n_acc, out, n_out
