"""Draft retrieval oracle: Retrieve(D, tail, K) of Eq. 5 (Section 3.3).

Test infrastructure only (see the package docstring).

A group's retrieval pool D is a token array made of documents separated by the
sentinel -1.  Section 3.2 stores D as a trie whose nodes are tokens; retrieving
with "the last n tokens as a prefix" returns the sub-tree under that path.  If
every window of every document is a branch, the node reached by (tail, c_1..c_j)
has frequency = number of places in the group where tail is followed by
c_1..c_j inside one document.  So the sub-tree is exactly the multiset of
continuations after every occurrence of the tail, and a linear scan over the
group is the plain definition.  The draft is the chain obtained by repeatedly
taking the most frequent next token (Section 3.3: when more than K tokens are
retrieved the most frequent ones are kept), ties to the smallest token id.
The suffix length n starts at n_max and shrinks while the draft is shorter than
min_draft (the dynamic adjustment of n in Section 3.3).
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np

SENTINEL = -1


def occurrences(pool: np.ndarray, lo: int, hi: int, tail: np.ndarray) -> np.ndarray:
    """Ascending end positions p in [lo, hi) with pool[p-n+1 .. p] == tail."""
    n = len(tail)
    size = hi - lo
    if n == 0 or size < n or (np.asarray(tail) < 0).any():
        return np.zeros(0, dtype=np.int64)
    g = pool[lo:hi]
    ok = np.ones(size - n + 1, dtype=bool)
    for j in range(n):
        ok &= g[j:size - n + 1 + j] == tail[j]
    return lo + np.nonzero(ok)[0].astype(np.int64) + (n - 1)


def walk(pool: np.ndarray, hi: int, occ: np.ndarray, K: int) -> List[int]:
    """Greedy max-frequency chain of continuations after the occurrences."""
    alive = occ
    out: List[int] = []
    for j in range(1, K + 1):
        alive = alive[alive + j < hi]              # stay inside the group
        if alive.size == 0:
            break
        nxt = pool[alive + j]
        keep = nxt != SENTINEL                     # stay inside the document
        alive, nxt = alive[keep], nxt[keep]
        if alive.size == 0:
            break
        vals, cnt = np.unique(nxt, return_counts=True)   # vals ascending
        best = int(vals[int(np.argmax(cnt))])            # first max = smallest id
        out.append(best)
        alive = alive[nxt == best]
    return out


def draft_one(pool: np.ndarray, lo: int, hi: int, tail: np.ndarray, K: int,
              n_min: int, n_max: int, min_draft: int = 1, max_occ: int = 0
              ) -> Tuple[List[int], int]:
    """Draft for one sequence.  tail = its last tokens (any length, most recent last).

    Returns (draft tokens, match_n).  For n = min(n_max, len(tail)) down to n_min the
    first draft of length >= min_draft wins; otherwise the longest (ties: larger n).
    An empty draft reports match_n = 0.
    """
    best: List[int] = []
    best_n = 0
    for n in range(min(n_max, len(tail)), n_min - 1, -1):
        occ = occurrences(pool, lo, hi, np.asarray(tail[len(tail) - n:]))
        if max_occ > 0:
            occ = occ[:max_occ]
        if occ.size == 0:
            continue
        d = walk(pool, hi, occ, K)
        if len(d) >= min_draft and len(d) > 0:
            return d, n
        if len(d) > len(best):
            best, best_n = d, n
    return best, (best_n if best else 0)


def draft_batch(pool: np.ndarray, group_offsets: np.ndarray, tails: np.ndarray,
                tail_len: np.ndarray, group_id: np.ndarray, K: int, n_min: int,
                n_max: int, min_draft: int = 1, max_occ: int = 0
                ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Batch form.  tails int32[B, n_max] right-aligned (last column = newest token).

    Returns draft int32[B, K] padded with -1, draft_len int32[B], match_n int32[B].
    """
    B = len(tail_len)
    draft = np.full((B, K), -1, dtype=np.int32)
    dlen = np.zeros(B, dtype=np.int32)
    mn = np.zeros(B, dtype=np.int32)
    width = tails.shape[1]
    for b in range(B):
        g = int(group_id[b])
        lo, hi = int(group_offsets[g]), int(group_offsets[g + 1])
        tl = int(tail_len[b])
        d, n = draft_one(pool, lo, hi, tails[b, width - tl:], K, n_min, n_max, min_draft, max_occ)
        draft[b, :len(d)] = d
        dlen[b] = len(d)
        mn[b] = n
    return draft, dlen, mn
