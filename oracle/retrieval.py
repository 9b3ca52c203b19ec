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

Temporary branches (Section 3.2): while one text is generated, its prompt and the
tokens generated so far are in the trie as well and leave it afterwards.  Here that
text (`history`) is one more document searched beside the group: its occurrences of the
tail that still have a following token join the occurrence list, ahead of the group's
(they are the text at hand), before the list is cut to max_occ; frequencies add up.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

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


def walk(pool: np.ndarray, hi: int, occ: np.ndarray, K: int,
         history: Optional[np.ndarray] = None, hocc: Optional[np.ndarray] = None) -> List[int]:
    """Greedy max-frequency chain of continuations after the occurrences.

    occ are positions in the pool (continuations stay inside the group and the document);
    hocc are positions in `history`, a single document of its own.
    """
    alive = occ
    halive = np.zeros(0, dtype=np.int64) if hocc is None else hocc
    out: List[int] = []
    for j in range(1, K + 1):
        alive = alive[alive + j < hi]              # stay inside the group
        nxt = pool[alive + j] if alive.size else np.zeros(0, dtype=np.int64)
        keep = nxt != SENTINEL                     # stay inside the document
        alive, nxt = alive[keep], nxt[keep]
        if history is not None:
            halive = halive[halive + j < len(history)]
            hnxt = history[halive + j] if halive.size else np.zeros(0, dtype=np.int64)
        else:
            hnxt = np.zeros(0, dtype=np.int64)
        if alive.size + halive.size == 0:
            break
        vals, cnt = np.unique(np.concatenate([np.asarray(nxt, dtype=np.int64),
                                              np.asarray(hnxt, dtype=np.int64)]), return_counts=True)
        best = int(vals[int(np.argmax(cnt))])      # vals ascending: first max = smallest id
        out.append(best)
        alive = alive[nxt == best]
        halive = halive[hnxt == best]
    return out


def draft_one(pool: np.ndarray, lo: int, hi: int, tail: np.ndarray, K: int,
              n_min: int, n_max: int, min_draft: int = 1, max_occ: int = 0,
              history: Optional[np.ndarray] = None) -> Tuple[List[int], int]:
    """Draft for one sequence.  tail = its last tokens (any length, most recent last).

    Returns (draft tokens, match_n).  For n = min(n_max, len(tail)) down to n_min the
    first draft of length >= min_draft wins; otherwise the longest (ties: larger n).
    An empty draft reports match_n = 0.  history (optional) = the sequence's own prompt
    and generated tokens, searched as a temporary branch.
    """
    best: List[int] = []
    best_n = 0
    hist = None if history is None else np.asarray(history, dtype=np.int64)
    for n in range(min(n_max, len(tail)), n_min - 1, -1):
        t = np.asarray(tail[len(tail) - n:])
        occ = occurrences(pool, lo, hi, t)
        hocc = np.zeros(0, dtype=np.int64)
        if hist is not None:
            hocc = occurrences(hist, 0, len(hist), t)
            hocc = hocc[hocc + 1 < len(hist)]      # an occurrence at the very end continues nowhere
        if max_occ > 0:
            hocc = hocc[:max_occ]
            occ = occ[:max_occ - len(hocc)]
        if occ.size + hocc.size == 0:
            continue
        d = walk(pool, hi, occ, K, hist, hocc)
        if len(d) >= min_draft and len(d) > 0:
            return d, n
        if len(d) > len(best):
            best, best_n = d, n
    return best, (best_n if best else 0)


def draft_batch(pool: np.ndarray, group_offsets: np.ndarray, tails: np.ndarray,
                tail_len: np.ndarray, group_id: np.ndarray, K: int, n_min: int,
                n_max: int, min_draft: int = 1, max_occ: int = 0,
                histories: Optional[Sequence[np.ndarray]] = None
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
        # a group id outside the pool searches nothing of the pool (the history alone, if given)
        lo, hi = (int(group_offsets[g]), int(group_offsets[g + 1])) if 0 <= g < len(group_offsets) - 1 else (0, 0)
        tl = int(tail_len[b])
        d, n = draft_one(pool, lo, hi, tails[b, width - tl:], K, n_min, n_max, min_draft, max_occ,
                         None if histories is None else histories[b])
        draft[b, :len(d)] = d
        dlen[b] = len(d)
        mn[b] = n
    return draft, dlen, mn
