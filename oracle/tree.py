"""Tree-based drafting oracle: sub-tree retrieval, pseudo-sequence, tree attention inputs and
verification of the token tree (Section 3.3 and the tree part of Section 3.4).

Test infrastructure only (see the package docstring).

Retrieve(D, tail, K) returns the sub-tree T_t of the group's trie under the matched tail: a
node is a sequence of continuation tokens, its frequency the number of occurrences of the
tail that are followed by that sequence inside one document.  When the sub-tree holds more
than K tokens the K of highest frequency are kept (Section 3.3); a parent is never rarer than
its child, so ranking nodes by (frequency descending, depth ascending, token path in
lexicographic order) keeps every kept node's parent, and among siblings prefers the one chain
drafting would follow.  The pseudo-sequence S_t lists the kept nodes in
depth-first order, children by (frequency descending, token id ascending), so its first branch
is the chain that greedy chain drafting follows; P_t is the node's depth and M_t lets a node
see its ancestors and itself (plus the whole cached context).

Verification walks the tree: a node is verified if its parent is (the root, the pending token,
always is) and its token passes the criterion on the distribution of its parent's row; the
verified node of greatest depth wins (the first in depth-first order among equals), its path is
accepted and one more token comes from its own row.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import accept as acc
from . import retrieval as ret


def continuations(pool: np.ndarray, hi: int, occ: np.ndarray, K: int,
                  history: Optional[np.ndarray] = None, hocc: Optional[np.ndarray] = None) -> List[List[int]]:
    """Up to K tokens following every occurrence, cut at the document's (group's, history's) end.
    History occurrences first, as in the occurrence list."""
    out: List[List[int]] = []
    if history is not None and hocc is not None:
        for p in hocc:
            out.append([int(t) for t in history[p + 1:p + 1 + K]])
    for p in occ:
        c: List[int] = []
        for j in range(1, K + 1):
            if p + j >= hi or pool[p + j] == ret.SENTINEL:
                break
            c.append(int(pool[p + j]))
        out.append(c)
    return out


def build_tree(conts: List[List[int]], K: int) -> Tuple[List[int], List[int]]:
    """The K most frequent nodes of the trie of `conts`, as (tokens, parents) in depth-first order.

    Index 0 is reserved for the root by the caller: parents are 0-based indices into
    [root] + nodes, i.e. parent 0 = the root, and node j of the result is row j + 1.
    """
    # every trie node: path tuple -> frequency
    freq: Dict[tuple, int] = {}
    for c in conts:
        for d in range(1, len(c) + 1):
            key = tuple(c[:d])
            freq[key] = freq.get(key, 0) + 1
    ranked = sorted(freq, key=lambda k: (-freq[k], len(k), k))[:K]
    kept = set(ranked)
    assert all(len(k) == 1 or k[:-1] in kept for k in kept)      # closed under taking parents
    tokens: List[int] = []
    parents: List[int] = []

    def visit(path: tuple, row: int) -> None:
        kids = [k for k in kept if len(k) == len(path) + 1 and k[:-1] == path]
        for k in sorted(kids, key=lambda k: (-freq[k], k[-1])):
            tokens.append(k[-1])
            parents.append(row)
            visit(k, len(tokens))
    visit((), 0)
    return tokens, parents


def draft_tree_one(pool: np.ndarray, lo: int, hi: int, tail: np.ndarray, K: int, n_min: int, n_max: int,
                   min_draft: int = 1, max_occ: int = 0, history: Optional[np.ndarray] = None
                   ) -> Tuple[List[int], List[int], int]:
    """Token tree for one sequence: (tokens, parents, match_n), K nodes at most, depth K at most.

    The suffix length n shrinks from n_max exactly as for chain drafting: the first n whose tree
    has at least min_draft nodes wins, otherwise the largest tree (ties: larger n).
    """
    best: Tuple[List[int], List[int]] = ([], [])
    best_n = 0
    hist = None if history is None else np.asarray(history, dtype=np.int64)
    for n in range(min(n_max, len(tail)), n_min - 1, -1):
        t = np.asarray(tail[len(tail) - n:])
        occ = ret.occurrences(pool, lo, hi, t)
        hocc = np.zeros(0, dtype=np.int64)
        if hist is not None:
            hocc = ret.occurrences(hist, 0, len(hist), t)
            hocc = hocc[hocc + 1 < len(hist)]
        if max_occ > 0:
            hocc = hocc[:max_occ]
            occ = occ[:max_occ - len(hocc)]
        if occ.size + hocc.size == 0:
            continue
        tk, pr = build_tree(continuations(pool, hi, occ, K, hist, hocc), K)
        if len(tk) >= min_draft and len(tk) > 0:
            return tk, pr, n
        if len(tk) > len(best[0]):
            best, best_n = (tk, pr), n
    return best[0], best[1], (best_n if best[0] else 0)


def depths(parents: Sequence[int]) -> List[int]:
    """Depth of every row of [root] + nodes given the nodes' parents (root = depth 0)."""
    d = [0]
    for p in parents:
        d.append(d[p] + 1)
    return d


def accept_tree(logits: np.ndarray, tokens: np.ndarray, parents: Sequence[int], n_rows: int, mode: int,
                k: int, p: float) -> Tuple[int, List[int], List[int]]:
    """logits [>= n_rows, V]; tokens[0] = pending token, tokens[1..] = tree nodes in depth-first order,
    parents[i-1] = row of node i's parent.  Returns (a, emitted, path): a accepted drafts, the tokens
    emitted (the accepted path and one token from the last accepted row), and the accepted rows."""
    ok = [True] + [False] * (n_rows - 1)
    dep = depths(parents[:n_rows - 1])
    for i in range(1, n_rows):
        par = int(parents[i - 1])
        ok[i] = ok[par] and acc.passes(logits[par], int(tokens[i]), mode, k, p)
    best = 0
    for i in range(1, n_rows):
        if ok[i] and dep[i] > dep[best]:
            best = i
    path = []
    i = best
    while i != 0:
        path.append(i)
        i = int(parents[i - 1])
    path.reverse()
    emitted = [int(tokens[i]) for i in path] + [acc.argmax_row(logits[best])]
    return len(path), emitted, path
