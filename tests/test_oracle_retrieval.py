"""Pins for the retrieval oracle: hand examples, a literal trie, invariants."""
import os

import numpy as np
import pytest

from oracle import retrieval as R

GOLD = os.path.join(os.path.dirname(__file__), "golden", "retrieval_hand_examples.txt")


def _ints(s):
    s = s.strip()
    return [int(x) for x in s.split(",")] if s else []


def _cases():
    out = []
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        out.append((_ints(f[0]), _ints(f[1]), *map(int, f[2:7]), _ints(f[7]), int(f[8])))
    return out


@pytest.mark.parametrize("case", _cases())
def test_hand_examples(case):
    pool, tail, K, n_min, n_max, min_draft, max_occ, want, want_n = case
    pool = np.asarray(pool, dtype=np.int32)
    d, n = R.draft_one(pool, 0, len(pool), np.asarray(tail), K, n_min, n_max, min_draft, max_occ)
    assert d == want and n == want_n


class Trie:
    """Literal per-group trie of Section 3.2: every window of every document, to a fixed
    depth, is inserted as a branch; each node counts how many branches pass through it."""

    def __init__(self):
        self.kids, self.count = {}, 0

    def insert(self, toks):
        node = self
        for t in toks:
            node = node.kids.setdefault(int(t), Trie())
            node.count += 1

    def descend(self, toks):
        node = self
        for t in toks:
            node = node.kids.get(int(t))
            if node is None:
                return None
        return node


def build_trie(pool, lo, hi, depth):
    root = Trie()
    doc = []
    for t in list(pool[lo:hi]) + [-1]:
        if t == -1:
            for i in range(len(doc)):
                root.insert(doc[i:i + depth])
            doc = []
        else:
            doc.append(int(t))
    return root


def trie_draft(root, tail, K, n_min, n_max):
    """Longest-suffix-first retrieval, then the greedy highest-frequency root-to-leaf path."""
    for n in range(min(n_max, len(tail)), n_min - 1, -1):
        node = root.descend(tail[len(tail) - n:])
        if node is None:
            continue
        d = []
        while len(d) < K and node.kids:
            best = max(node.kids.items(), key=lambda kv: (kv[1].count, -kv[0]))
            d.append(best[0])
            node = best[1]
        if d:
            return d, n
    return [], 0


def _random_pool(rng, n_groups, vocab, max_len):
    toks, offs = [], [0]
    for _ in range(n_groups):
        ln = int(rng.integers(1, max_len))
        g = rng.integers(0, vocab, size=ln)
        g[rng.random(ln) < 0.08] = -1
        toks.extend(g.tolist())
        offs.append(len(toks))
    return np.asarray(toks, dtype=np.int32), np.asarray(offs, dtype=np.int64)


def test_matches_literal_trie():
    rng = np.random.default_rng(5)
    for trial in range(150):
        vocab = int(rng.integers(2, 7))
        pool, offs = _random_pool(rng, 3, vocab, 120)
        K, n_max = int(rng.integers(1, 7)), int(rng.integers(1, 5))
        n_min = int(rng.integers(1, n_max + 1))
        tries = [build_trie(pool, offs[g], offs[g + 1], n_max + K) for g in range(3)]
        for _ in range(20):
            g = int(rng.integers(0, 3))
            tail = rng.integers(0, vocab, size=int(rng.integers(1, 6))).tolist()
            want = trie_draft(tries[g], tail, K, n_min, n_max)
            got = R.draft_one(pool, int(offs[g]), int(offs[g + 1]), np.asarray(tail), K, n_min, n_max, 1, 0)
            assert got == want, (trial, pool.tolist(), tail, K, n_min, n_max)


def test_brute_force_occurrences_and_invariants():
    rng = np.random.default_rng(6)
    for trial in range(100):
        vocab = int(rng.integers(2, 6))
        pool, offs = _random_pool(rng, 2, vocab, 200)
        K, max_occ = 5, int(rng.integers(0, 4))
        for _ in range(10):
            g = int(rng.integers(0, 2))
            lo, hi = int(offs[g]), int(offs[g + 1])
            tail = rng.integers(0, vocab, size=3)
            for n in (1, 2, 3):
                occ = R.occurrences(pool, lo, hi, tail[3 - n:])
                brute = [p for p in range(lo + n - 1, hi)
                         if all(pool[p - n + 1 + j] == tail[3 - n + j] for j in range(n))]
                assert occ.tolist() == brute
            d, n = R.draft_one(pool, lo, hi, tail, K, 1, 3, 1, max_occ)
            assert len(d) <= K and (n == 0) == (len(d) == 0)
            if d:
                # every prefix of the draft follows some occurrence of the matched suffix
                occ = R.occurrences(pool, lo, hi, tail[3 - n:])
                if max_occ:
                    occ = occ[:max_occ]
                ok = [p for p in occ if p + len(d) < hi and pool[p + 1:p + 1 + len(d)].tolist() == d]
                assert ok
                # a longer suffix found nothing usable
                for n2 in range(3, n, -1):
                    o2 = R.occurrences(pool, lo, hi, tail[3 - n2:])
                    if max_occ:
                        o2 = o2[:max_occ]
                    assert R.walk(pool, hi, o2, K) == []


def test_min_draft_and_batch_layout():
    pool = np.asarray([1, 2, 3, 4, -1, 1, 2, 3, 5, -1, 1, 2, 3, 5, 9], dtype=np.int32)
    offs = np.asarray([0, 15], dtype=np.int64)
    tails = np.asarray([[0, 2, 3], [0, 0, 7], [6, 2, 3]], dtype=np.int32)
    tl = np.asarray([2, 1, 3], dtype=np.int32)
    d, ln, mn = R.draft_batch(pool, offs, tails, tl, np.zeros(3, np.int32), 4, 1, 3)
    assert d.tolist() == [[5, 9, -1, -1], [-1, -1, -1, -1], [5, 9, -1, -1]]
    assert ln.tolist() == [2, 0, 2] and mn.tolist() == [2, 0, 2]
    # groups do not leak into each other
    offs2 = np.asarray([0, 5, 15], dtype=np.int64)
    d, ln, mn = R.draft_batch(pool, offs2, tails[:1], tl[:1], np.asarray([0], np.int32), 4, 1, 3)
    assert d[0].tolist() == [4, -1, -1, -1] and mn[0] == 2


# ---- temporary branches (Section 3.2): the sequence's own text is one more document ----
TEMP_GOLD = os.path.join(os.path.dirname(__file__), "golden", "retrieval_temp_hand_examples.txt")


def _temp_cases():
    out = []
    for line in open(TEMP_GOLD):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        out.append((_ints(f[0]), _ints(f[1]), _ints(f[2]), *map(int, f[3:8]), _ints(f[8]), int(f[9])))
    return out


@pytest.mark.parametrize("case", _temp_cases())
def test_temp_hand_examples(case):
    pool, history, tail, K, n_min, n_max, min_draft, max_occ, want, want_n = case
    pool = np.asarray(pool, dtype=np.int32)
    d, n = R.draft_one(pool, 0, len(pool), np.asarray(tail), K, n_min, n_max, min_draft, max_occ,
                       history=np.asarray(history, dtype=np.int32))
    assert d == want and n == want_n


def test_temp_matches_literal_trie():
    """Inserting the history's windows into the group's trie as one more document and walking
    the trie gives the same draft as the oracle with `history` (no occurrence cap)."""
    rng = np.random.default_rng(15)
    for trial in range(120):
        vocab = int(rng.integers(2, 6))
        pool, offs = _random_pool(rng, 2, vocab, 100)
        K, n_max = int(rng.integers(1, 7)), int(rng.integers(1, 5))
        n_min = int(rng.integers(1, n_max + 1))
        for _ in range(12):
            g = int(rng.integers(0, 2))
            hist = rng.integers(0, vocab, size=int(rng.integers(1, 40)))
            root = build_trie(pool, offs[g], offs[g + 1], n_max + K)
            for i in range(len(hist)):
                root.insert(hist[i:i + n_max + K].tolist())
            tail = hist[-int(rng.integers(1, 6)):].tolist()      # the tail is the end of the history
            want = trie_draft(root, tail, K, n_min, n_max)
            got = R.draft_one(pool, int(offs[g]), int(offs[g + 1]), np.asarray(tail), K, n_min, n_max, 1, 0,
                              history=hist)
            assert got == want, (trial, pool.tolist(), hist.tolist(), tail, K, n_min, n_max)


def test_temp_history_first_under_cap_and_reduces_to_plain():
    rng = np.random.default_rng(16)
    for trial in range(60):
        vocab = int(rng.integers(2, 5))
        pool, offs = _random_pool(rng, 1, vocab, 150)
        hist = rng.integers(0, vocab, size=30)
        tail = hist[-3:]
        # an empty history, or one too short to hold a continuation, changes nothing
        a = R.draft_one(pool, 0, len(pool), tail, 5, 1, 3, 1, 0)
        assert R.draft_one(pool, 0, len(pool), tail, 5, 1, 3, 1, 0, history=np.zeros(0, dtype=np.int32)) == a
        assert R.draft_one(pool, 0, len(pool), tail, 5, 1, 3, 1, 0, history=tail[-1:]) == a
        # with a cap of one occurrence and a history hit, only the history speaks
        for n in (3, 2, 1):
            hocc = R.occurrences(hist.astype(np.int64), 0, len(hist), tail[3 - n:])
            hocc = hocc[hocc + 1 < len(hist)]
            if hocc.size:
                d, nn = R.draft_one(pool, 0, len(pool), tail, 4, n, n, 1, 1, history=hist)
                p = int(hocc[0])
                assert nn == n and d == hist[p + 1:p + 1 + 4].tolist()
                break
