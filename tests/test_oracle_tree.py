"""Pins for the tree-drafting oracle: hand examples, a literal trie, the chain as a special case,
branch-by-branch equivalence of the tree forward and of tree verification."""
import os

import numpy as np
import pytest
import torch

from oracle import accept as A
from oracle import forward as O
from oracle import retrieval as R
from oracle import tree as T
from paper_2408_05676_b200 import synth
from test_oracle_retrieval import _ints, _random_pool, build_trie

GOLD = os.path.join(os.path.dirname(__file__), "golden", "tree_hand_examples.txt")


def _cases():
    out = []
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        out.append((_ints(f[0]), _ints(f[1]), *map(int, f[2:7]), _ints(f[7]), _ints(f[8]), int(f[9])))
    return out


@pytest.mark.parametrize("case", _cases())
def test_hand_examples(case):
    pool, tail, K, n_min, n_max, min_draft, max_occ, want_t, want_p, want_n = case
    pool = np.asarray(pool, dtype=np.int32)
    tk, pr, n = T.draft_tree_one(pool, 0, len(pool), np.asarray(tail), K, n_min, n_max, min_draft, max_occ)
    assert (tk, pr, n) == (want_t, want_p, want_n)


def _paths(tokens, parents):
    """Root path (token tuple) of every node."""
    out = []
    for i, t in enumerate(tokens):
        out.append((out[parents[i] - 1] if parents[i] else ()) + (t,))
    return out


def test_matches_literal_trie_and_chain():
    rng = np.random.default_rng(21)
    n_cut = 0
    for trial in range(120):
        vocab = int(rng.integers(2, 6))
        pool, offs = _random_pool(rng, 2, vocab, 150)
        K, n_max = int(rng.integers(1, 9)), int(rng.integers(1, 4))
        for _ in range(12):
            g = int(rng.integers(0, 2))
            lo, hi = int(offs[g]), int(offs[g + 1])
            tail = rng.integers(0, vocab, size=n_max).tolist()
            tk, pr, n = T.draft_tree_one(pool, lo, hi, np.asarray(tail), K, 1, n_max, 1, 0)
            chain, cn = R.draft_one(pool, lo, hi, np.asarray(tail), K, 1, n_max, 1, 0)
            assert (n == 0) == (len(tk) == 0) and n == cn and len(tk) <= K
            if not tk:
                continue
            assert all(0 <= p <= i for i, p in enumerate(pr))           # a parent is an earlier row
            paths = _paths(tk, pr)
            assert len(set(paths)) == len(paths)
            # frequencies are the literal trie's counts; nothing left out is more frequent than
            # anything kept; when nothing had to be cut the whole sub-tree is there
            root = build_trie(pool, lo, hi, n + K).descend(tail[len(tail) - n:])
            fr = [root.descend(p).count for p in paths]
            everything = {}
            def collect(node, path):
                for t, kid in node.kids.items():
                    if len(path) < K:
                        everything[path + (t,)] = kid.count
                        collect(kid, path + (t,))
            collect(root, ())
            left_out = [c for p, c in everything.items() if p not in set(paths)]
            if left_out:
                n_cut += 1
                assert len(tk) == K and max(left_out) <= min(fr)
            else:
                assert len(tk) == len(everything)
            # depth-first order: a node's subtree is a contiguous run right after it; siblings by
            # (frequency descending, token ascending)
            for i in range(len(tk)):
                sub = [j for j in range(len(tk)) if paths[j][:len(paths[i])] == paths[i]]
                assert sub == list(range(i, i + len(sub)))
            for par in set(pr):
                kids = [i for i in range(len(tk)) if pr[i] == par]
                keys = [(-fr[i], tk[i]) for i in kids]
                assert keys == sorted(keys)
            # the first branch is the greedy chain, as far as the tree keeps it
            first, row = [], 0
            while True:
                kids = [i for i in range(len(tk)) if pr[i] == row]
                if not kids:
                    break
                first.append(tk[kids[0]])
                row = kids[0] + 1
            assert first == chain[:len(first)] and first
    assert n_cut > 50


def test_tree_with_history_counts_both_sources():
    pool = np.asarray([2, 3, 4, -1, 2, 3, 5], np.int32)
    hist = np.asarray([2, 3, 5, 7, 2, 3], np.int32)
    tk, pr, n = T.draft_tree_one(pool, 0, len(pool), np.asarray([2, 3]), 4, 1, 2, 1, 0, history=hist)
    # after "2,3": history 5,7,2,3 ; pool 4 ; pool 5  ->  5 (x2), 4 (x1), 5-7 (x1), then 5-7-2
    assert (tk, pr, n) == ([5, 7, 2, 4], [0, 1, 2, 0], 2)


@pytest.fixture(scope="module")
def model():
    cfg = synth.model_cfg("tiny")
    return cfg, synth.make_weights(cfg, seed=0)


def _random_tree(rng, m, vocab):
    parents = [int(rng.integers(0, i + 1)) for i in range(m)]
    # depth-first order: re-index so that every subtree is contiguous
    kids = {}
    for i, p in enumerate(parents):
        kids.setdefault(p, []).append(i + 1)
    order, par_new = [], []
    def visit(row, new_row):
        for k in kids.get(row, []):
            order.append(k)
            par_new.append(new_row)
            visit(k, len(order))
    visit(0, 0)
    return rng.integers(0, vocab, size=m + 1).astype(np.int32), par_new


def test_tree_forward_equals_chain_forward_on_every_branch(model):
    """A node's logits and cached K/V depend only on its root path: running that path as a chain
    (the pinned chain forward) gives the same values, at cache slot ctx + depth."""
    cfg, W = model
    rng = np.random.default_rng(3)
    kv = O.KVCache(cfg, 1, 64)
    ctx_tok = rng.integers(0, cfg["vocab"], size=11)
    O.forward(W, cfg, kv, [0], [ctx_tok])
    kv.ctx[0] = 11
    for trial in range(3):
        tokens, parents = _random_tree(rng, 7, cfg["vocab"])
        kt = kv.clone()
        lg = O.forward(W, cfg, kt, [0], [tokens], parents=[parents])[0]
        dep = T.depths(parents)
        for i in range(len(tokens)):
            path, r = [], i
            while r:
                path.append(r)
                r = parents[r - 1]
            path = [0] + path[::-1]
            kc = kv.clone()
            lc = O.forward(W, cfg, kc, [0], [tokens[path]])[0]
            assert torch.allclose(lg[i], lc[-1], rtol=0, atol=1e-9)
            assert dep[i] == len(path) - 1
            assert torch.equal(kt.k[:, 0, 11 + i], kc.k[:, 0, 11 + dep[i]])
            assert torch.equal(kt.v[:, 0, 11 + i], kc.v[:, 0, 11 + dep[i]])
    # a chain given as a tree is the chain
    tokens = rng.integers(0, cfg["vocab"], size=5).astype(np.int32)
    a = O.forward(W, cfg, kv.clone(), [0], [tokens])[0]
    b = O.forward(W, cfg, kv.clone(), [0], [tokens], parents=[[0, 1, 2, 3]])[0]
    assert torch.equal(a, b)


def test_tree_acceptance_is_the_best_branch():
    rng = np.random.default_rng(8)
    V = 12
    for trial in range(300):
        m = int(rng.integers(0, 9))
        tokens, parents = _random_tree(rng, m, V)
        logits = rng.normal(size=(m + 1, V)).astype(np.float32)
        for i in range(1, m + 1):                       # make many nodes pass
            if rng.random() < 0.6:
                logits[parents[i - 1], tokens[i]] = 5.0 + rng.random()
        mode = int(rng.integers(0, 4))
        a, em, path = T.accept_tree(logits, tokens, parents, m + 1, mode, 2, 0.2)
        # brute force: chain acceptance along every root-to-node path
        best = (0, [A.argmax_row(logits[0])], [])
        for i in range(1, m + 1):
            p, r = [], i
            while r:
                p.append(r)
                r = parents[r - 1]
            p = p[::-1]
            rows = [0] + p
            ca, cem = A.accept_one(logits[rows], tokens[rows], len(rows), mode, 2, 0.2)
            if ca == len(p) and ca > best[0]:           # the whole path verified, deeper than before
                best = (ca, cem, p)
        assert (a, em, path) == best
        assert len(em) == a + 1 and all(parents[path[j] - 1] == (path[j - 1] if j else 0) for j in range(a))
    # a chain given as a tree accepts what chain acceptance accepts
    for trial in range(100):
        m = int(rng.integers(0, 8))
        tokens = rng.integers(0, V, size=m + 1).astype(np.int32)
        logits = rng.normal(size=(m + 1, V)).astype(np.float32)
        for i in range(m):
            if rng.random() < 0.7:
                logits[i, tokens[i + 1]] = 6.0
        a, em, _ = T.accept_tree(logits, tokens, list(range(m)), m + 1, A.STRICT, 1, 0.0)
        assert (a, em) == A.accept_one(logits, tokens, m + 1, A.STRICT, 1, 0.0)


def test_tree_generation_is_lossless_and_no_slower_than_chain(model):
    """Strict verification of a token tree emits exactly the greedy text (Section 2.1), in no more
    steps than chain drafting on the same pool, and leaves the cache as the plain run does."""
    from oracle import generate as G
    cfg, W = model
    prompts = [synth.make_prompt(12, cfg["vocab"], 70 + b) for b in range(2)]
    plain = G.greedy(W, cfg, prompts, 24)
    rng = np.random.default_rng(2)
    docs = []
    for o in plain["out"]:                      # the pool: the text itself and corrupted variants
        for rep in range(3):
            d = list(o)
            for i in range(2 + rep, len(d), 5 + rep):
                d[i] = int(rng.integers(0, cfg["vocab"]))
            docs.append(d)
    pool, offs = synth.pool_from_documents([docs])
    kw = dict(K=6, n_min=1, n_max=3, max_new=24, max_occ=0)
    chain = G.generate(W, cfg, prompts, [0, 0], pool, offs, **kw)
    tree = G.generate(W, cfg, prompts, [0, 0], pool, offs, tree=True, **kw)
    assert tree["out"] == plain["out"] == chain["out"]
    assert tree["steps"] <= chain["steps"] and tree["accepted"] >= chain["accepted"]
    assert tree["accepted"] > 0 and (tree["ctx"] == plain["ctx"]).all()
