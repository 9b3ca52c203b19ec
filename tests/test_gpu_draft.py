"""laser_pool_build + laser_draft against the retrieval oracle: bit-exact drafts, lengths and
matched suffix lengths on hand examples, collision-heavy tiny vocabularies, ragged groups,
capped and unlimited occurrence lists, and a Zipf/template pool of the benchmark's recipe."""
import os

import numpy as np
import pytest
import torch

from helpers import dev_i32, ensure_built
from oracle import retrieval as R
from paper_2408_05676_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def _compare(L, pool_np, offs, tails, tail_len, gid, K, n_min, n_max, min_draft, max_occ, pool=None):
    own = pool is None
    if own:
        pool = L.pool_build(pool_np, offs, n_min, n_max)
    prm = L.make_params(K=K, n_min=n_min, n_max=n_max, min_draft=min_draft, max_occ=max_occ)
    d, dl, mn = L.draft(pool, dev_i32(tails), dev_i32(tail_len), dev_i32(gid), prm)
    torch.cuda.synchronize()
    wd, wl, wn = R.draft_batch(pool_np, offs, tails, tail_len, gid, K, n_min, n_max, min_draft, max_occ)
    assert (dl.cpu().numpy() == wl).all()
    assert (mn.cpu().numpy() == wn).all()
    assert (d.cpu().numpy() == wd).all()
    if own:
        pool.free()
    return wl


def test_hand_examples(L):
    gold = os.path.join(os.path.dirname(__file__), "golden", "retrieval_hand_examples.txt")
    for line in open(gold):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        ints = lambda s: [int(x) for x in s.split(",")] if s else []
        pool, tail = np.asarray(ints(f[0]), np.int32), ints(f[1])
        K, n_min, n_max, min_draft, max_occ = map(int, f[2:7])
        tails = np.full((1, n_max), -1, np.int32)
        t = tail[-n_max:]
        tails[0, n_max - len(t):] = t
        _compare(L, pool, np.asarray([0, len(pool)], np.int64), tails, np.asarray([len(t)], np.int32),
                 np.zeros(1, np.int32), K, n_min, n_max, min_draft, max_occ)


@pytest.mark.parametrize("vocab,max_occ,seed", [(3, 0, 1), (5, 0, 2), (4, 3, 3), (6, 64, 4), (3, 100, 5), (50, 0, 6)])
def test_random_small_pools(L, vocab, max_occ, seed):
    rng = np.random.default_rng(seed)
    G = 5
    toks, offs = [], [0]
    for g in range(G):
        ln = int(rng.integers(0 if g == 2 else 1, 1500))
        x = rng.integers(0, vocab, size=ln)
        x[rng.random(ln) < 0.03] = -1
        toks.extend(x.tolist())
        offs.append(len(toks))
    pool, offs = np.asarray(toks, np.int32), np.asarray(offs, np.int64)
    Q, n_max = 300, 4
    tails = rng.integers(0, vocab, size=(Q, n_max)).astype(np.int32)
    tail_len = rng.integers(0, n_max + 1, size=Q).astype(np.int32)
    for q in range(Q):
        tails[q, :n_max - tail_len[q]] = -1
    gid = rng.integers(0, G, size=Q).astype(np.int32)
    for K, n_min, min_draft in ((8, 1, 1), (16, 2, 4), (1, 1, 1), (64, 1, 70)):
        lens = _compare(L, pool, offs, tails, tail_len, gid, K, n_min, n_max, min_draft, max_occ)
    assert lens.max() > 0


def test_zipf_template_pool(L):
    pool, offs = synth.make_zipf_pool(2_000_000, 400, vocab=32000, seed=42)
    tails, tail_len, gid = synth.make_queries(pool, offs, 512, n_tail=4, seed=44)
    h = L.pool_build(pool, offs, 1, 4)
    info = h.info()
    assert info["n_tokens"] == len(pool) and info["n_keys"] > len(pool)
    hit = 0
    for max_occ in (64, 0, 1):
        lens = _compare(L, pool, offs, tails, tail_len, gid, 16, 1, 4, 1, max_occ, pool=h)
        hit += int((lens > 0).sum())
    assert hit > 512
    # device-resident token array as the build input gives the same index
    h2 = L.pool_build(torch.as_tensor(pool, device="cuda"), offs, 1, 4)
    _compare(L, pool, offs, np.ascontiguousarray(tails[:, 1:]), np.minimum(tail_len, 3), gid, 16, 2, 3, 1, 64, pool=h2)


def test_make_rows(L):
    last = dev_i32([5, -1, 9])
    draft = dev_i32([[1, 2, 3], [4, 5, 6], [7, -1, -1]])
    dl = dev_i32([3, 2, 1])
    tokens, n_rows = L.make_rows(last, draft, dl, 3)
    assert tokens.cpu().tolist() == [[5, 1, 2, 3], [-1, -1, -1, -1], [9, 7, -1, -1]]
    assert n_rows.cpu().tolist() == [4, 0, 2]


def test_rejects_bad_arguments(L):
    pool = np.arange(10, dtype=np.int32)
    with pytest.raises(L.LaserError):
        L.pool_build(pool, np.asarray([0, 5], np.int64), 1, 4)       # offsets do not span the pool
    with pytest.raises(L.LaserError):
        L.pool_build(pool, np.asarray([0, 10], np.int64), 1, 9)      # n_max above the limit
    h = L.pool_build(pool, np.asarray([0, 10], np.int64), 2, 3)
    t = dev_i32(np.zeros((1, 4)))
    with pytest.raises(L.LaserError):
        L.draft(h, t, dev_i32([4]), dev_i32([0]), L.make_params(K=4, n_min=1, n_max=4))


# ---- temporary branches: laser_draft_temp against the oracle with `history` ------------------
def _compare_temp(L, pool, pool_np, offs, tails, tail_len, gid, hists, K, n_min, n_max, min_draft, max_occ):
    B = len(tail_len)
    stride = max(1, max(len(h) for h in hists))
    hist = np.zeros((B, stride), np.int32)
    hl = np.zeros(B, np.int32)
    for b, h in enumerate(hists):
        hist[b, :len(h)] = h
        hl[b] = len(h)
    prm = L.make_params(K=K, n_min=n_min, n_max=n_max, min_draft=min_draft, max_occ=max_occ)
    d, dl, mn = L.draft_temp(pool, dev_i32(tails), dev_i32(tail_len), dev_i32(gid), dev_i32(hist), dev_i32(hl), prm)
    torch.cuda.synchronize()
    wd, wl, wn = R.draft_batch(pool_np, offs, tails, tail_len, gid, K, n_min, n_max, min_draft, max_occ,
                               histories=hists)
    assert (dl.cpu().numpy() == wl).all()
    assert (mn.cpu().numpy() == wn).all()
    assert (d.cpu().numpy() == wd).all()
    return wl


def test_temp_hand_examples(L):
    gold = os.path.join(os.path.dirname(__file__), "golden", "retrieval_temp_hand_examples.txt")
    ints = lambda s: [int(x) for x in s.split(",")] if s else []
    for line in open(gold):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        pool_np, hist, tail = np.asarray(ints(f[0]), np.int32), np.asarray(ints(f[1]), np.int32), ints(f[2])
        K, n_min, n_max, min_draft, max_occ = map(int, f[3:8])
        max_occ = max_occ or 64              # the kernel keeps 1..64 occurrences; the examples have fewer
        tails = np.full((1, n_max), -1, np.int32)
        t = tail[-n_max:]
        tails[0, n_max - len(t):] = t
        offs = np.asarray([0, len(pool_np)], np.int64)
        pool = L.pool_build(pool_np, offs, n_min, n_max)
        wl = _compare_temp(L, pool, pool_np, offs, tails, np.asarray([len(t)], np.int32), np.zeros(1, np.int32),
                           [hist], K, n_min, n_max, min_draft, max_occ)
        assert wl[0] == len(ints(f[8]))
        pool.free()


@pytest.mark.parametrize("vocab,max_occ,seed", [(3, 64, 11), (4, 3, 12), (6, 1, 13), (40, 64, 14)])
def test_temp_random(L, vocab, max_occ, seed):
    """Histories of ragged lengths (empty, shorter than the tail, longer than a warp's sweep) that end
    with the tail, tiny vocabularies so that history and pool both match, capped lists."""
    rng = np.random.default_rng(seed)
    G = 4
    toks, offs = [], [0]
    for g in range(G):
        ln = int(rng.integers(1, 900))
        t = rng.integers(0, vocab, size=ln)
        t[rng.random(ln) < 0.05] = -1
        toks.extend(t.tolist())
        offs.append(len(toks))
    pool_np, offs = np.asarray(toks, np.int32), np.asarray(offs, np.int64)
    n_min, n_max, K = 1, 4, 8
    pool = L.pool_build(pool_np, offs, n_min, n_max)
    B = 150
    hists, tails, tl = [], np.full((B, n_max), -1, np.int32), np.zeros(B, np.int32)
    for b in range(B):
        hl = int(rng.choice([0, 1, 2, 3, 7, 33, 64, 65, 200, 700]))
        h = rng.integers(0, vocab, size=hl).astype(np.int32)
        if hl >= 12 and rng.random() < 0.6:      # plant a repeat so the history itself matches
            h[-4:] = h[hl // 2 - 4:hl // 2]
        hists.append(h)
        if rng.random() < 0.8 and hl > 0:
            t = h[-n_max:]
        else:                                     # a tail that is not the end of the history
            t = rng.integers(0, vocab, size=int(rng.integers(0, n_max + 1))).astype(np.int32)
        tails[b, n_max - len(t):] = t
        tl[b] = len(t)
    gid = rng.integers(0, G, size=B).astype(np.int32)
    gid[::17] = -1                                # no group: the history alone
    for min_draft in (1, 4):
        wl = _compare_temp(L, pool, pool_np, offs, tails, tl, gid, hists, K, n_min, n_max, min_draft, max_occ)
    assert (wl > 0).mean() > 0.3
    pool.free()


def test_temp_rejects_uncapped(L):
    pool_np, offs = np.asarray([1, 2, 3], np.int32), np.asarray([0, 3], np.int64)
    pool = L.pool_build(pool_np, offs, 1, 2)
    z = dev_i32(np.zeros((1, 2), np.int32))
    one = dev_i32(np.zeros(1, np.int32))
    with pytest.raises(L.LaserError):
        L.draft_temp(pool, z, one, one, z, one, L.make_params(K=4, n_min=1, n_max=2, max_occ=0))
    pool.free()
