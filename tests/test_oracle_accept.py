"""Pins for the acceptance oracle: hand examples and closed forms of Eq. 4 / Eq. 8."""
import os

import numpy as np
import pytest

from oracle import accept as A
from paper_2408_05676_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "accept_hand_examples.txt")
MODES = dict(STRICT=A.STRICT, RELAXED=A.RELAXED, TOPK=A.TOPK, TOPP=A.TOPP, RELAXED_ARGMAX=A.RELAXED_ARGMAX)


def _cases():
    cases, cur = [], None
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("case"):
            f = dict(kv.split("=") for kv in line.split()[1:])
            cur = dict(V=int(f["V"]), tokens=[int(x) for x in f["tokens"].split(",")], rows=[])
        elif line.startswith("row"):
            cur["rows"].append([float(x) for x in line[3:].split(",")])
        else:
            lhs, rhs = line[len("expect"):].split("->")
            mode, k, p = lhs.split()
            a, em = rhs.split("|")
            cases.append((cur, MODES[mode], int(k), float(p), int(a), [int(x) for x in em.split(",")]))
    return cases


@pytest.mark.parametrize("case", _cases())
def test_hand_examples(case):
    cur, mode, k, p, want_a, want_em = case
    logits = np.asarray(cur["rows"], dtype=np.float32)
    assert logits.shape[1] == cur["V"]
    a, em = A.accept_one(logits, np.asarray(cur["tokens"]), len(cur["tokens"]), mode, k, p)
    assert (a, em) == (want_a, want_em)


def test_hand_probabilities():
    assert abs(A.prob_of(np.float32([0, 1, 3, 2]), 2) - 0.6439) < 5e-5
    assert abs(A.prob_of(np.float32([2, 1.5, 0, 0]), 1) - 0.3231) < 5e-5
    row = np.zeros(16, np.float32); row[5] = 0.1
    assert abs(A.prob_of(row, 5) - 0.0686) < 5e-5
    rng = np.random.default_rng(0)
    r = rng.standard_normal(1000).astype(np.float32) * 5
    assert abs(sum(A.prob_of(r, t) for t in range(1000)) - 1.0) < 1e-12
    assert sorted(A.rank_of(r, t) for t in range(1000)) == list(range(1000))


def test_closed_forms():
    logits, tokens, n_rows = synth.make_accept_case(24, 8, 257, seed=3)
    s = A.accept_batch(logits, tokens, n_rows, A.STRICT)
    # RELAXED with k=1, p=0 is STRICT (every probability is > 0)
    r = A.accept_batch(logits, tokens, n_rows, A.RELAXED, 1, 0.0)
    for x, y in zip(s, r):
        assert (x == y).all()
    # p >= 1 accepts nothing; the emitted token is then the arg-max of row 0
    z = A.accept_batch(logits, tokens, n_rows, A.RELAXED, 2, 1.0)
    assert (z[0] == 0).all() and (z[2] == 1).all()
    assert (z[1][:, 0] == logits[:, 0].argmax(-1)).all()
    # TOPK accepts at least what RELAXED accepts; TOPP at least what STRICT accepts
    rv = A.accept_batch(logits, tokens, n_rows, A.RELAXED, 2, 0.1)
    tk = A.accept_batch(logits, tokens, n_rows, A.TOPK, 2, 0.1)
    tp = A.accept_batch(logits, tokens, n_rows, A.TOPP, 2, 0.1)
    assert (tk[0] >= rv[0]).all() and (tp[0] >= s[0]).all()
    assert (rv[0] != s[0]).any() and (tk[0] != rv[0]).any()
    # RELAXED_ARGMAX passes a token exactly when STRICT or RELAXED does, row by row, so its prefix is at
    # least as long as either; with k = 1 it is STRICT (the only top-1 token is the arg-max), and it is
    # inside TOPP (arg-max or > p, without the top-k condition)
    ra = A.accept_batch(logits, tokens, n_rows, A.RELAXED_ARGMAX, 2, 0.1)
    assert (ra[0] >= np.maximum(s[0], rv[0])).all() and (ra[0] <= tp[0]).all()
    for b in range(len(n_rows)):
        for i in range(int(n_rows[b]) - 1):
            t = int(tokens[b, i + 1])
            assert A.passes(logits[b, i], t, A.RELAXED_ARGMAX, 2, 0.1) == (
                A.passes(logits[b, i], t, A.STRICT, 2, 0.1) or A.passes(logits[b, i], t, A.RELAXED, 2, 0.1))
    r1 = A.accept_batch(logits, tokens, n_rows, A.RELAXED_ARGMAX, 1, 0.1)
    for x, y in zip(s, r1):
        assert (x == y).all()
    for n_acc, out, n_out in (s, rv, tk, tp, ra):
        assert (n_out == n_acc + 1).all() and (n_acc <= n_rows - 1).all()
        for b in range(len(n_rows)):
            a = n_acc[b]
            assert (out[b, :a] == tokens[b, 1:1 + a]).all()
            assert out[b, a] == logits[b, a].argmax()
            assert (out[b, a + 1:] == -1).all()


def test_relaxed_dominates_strict_when_argmax_clears_threshold():
    rng = np.random.default_rng(9)
    logits = rng.standard_normal((16, 6, 50)).astype(np.float32)
    logits[np.arange(16)[:, None], np.arange(6)[None, :], rng.integers(0, 50, (16, 6))] += 6.0
    tokens = rng.integers(0, 50, (16, 6)).astype(np.int32)
    tokens[:, 1:] = np.where(rng.random((16, 5)) < 0.7, logits[:, :5].argmax(-1), tokens[:, 1:])
    n_rows = np.full(16, 6, np.int32)
    for b in range(16):
        for i in range(6):
            assert A.prob_of(logits[b, i], int(logits[b, i].argmax())) > 0.1
    s = A.accept_batch(logits, tokens, n_rows, A.STRICT)
    r = A.accept_batch(logits, tokens, n_rows, A.RELAXED, 2, 0.1)
    assert (r[0] >= s[0]).all()


def test_inactive_sequence():
    logits, tokens, n_rows = synth.make_accept_case(4, 3, 33, seed=1)
    n_rows[2] = 0
    n_acc, out, n_out = A.accept_batch(logits, tokens, n_rows, A.STRICT)
    assert n_acc[2] == 0 and n_out[2] == 0 and (out[2] == -1).all()


def test_probability_from_per_tile_sums_agrees_with_the_two_pass_rule():
    """The fused acceptance (laser_verify_accept) cannot know a row's max before its first exponential: it sums
    exp(l - tile max) per 128-token tile in fp32 and combines the tiles in fp64 with exp(tile max - row max).
    Written out here in numpy, that decomposition agrees with the oracle's two-pass probability to a few 1e-6
    relative (the oracle's own fp32 rounding of l - max is the larger part of it for logits far below the
    max) - inside the 1e-5 margin the parity test of the fused path leaves around the threshold p."""
    rng = np.random.default_rng(12)
    worst = 0.0
    for V, scale in ((32000, 1.3), (32000, 6.0), (2000, 1.0), (4096, 12.0)):
        for _ in range(8):
            row = (rng.standard_normal(V) * scale).astype(np.float32)
            t = int(rng.integers(0, V))
            tiles = [row[i:i + 128] for i in range(0, V, 128)]
            tmax = np.asarray([x.max() for x in tiles], np.float32)
            tsum = np.asarray([np.exp((x - m).astype(np.float32)).astype(np.float32).sum(dtype=np.float32)
                               for x, m in zip(tiles, tmax)], np.float32)
            M = tmax.max()
            denom = float((tsum.astype(np.float64) * np.exp(tmax.astype(np.float64) - float(M))).sum())
            fused = float(np.exp(float(row[t]) - float(M))) / denom
            want = A.prob_of(row, t)
            worst = max(worst, abs(fused - want) / want)
    assert worst <= 5e-6, worst

