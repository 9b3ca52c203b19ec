"""Pins for the generation-loop oracle: the lossless property of strict verification
(Section 2.1: greedy verification keeps the output identical to autoregressive decoding),
degenerate relaxed verification, and token conservation."""
import numpy as np

from oracle import accept as A
from oracle import generate as G
from paper_2408_05676_b200 import synth

CFG = synth.model_cfg("tiny", n_layers=2, d_model=64, n_heads=4, n_kv_heads=4, head_dim=16,
                      d_ffn=96, vocab=96)


def _setup(std=0.6):
    W = synth.make_weights(CFG, seed=21, std=std, gain_jitter=0.2)
    prompts = [synth.make_prompt(10 + 3 * b, CFG["vocab"], 300 + b) for b in range(3)]
    others = [synth.make_prompt(12, CFG["vocab"], 400 + b) for b in range(6)]
    docs = G.greedy(W, CFG, others, 40)["out"]
    # corrupt some documents so drafts are sometimes wrong
    rng = np.random.default_rng(0)
    for d in docs[::2]:
        for i in range(5, len(d), 7):
            d[i] = int(rng.integers(0, CFG["vocab"]))
    pool, offs = synth.pool_from_documents([docs[:3], docs[3:]])
    return W, prompts, pool, offs


def test_strict_speculative_equals_plain_greedy():
    W, prompts, pool, offs = _setup()
    want = G.greedy(W, CFG, prompts, 48)
    assert want["steps"] == 3 * 48 and want["accepted"] == 0
    for K, max_occ, gid in ((4, 0, [0, 1, 0]), (8, 2, [1, 1, 0])):
        got = G.generate(W, CFG, prompts, gid, pool, offs, K=K, n_min=1, n_max=3, max_new=48,
                         max_occ=max_occ)
        assert got["out"] == want["out"]
        assert got["emitted"] == 3 * 48
        assert got["steps"] < want["steps"] and got["accepted"] > 0
        for b in range(3):
            assert got["ctx"][b] == len(prompts[b]) - 1 + 48


def test_self_pool_accepts_everything():
    W, prompts, _, _ = _setup()
    want = G.greedy(W, CFG, prompts, 40)
    pool, offs = synth.pool_from_documents([[list(p) + o] for p, o in zip(prompts, want["out"])])
    got = G.generate(W, CFG, prompts, [0, 1, 2], pool, offs, K=7, n_min=1, n_max=4, max_new=40,
                     min_draft=1)
    assert got["out"] == want["out"]
    for b in range(3):                       # a draft that matches the future is accepted whole
        at, hits = 0, 0
        for draft, a, em in got["trace"][b]:
            future = want["out"][b][at:at + len(draft)]
            if draft and draft == future:
                assert a == len(draft)
                hits += 1
            at += len(em)
        assert hits > 0


def test_relaxed_below_threshold_is_plain_greedy():
    # tiny logits -> max probability ~ 1/V << p: literal Eq. 8 accepts nothing
    W, prompts, pool, offs = _setup(std=0.02)
    want = G.greedy(W, CFG, prompts, 24)
    got = G.generate(W, CFG, prompts, [0, 1, 0], pool, offs, K=4, n_min=1, n_max=3, max_new=24,
                     mode=A.RELAXED, topk=2, p=0.1)
    assert got["out"] == want["out"] and got["accepted"] == 0 and got["steps"] == 3 * 24


def test_relaxed_accepts_more_and_conserves_tokens():
    W, prompts, pool, offs = _setup()
    s = G.generate(W, CFG, prompts, [0, 1, 0], pool, offs, K=6, n_min=1, n_max=3, max_new=40)
    r = G.generate(W, CFG, prompts, [0, 1, 0], pool, offs, K=6, n_min=1, n_max=3, max_new=40,
                   mode=A.TOPK, topk=3, p=0.0)
    for res in (s, r):
        assert res["emitted"] == sum(len(o) for o in res["out"]) == 3 * 40
        for b in range(3):
            assert sum(len(em) for _, _, em in res["trace"][b]) == 40
            for draft, a, em in res["trace"][b]:
                assert em[:a] == draft[:a][:len(em)] and len(em) <= a + 1
    assert r["steps"] <= s["steps"]


def test_eos_stops_generation():
    W, prompts, pool, offs = _setup()
    full = G.greedy(W, CFG, prompts, 30)["out"]
    eos = full[0][9]
    got = G.generate(W, CFG, prompts, [0, 1, 0], pool, offs, K=4, n_min=1, n_max=3, max_new=30, eos_id=eos)
    for b in range(3):
        want = full[b][:full[b].index(eos) + 1] if eos in full[b] else full[b]
        assert got["out"][b] == want
