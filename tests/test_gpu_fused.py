"""Acceptance fused into the LM head (`laser_verify_accept`): the verdicts, emitted tokens and commits
equal the oracle's rule (Eq. 4, Eq. 7, Eq. 8, Section 4.3.2) applied to the logits that the same launch
stored on request, in every mode; without a logits buffer the outputs are the same.

Drafts are built so that the rule has something to decide: token i+1 of a sequence is taken from the
top of row i's distribution (rank 0, 1, 2 or further down), pass by pass, and rows of the LM head are
duplicated, so that equal logits occur inside a vocabulary tile, across tiles and at the top of a row
(ties rank the smaller id first).  The arg max and the rank test must agree exactly.  The probability
of a draft is combined from per-tile fp32 sums; a sequence is left out of the comparison of a
probability rule when one of its drafts has a probability within 1e-5 (relative) of the threshold."""
import numpy as np
import pytest
import torch

from helpers import dev_i32, ensure_built, weights_to
from oracle import accept as A
from paper_2408_05676_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def _plant_duplicates(W, rng, n_pairs):
    """Copies rows of the LM head over other rows: those tokens get bit-equal logits in every row."""
    V = W["lm_head"].shape[0]
    head = W["lm_head"].clone()
    for _ in range(n_pairs):
        a, b = (int(x) for x in rng.integers(0, V, 2))
        head[b] = head[a]
    # a pair inside one 128-token tile, a pair in neighbouring lanes, a triple across tiles
    head[5] = head[3]
    head[min(V - 1, 130)] = head[7]
    head[min(V - 1, 2 * 128 + 7)] = head[7]
    return dict(W, lm_head=head)


def _drafts_from_the_top(L, model, kv, seq_ids, B, K, passes, V, ctx, rng, n_rows):
    """tokens[b, i+1] from the top of row i's distribution given tokens[b, :i+1] (rank 0 mostly) for the first
    `passes` drafts, random tokens after them."""
    tokens = rng.integers(0, V, (B, K + 1)).astype(np.int32)
    d_n = dev_i32(n_rows)
    for i in range(passes):
        L.kv_set_len(kv, [int(s) for s in seq_ids.cpu()], ctx)
        fill = np.where(tokens < 0, 0, tokens).astype(np.int32)
        lg = L.verify_step(model, kv, seq_ids, dev_i32(fill), d_n)
        order = torch.argsort(lg[:, i].double(), dim=-1, descending=True, stable=True)[:, :8].cpu().numpy()
        pick = rng.choice([0, 0, 0, 0, 1, 1, 2, 3, 7], size=B)
        tokens[:, i + 1] = order[np.arange(B), pick]
    for b in range(B):
        tokens[b, max(int(n_rows[b]), 0):] = -1
    return tokens


CASES = [
    # vocabulary of 32 tiles: the LM head runs as K-split clusters; ragged rows and an inactive sequence
    ("tiny", dict(), 6, 4),
    # 15.6 tiles: the last vocabulary tile is ragged
    ("tiny", dict(n_layers=1, d_model=320, vocab=2000), 5, 5),
    # two token tiles (270 rows), short rows
    ("tiny", dict(max_draft=8), 30, 3),
    # 7B width, 250 vocabulary tiles, one CTA per tile
    ("7b", dict(n_layers=1), 16, 8),
    # 13B width with six token tiles: two vocabulary tiles per CTA
    ("13b", dict(n_layers=1, max_draft=16), 64, 16),
]


@pytest.mark.parametrize("name,over,B,K", CASES)
def test_fused_verdicts_equal_the_rule_on_the_stored_logits(L, name, over, B, K):
    cfg = synth.model_cfg(name, **dict(over, max_draft=K))
    V = cfg["vocab"]
    rng = np.random.default_rng(11 + B)
    big = name != "tiny"
    W = synth.make_weights(cfg, seed=0, device="cuda" if big else "cpu", gain_jitter=0.0 if big else 0.1)
    W = _plant_duplicates(W, rng, 40)
    model = L.model_create(cfg, W if big else weights_to(W, "cuda"), max_batch=B)
    kv = L.kv_create(model, B, B * 6)
    seq_ids = torch.arange(B, dtype=torch.int32, device="cuda")
    ctx = [int(x) for x in rng.integers(0, 40, B)]
    width = cfg["n_kv_heads"] * cfg["head_dim"]
    for l in range(cfg["n_layers"]):
        for b in range(B):
            if ctx[b]:
                k, v = synth.make_kv_layer(ctx[b], width, 3 + b, l, device="cuda")
                L.kv_import(kv, b, l, 0, k, v)
    n_rows = rng.integers(1, K + 2, B).astype(np.int32)
    n_rows[0] = K + 1
    if B > 2:
        n_rows[2] = 0                       # an inactive sequence
        n_rows[1] = 1                       # nothing to verify: one bonus token
    passes = K if not big else min(K, 4)    # the large shapes: drafts from the top for the first rows only
    tokens = _drafts_from_the_top(L, model, kv, seq_ids, B, K, passes, V, ctx, rng, n_rows)
    fill = np.where(tokens < 0, 0, tokens).astype(np.int32)
    d_tok, d_n = dev_i32(fill), dev_i32(n_rows)
    L.kv_set_len(kv, list(range(B)), ctx)
    plain = L.verify_step(model, kv, seq_ids, d_tok, d_n)
    L.check(model)
    # thresholds where the probability rule really decides: around the drafts' own probabilities
    plain_np = plain.cpu().numpy()
    probs = [A.prob_of(plain_np[b, i], int(fill[b, i + 1])) for b in range(B) for i in range(int(n_rows[b]) - 1)]
    p_mid = float(np.median(probs)) * 1.003 if probs else 0.1   # not on a draft's own probability
    modes = [(L.MODE_STRICT, 1, 0.0), (L.MODE_TOPK, 1, 0.0), (L.MODE_TOPK, 2, 0.0), (L.MODE_TOPK, 4, 0.0),
             (L.MODE_RELAXED, 2, p_mid), (L.MODE_RELAXED, 3, 1e-4), (L.MODE_TOPP, 1, p_mid), (L.MODE_RELAXED_ARGMAX, 2, p_mid)]
    decided = 0
    for mode, k, p in modes:
        prm = L.make_params(K=K, mode=mode, topk=k, p=p)
        stored = torch.full((B, K + 1, V), float("nan"), dtype=torch.float32, device="cuda")
        L.kv_set_len(kv, list(range(B)), ctx)
        got = [t.cpu().numpy() for t in L.verify_accept(model, kv, seq_ids, d_tok, d_n, prm, commit=True, logits=stored)]
        L.check(model)
        lens = L.kv_get_len(kv, list(range(B)))
        lg = stored.cpu().numpy()
        for b in range(B):                   # the stored logits are the plain call's, bit for bit
            nr = int(n_rows[b])
            assert (lg[b, :nr] == plain_np[b, :nr]).all()
        p32 = float(np.float32(p))
        ref = A.accept_batch(np.nan_to_num(lg, nan=0.0), fill, n_rows, mode, k, p32)
        skip = np.zeros(B, bool)
        if mode in (L.MODE_RELAXED, L.MODE_TOPP, L.MODE_RELAXED_ARGMAX):
            for b in range(B):
                for i in range(int(n_rows[b]) - 1):
                    q = A.prob_of(lg[b, i], int(fill[b, i + 1]))
                    skip[b] |= abs(q - p32) <= 1e-5 * p32
        assert skip.mean() <= 0.05
        keep = ~skip
        for g, w in zip(got, ref):
            assert (g[keep] == w[keep]).all(), (mode, k, p)
        assert (lens[keep] == np.asarray(ctx)[keep] + ref[2][keep]).all()
        decided += int(ref[0].sum())
        # without a logits buffer: the same outputs, nothing committed when not asked to
        L.kv_set_len(kv, list(range(B)), ctx)
        again = [t.cpu().numpy() for t in L.verify_accept(model, kv, seq_ids, d_tok, d_n, prm, commit=False)]
        L.check(model)
        for g, w in zip(again, got):
            assert (g == w).all()
        assert (L.kv_get_len(kv, list(range(B))) == np.asarray(ctx)).all()
        # and the two-kernel path on the plain call's logits
        two = [t.cpu().numpy() for t in L.accept_commit(None, None, plain, d_tok, d_n, prm)]
        for g, w in zip(two, got):
            assert (g[keep] == w[keep]).all()
    assert decided > 0                       # drafts were accepted somewhere: the rule had work to do


def test_rank_rules_beyond_four_are_refused(L):
    cfg = synth.model_cfg("tiny", n_layers=1)
    model = L.model_create(cfg, weights_to(synth.make_weights(cfg, 0), "cuda"), max_batch=2)
    kv = L.kv_create(model, 2, 8)
    ids = torch.arange(2, dtype=torch.int32, device="cuda")
    tok = dev_i32(np.ones((2, cfg["max_draft"] + 1)))
    with pytest.raises(L.LaserError) as e:
        L.verify_accept(model, kv, ids, tok, dev_i32([2, 2]), L.make_params(K=cfg["max_draft"], mode=L.MODE_TOPK, topk=5))
    assert e.value.status == -6          # UNSUPPORTED
    L.verify_accept(model, kv, ids, tok, dev_i32([2, 2]), L.make_params(K=cfg["max_draft"], mode=L.MODE_TOPP, topk=9, p=0.5))
    L.check(model)


def test_generation_with_fused_acceptance_is_the_same_text(L):
    cfg = synth.model_cfg("tiny")
    K, NEW, B = cfg["max_draft"], 48, 6
    model = L.model_create(cfg, weights_to(synth.make_weights(cfg, 0), "cuda"), max_batch=B)
    kv = L.kv_create(model, B, B * 16)
    prompts = [synth.make_prompt(20 + 7 * b, cfg["vocab"], 50 + b) for b in range(B)]
    greedy = L.generate(model, kv, None, prompts, [0] * B, L.make_params(K=K, max_new=NEW))["out"]
    docs = np.concatenate([np.asarray([synth.SENTINEL] + g, np.int32) for g in greedy])
    pool = L.pool_build(docs, np.asarray([0, len(docs)], np.int64), 1, 4)
    for fused in (0, 1):
        r = L.generate(model, kv, pool, prompts, [0] * B, L.make_params(K=K, max_new=NEW, fused_accept=fused))
        assert r["out"] == greedy
        assert r["accepted"] > 0
    r = L.generate(model, kv, None, prompts, [0] * B, L.make_params(K=K, max_new=NEW, fused_accept=1))
    assert r["out"] == greedy
