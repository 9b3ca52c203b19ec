"""laser_verify_step against the forward oracle: logits within 2e-2 max-abs (bf16 operands,
fp32 accumulation, against fp64), K/V written to the pages as the oracle caches them, with a
shuffled page table, ragged row counts, inactive sequences and multi-step continuation."""
import numpy as np
import pytest
import torch

from helpers import dev_i32, ensure_built, weights_to
from oracle import forward as O
from paper_2408_05676_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2   # max-abs logit error allowed for the bf16 / fp32-accumulate path


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def _fill_both(L, cfg, kv, okv, seqs, ctx, seed):
    """Same synthetic N(0,1) bf16 cache contents on both sides."""
    w = cfg["n_kv_heads"] * cfg["head_dim"]
    for l in range(cfg["n_layers"]):
        for s, c in zip(seqs, ctx):
            if c == 0:
                continue
            k, v = synth.make_kv_layer(c, w, seed + 17 * s, l)
            okv.k[l, s, :c] = k.view(c, cfg["n_kv_heads"], cfg["head_dim"])
            okv.v[l, s, :c] = v.view(c, cfg["n_kv_heads"], cfg["head_dim"])
            L.kv_import(kv, s, l, 0, k.cuda(), v.cuda())
    for s, c in zip(seqs, ctx):
        okv.ctx[s] = c
    L.kv_set_len(kv, list(seqs), list(ctx))


def _step(L, m, kv, cfg, W, okv, seq_ids, rows):
    """One verify step on both sides; returns max-abs logit error over the active rows."""
    Rs = cfg["max_draft"] + 1
    B = len(seq_ids)
    tokens = np.full((B, Rs), -1, np.int32)
    n_rows = np.zeros(B, np.int32)
    for b, r in enumerate(rows):
        tokens[b, :len(r)] = r
        n_rows[b] = len(r)
    logits = L.verify_step(m, kv, dev_i32(seq_ids), dev_i32(tokens), dev_i32(n_rows))
    L.check(m)
    act = [b for b in range(B) if n_rows[b] > 0]
    want = O.forward(W, cfg, okv, [seq_ids[b] for b in act], [rows[b] for b in act])
    err = 0.0
    got = logits.cpu().double()
    for b, w in zip(act, want):
        err = max(err, float((got[b, :n_rows[b]] - w).abs().max()))
    return err, logits


def _check_new_kv(L, kv, okv, cfg, seq, n_new):
    c = int(okv.ctx[seq])
    for l in sorted(x for x in {0, cfg["n_layers"] - 1} if 0 <= x < cfg["n_layers"]):
        k, v = L.kv_export(kv, seq, l, c, n_new)
        wk = okv.k[l, seq, c:c + n_new].reshape(n_new, -1).float()
        wv = okv.v[l, seq, c:c + n_new].reshape(n_new, -1).float()
        # bf16 values computed from bf16-rounded activations: a few rounding steps apart at most
        assert (k.cpu().float() - wk).abs().max() <= 2.0 ** -7 * max(1.0, float(wk.abs().max()))
        assert (v.cpu().float() - wv).abs().max() <= 2.0 ** -7 * max(1.0, float(wv.abs().max()))
        assert (k.cpu().float() - wk).abs().mean() <= 2.0 ** -9 * max(1.0, float(wk.abs().max()))


@pytest.mark.parametrize("name,over,B,ctx", [
    ("tiny", dict(n_layers=0, d_model=320, vocab=2000), 2, [0, 0]),     # embedding -> norm -> LM head only
    ("tiny", dict(), 4, [150, 0, 170, 5]),
    ("tiny", dict(n_layers=3, d_model=512, n_heads=4, n_kv_heads=4, head_dim=128, d_ffn=1376, vocab=8192), 3, [130, 16, 1]),
    ("tiny", dict(n_layers=2, d_model=256, n_heads=8, n_kv_heads=2, head_dim=32, d_ffn=256, vocab=1000, max_draft=3), 5, [9, 33, 2, 0, 17]),
    # 30 sequences x 9 rows = 270 rows: two token tiles in every GEMM, the second one overhanging
    ("tiny", dict(), 30, [int(x) for x in np.random.default_rng(3).integers(0, 150, 30)]),
])
def test_logits_and_cache_match_oracle(L, name, over, B, ctx):
    cfg = synth.model_cfg(name, **over)
    Wc = synth.make_weights(cfg, seed=0, gain_jitter=0.1)
    m = L.model_create(cfg, weights_to(Wc, "cuda"), max_batch=B + 1)
    pages_per_seq = 12
    kv = L.kv_create(m, B + 2, (B + 2) * pages_per_seq)
    rng = np.random.default_rng(0)
    L.kv_set_page_table(kv, rng.permutation((B + 2) * pages_per_seq).astype(np.int32))
    okv = O.KVCache(cfg, B + 2, pages_per_seq * 16)
    seq_ids = list(rng.permutation(B + 2)[:B])
    _fill_both(L, cfg, kv, okv, seq_ids, ctx, seed=7)
    Rs = cfg["max_draft"] + 1
    worst = 0.0
    for step in range(3):
        rows = [synth.make_prompt(int(rng.integers(1, Rs + 1)), cfg["vocab"], 100 * step + b) for b in range(B)]
        if step == 1:
            rows[1] = rows[1][:0]          # an inactive sequence
            rows[0] = synth.make_prompt(Rs, cfg["vocab"], 999)
        err, _ = _step(L, m, kv, cfg, Wc, okv, seq_ids, rows)
        print("step", step, "max-abs logit error", err)
        worst = max(worst, err)
        for b in range(B):
            if len(rows[b]):
                _check_new_kv(L, kv, okv, cfg, seq_ids[b], len(rows[b]))
            keep = int(rng.integers(1, len(rows[b]) + 1)) if len(rows[b]) else 0   # commit a prefix
            okv.ctx[seq_ids[b]] += keep
        L.kv_set_len(kv, seq_ids, [int(okv.ctx[s]) for s in seq_ids])
    print("max-abs logit error", worst)
    assert worst <= TOL


def test_capacity_error_is_reported_not_faulted(L):
    cfg = synth.model_cfg("tiny", n_layers=1)
    m = L.model_create(cfg, weights_to(synth.make_weights(cfg, 0), "cuda"), max_batch=2)
    kv = L.kv_create(m, 2, 4)            # 2 pages = 32 tokens per sequence
    L.kv_set_len(kv, [0, 1], [30, 3])
    tokens = np.zeros((2, 9), np.int32)
    logits = L.verify_step(m, kv, dev_i32([0, 1]), dev_i32(tokens), dev_i32([9, 9]))
    with pytest.raises(L.LaserError) as e:
        L.check(m)
    assert e.value.status == -4
    L.check(m)                            # cleared
    assert torch.isfinite(logits[1]).all()
    with pytest.raises(L.LaserError):
        L.verify_step(m, kv, dev_i32([0, 1, 1]), dev_i32(np.zeros((3, 9))), dev_i32([1, 1, 1]))
