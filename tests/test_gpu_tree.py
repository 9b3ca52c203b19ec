"""Tree-based drafting on the GPU (Section 3.3): tree attention in the verify forward, tree
verification with cache compaction, tree retrieval and the tree mode of the generation loop,
each against the tree oracle."""
import os

import numpy as np
import pytest
import torch

from helpers import dev_i32, ensure_built, weights_to
from oracle import accept as A
from oracle import forward as O
from oracle import tree as T
from paper_2408_05676_b200 import synth
from test_gpu_forward import TOL, _fill_both

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def random_tree(rng, m):
    """Parents (rows of [root] + nodes) of a random tree with m nodes, in depth-first order."""
    raw = [int(rng.integers(0, i + 1)) for i in range(m)]
    kids = {}
    for i, p in enumerate(raw):
        kids.setdefault(p, []).append(i + 1)
    par = []
    def visit(row, new_row):
        for k in kids.get(row, []):
            par.append(new_row)
            visit(k, len(par))
    visit(0, 0)
    return par


@pytest.mark.parametrize("over,B,ctx", [
    (dict(), 5, [150, 0, 37, 16, 5]),                                                     # TMA attention, dh 64
    (dict(n_layers=2, d_model=512, n_heads=4, n_kv_heads=4, head_dim=128, d_ffn=688, vocab=4096), 3, [130, 15, 1]),
    (dict(n_layers=2, d_model=256, n_heads=8, n_kv_heads=2, head_dim=32, d_ffn=256, vocab=1000, max_draft=5), 4, [9, 33, 0, 17]),  # plain attention kernel
])
def test_tree_forward_matches_oracle(L, over, B, ctx):
    cfg = synth.model_cfg("tiny", **over)
    Wc = synth.make_weights(cfg, seed=0, gain_jitter=0.1)
    m = L.model_create(cfg, weights_to(Wc, "cuda"), max_batch=B)
    pages_per_seq = 12
    kv = L.kv_create(m, B, B * pages_per_seq)
    rng = np.random.default_rng(4)
    L.kv_set_page_table(kv, rng.permutation(B * pages_per_seq).astype(np.int32))
    okv = O.KVCache(cfg, B, pages_per_seq * 16)
    seq_ids = list(rng.permutation(B))
    _fill_both(L, cfg, kv, okv, seq_ids, ctx, seed=9)
    Rs = cfg["max_draft"] + 1
    for step in range(2):
        tokens = np.full((B, Rs), -1, np.int32)
        parents = np.full((B, Rs), -1, np.int32)
        n_rows = np.zeros(B, np.int32)
        rows, pars = [], []
        for b in range(B):
            nr = Rs if b == 0 else int(rng.integers(1, Rs + 1))
            if step == 1 and b == 1:
                nr = 0                                                   # an inactive sequence
            par = random_tree(rng, max(nr - 1, 0)) if b != 2 else list(range(max(nr - 1, 0)))   # b = 2: a chain
            r = synth.make_prompt(nr, cfg["vocab"], 50 * step + b) if nr else np.zeros(0, np.int32)
            tokens[b, :nr] = r
            parents[b, 1:nr] = par
            n_rows[b] = nr
            rows.append(r)
            pars.append(par)
        logits = L.verify_step_tree(m, kv, dev_i32(seq_ids), dev_i32(tokens), dev_i32(parents), dev_i32(n_rows))
        L.check(m)
        act = [b for b in range(B) if n_rows[b] > 0]
        want = O.forward(Wc, cfg, okv, [seq_ids[b] for b in act], [rows[b] for b in act], parents=[pars[b] for b in act])
        got = logits.cpu().double()
        err = max(float((got[b, :n_rows[b]] - w).abs().max()) for b, w in zip(act, want))
        print("step", step, "max-abs logit error", err)
        assert err <= TOL
        for b in act:                     # K and V of row i sit in slot ctx + i on both sides
            s, c, n = seq_ids[b], int(okv.ctx[seq_ids[b]]), int(n_rows[b])
            for l in (0, cfg["n_layers"] - 1):
                k, v = L.kv_export(kv, s, l, c, n)
                wk = okv.k[l, s, c:c + n].reshape(n, -1).float()
                wv = okv.v[l, s, c:c + n].reshape(n, -1).float()
                assert (k.cpu().float() - wk).abs().max() <= 2.0 ** -7 * max(1.0, float(wk.abs().max()))
                assert (v.cpu().float() - wv).abs().max() <= 2.0 ** -7 * max(1.0, float(wv.abs().max()))
        # a chain given as a tree is bit-identical to the chain entry point
        if step == 0:
            chain = np.tile(np.arange(-1, Rs - 1, dtype=np.int32), (B, 1))
            a = L.verify_step_tree(m, kv, dev_i32(seq_ids), dev_i32(tokens), dev_i32(chain), dev_i32(n_rows)).clone()
            b_ = L.verify_step(m, kv, dev_i32(seq_ids), dev_i32(tokens), dev_i32(n_rows))
            assert torch.equal(a, b_)


def test_bad_parent_is_reported(L):
    cfg = synth.model_cfg("tiny")
    m = L.model_create(cfg, weights_to(synth.make_weights(cfg, seed=0), "cuda"), max_batch=1)
    kv = L.kv_create(m, 1, 8)
    Rs = cfg["max_draft"] + 1
    tokens = np.zeros((1, Rs), np.int32)
    parents = np.tile(np.arange(-1, Rs - 1, dtype=np.int32), (1, 1))
    parents[0, 3] = 3                       # a row cannot be its own parent
    L.verify_step_tree(m, kv, dev_i32([0]), dev_i32(tokens), dev_i32(parents), dev_i32([Rs]))
    with pytest.raises(L.LaserError):
        L.check(m)
