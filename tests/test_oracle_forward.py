"""Pins for the forward oracle: an independently composed full-sequence forward built
from library routines, and special cases with textbook answers."""
import math

import numpy as np
import torch
import torch.nn.functional as F

from oracle import forward as O
from paper_2408_05676_b200 import synth

CFG = synth.model_cfg("tiny", n_layers=2, d_model=64, n_heads=4, n_kv_heads=4, head_dim=16,
                      d_ffn=96, vocab=128)


def library_forward(W, cfg, toks):
    """Whole sequence at once, no cache: library rms_norm / sdpa / silu, RoPE as a complex
    multiplication.  K and V pass through bf16 exactly where the cache contract says."""
    H, Hkv, dh = cfg["n_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    T = len(toks)
    x = W["tok_emb"].double()[torch.as_tensor(toks, dtype=torch.long)]
    inv = 1.0 / (cfg["rope_theta"] ** (torch.arange(0, dh, 2, dtype=torch.float64) / dh))
    rot = torch.polar(torch.ones(T, dh // 2, dtype=torch.float64),
                      torch.arange(T, dtype=torch.float64)[:, None] * inv[None, :])   # e^{i pos w}

    def rope_c(t):                       # t [T, heads, dh]; pair (i, i + dh/2) is one complex number
        z = torch.complex(t[..., :dh // 2], t[..., dh // 2:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    for lw in W["layers"]:
        h = F.rms_norm(x, (x.shape[-1],), lw["attn_norm"].double(), cfg["rms_eps"])
        q = rope_c(F.linear(h, lw["wq"].double()).view(T, H, dh))
        k = rope_c(F.linear(h, lw["wk"].double()).view(T, Hkv, dh)).bfloat16().double()
        v = F.linear(h, lw["wv"].double()).view(T, Hkv, dh).bfloat16().double()
        k = k.repeat_interleave(H // Hkv, dim=1)
        v = v.repeat_interleave(H // Hkv, dim=1)
        a = F.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1),
                                           is_causal=True).transpose(0, 1).reshape(T, H * dh)
        x = x + F.linear(a, lw["wo"].double())
        h = F.rms_norm(x, (x.shape[-1],), lw["ffn_norm"].double(), cfg["rms_eps"])
        x = x + F.linear(F.silu(F.linear(h, lw["w_gate"].double())) * F.linear(h, lw["w_up"].double()),
                         lw["w_down"].double())
    return F.linear(F.rms_norm(x, (x.shape[-1],), W["final_norm"].double(), cfg["rms_eps"]),
                    W["lm_head"].double())


def test_incremental_cache_equals_full_sequence_library_forward():
    for cfg in (CFG, dict(CFG, n_kv_heads=2)):
        W = synth.make_weights(cfg, seed=11, std=0.2, gain_jitter=0.3)
        toks = synth.make_prompt(37, cfg["vocab"], 5)
        want = library_forward(W, cfg, toks)
        kv = O.KVCache(cfg, 2, 64)
        got, i = [], 0
        for chunk in (5, 1, 9, 1, 1, 13, 7):        # uneven steps, as drafting produces
            got.append(O.forward(W, cfg, kv, [1], [toks[i:i + chunk]])[0])
            kv.ctx[1] += chunk
            i += chunk
        got = torch.cat(got)
        assert got.shape == want.shape
        assert (got - want).abs().max() < 1e-9 * max(1.0, want.abs().max())
        assert want.abs().max() > 0.1


def test_batched_sequences_are_independent_and_discarded_rows_are_overwritten():
    W = synth.make_weights(CFG, seed=2, std=0.2)
    a, b = synth.make_prompt(12, CFG["vocab"], 1), synth.make_prompt(9, CFG["vocab"], 2)
    kv = O.KVCache(CFG, 2, 32)
    la, lb = O.forward(W, CFG, kv, [0, 1], [a, b])
    kv1 = O.KVCache(CFG, 2, 32)
    la1 = O.forward(W, CFG, kv1, [0], [a])[0]
    lb1 = O.forward(W, CFG, kv1, [1], [b])[0]
    assert torch.equal(la, la1) or (la - la1).abs().max() < 1e-12
    assert (lb - lb1).abs().max() < 1e-12
    # commit only 5 of the 12 rows, then continue with different tokens: the result must
    # equal a fresh run over the committed prefix + new tokens (stale rows are dead)
    kv.ctx[0] += 5
    new = synth.make_prompt(4, CFG["vocab"], 3)
    cont = O.forward(W, CFG, kv, [0], [new])[0]
    want = library_forward(W, CFG, np.concatenate([a[:5], new]))[5:]
    assert (cont - want).abs().max() < 1e-9


def test_zero_layers_is_norm_then_lm_head():
    cfg = dict(CFG, n_layers=0)
    W = synth.make_weights(cfg, seed=3, std=0.5, gain_jitter=0.2)
    toks = np.asarray([3, 77, 3])
    got = O.forward(W, cfg, O.KVCache(cfg, 1, 8), [0], [toks])[0]
    e = W["tok_emb"].double()[torch.as_tensor(toks)]
    n = e / torch.sqrt((e ** 2).mean(-1, keepdim=True) + cfg["rms_eps"]) * W["final_norm"].double()
    assert (got - n @ W["lm_head"].double().T).abs().max() < 1e-12
    assert torch.equal(got[0], got[2])


def test_attention_special_cases():
    dh, H = 16, 4
    # one visible token: output is exactly its V row (first row of an empty cache)
    cfg = dict(CFG, n_layers=1)
    W = synth.make_weights(cfg, seed=4, std=0.3)
    lw = W["layers"][0]
    kv = O.KVCache(cfg, 1, 8)
    tok = np.asarray([5])
    O.forward(W, cfg, kv, [0], [tok])
    x = W["tok_emb"].double()[5]
    h = O.rmsnorm(x, lw["attn_norm"].double(), cfg["rms_eps"])
    v = (h @ lw["wv"].double().T).bfloat16()
    assert torch.equal(kv.v[0, 0, 0].reshape(-1), v)
    # position 0 is not rotated: cached K equals bf16(Wk h)
    assert torch.equal(kv.k[0, 0, 0].reshape(-1), (h @ lw["wk"].double().T).bfloat16())
    # identical K rows -> uniform softmax -> mean of V: wipe the cache keys to a constant
    kv.k[0, 0, :4] = 0
    kv.v[0, 0, :4] = torch.randn(4, H, dh).bfloat16()
    kv.ctx[0] = 4
    lw["wk"].zero_()                    # new row's key is 0 as well
    W["lm_head"].copy_(torch.eye(cfg["vocab"], cfg["d_model"]).bfloat16())
    lw["wo"].copy_(torch.eye(cfg["d_model"]).bfloat16())
    lw["w_down"].zero_()
    out = O.forward(W, cfg, kv, [0], [tok])[0][0]
    mean_v = kv.v[0, 0, :5].double().mean(0).reshape(-1)      # 4 cached + the new row
    resid = x + mean_v
    want = resid / torch.sqrt((resid ** 2).mean() + cfg["rms_eps"]) * W["final_norm"].double()
    assert (out[:cfg["d_model"]] - want).abs().max() < 1e-12


def test_rope_properties():
    x = torch.randn(3, 2, 16, dtype=torch.float64)
    y = torch.randn(3, 2, 16, dtype=torch.float64)
    p = torch.tensor([0, 7, 100])
    # shift invariance of scores; norm preservation; position 0 = identity
    s0 = (O.rope(x, p, 1e4) * O.rope(y, p + 3, 1e4)).sum(-1)
    s1 = (O.rope(x, p + 50, 1e4) * O.rope(y, p + 53, 1e4)).sum(-1)
    assert (s0 - s1).abs().max() < 1e-10
    assert (O.rope(x, p, 1e4).norm(dim=-1) - x.norm(dim=-1)).abs().max() < 1e-12
    assert torch.equal(O.rope(x, torch.zeros(3, dtype=torch.long), 1e4), x)
    # explicit 2x2 rotation of the pair (i, i + dh/2) at pos 7, i = 1: angle 7 * 1e4^(-2/16)
    ang = 7 * 1e4 ** (-2 / 16)
    r = O.rope(x, p, 1e4)[1, 0]
    assert abs(r[1] - (x[1, 0, 1] * math.cos(ang) - x[1, 0, 9] * math.sin(ang))) < 1e-12
    assert abs(r[9] - (x[1, 0, 9] * math.cos(ang) + x[1, 0, 1] * math.sin(ang))) < 1e-12


# ---- the bf16-operand yardstick (mirror_bf16 = True) -------------------------------------------------

def _bf(t):
    return t.bfloat16().double()


def _hand_mirror_forward(W, cfg, toks, round_sites=True, extra_site=False, skip_site=0):
    """Whole-sequence, cache-free composition from library routines that rounds to bf16 exactly the
    six kinds of matrix-product operands the yardstick names (norm output, rotated Q, attention output,
    FFN-norm output, SwiGLU output, final-norm output) - and K, V by the cache contract."""
    r = _bf if round_sites else (lambda t: t)
    ident = lambda t: t
    H, Hkv, dh = cfg["n_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    T = len(toks)
    x = W["tok_emb"].double()[torch.as_tensor(toks, dtype=torch.long)]
    inv = 1.0 / (cfg["rope_theta"] ** (torch.arange(0, dh, 2, dtype=torch.float64) / dh))
    rot = torch.polar(torch.ones(T, dh // 2, dtype=torch.float64),
                      torch.arange(T, dtype=torch.float64)[:, None] * inv[None, :])

    def rope_c(t):
        z = torch.complex(t[..., :dh // 2], t[..., dh // 2:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    for lw in W["layers"]:
        h = r(F.rms_norm(x, (x.shape[-1],), lw["attn_norm"].double(), cfg["rms_eps"]))            # site 1
        q = r(rope_c(F.linear(h, lw["wq"].double()).view(T, H, dh)))                               # site 2
        k = _bf(rope_c(F.linear(h, lw["wk"].double()).view(T, Hkv, dh)))
        v = _bf(F.linear(h, lw["wv"].double()).view(T, Hkv, dh))
        k = k.repeat_interleave(H // Hkv, dim=1)
        v = v.repeat_interleave(H // Hkv, dim=1)
        a = F.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1),
                                           is_causal=True).transpose(0, 1).reshape(T, H * dh)
        x = x + F.linear((ident if skip_site == 3 else r)(a), lw["wo"].double())                   # site 3
        h = r(F.rms_norm(x, (x.shape[-1],), lw["ffn_norm"].double(), cfg["rms_eps"]))             # site 4
        gate = F.linear(h, lw["w_gate"].double())
        if extra_site:
            gate = _bf(gate)                                                                       # not a site
        act = r(F.silu(gate) * F.linear(h, lw["w_up"].double()))                                   # site 5
        x = x + F.linear(act, lw["w_down"].double())
    return F.linear(r(F.rms_norm(x, (x.shape[-1],), W["final_norm"].double(), cfg["rms_eps"])),   # final site
                    W["lm_head"].double())


def test_mirror_with_identity_rounding_is_the_exact_forward_bit_for_bit(monkeypatch):
    W = synth.make_weights(CFG, seed=21, std=0.2, gain_jitter=0.3)
    toks = synth.make_prompt(11, CFG["vocab"], 6)
    exact = O.forward(W, CFG, O.KVCache(CFG, 1, 16), [0], [toks])[0]
    monkeypatch.setattr(O, "_r", lambda x, mirror: x)
    kv = O.KVCache(CFG, 1, 16)
    got = O.forward(W, CFG, kv, [0], [toks], mirror_bf16=True)[0]
    assert torch.equal(got, exact)


def test_mirror_rounds_exactly_the_named_operand_sites(monkeypatch):
    calls = []
    real = O._r

    def spy(x, mirror):
        calls.append((tuple(x.shape), bool(mirror)))
        return real(x, mirror)

    monkeypatch.setattr(O, "_r", spy)
    W = synth.make_weights(CFG, seed=22, std=0.2)
    toks = synth.make_prompt(7, CFG["vocab"], 7)
    O.forward(W, CFG, O.KVCache(CFG, 1, 8), [0], [toks], mirror_bf16=True)
    L, d, f = CFG["n_layers"], CFG["d_model"], CFG["d_ffn"]
    assert O.MIRROR_SITES_PER_LAYER == 5 and O.MIRROR_SITES_FINAL == 1
    assert len(calls) == L * O.MIRROR_SITES_PER_LAYER + O.MIRROR_SITES_FINAL
    assert all(m for _, m in calls)
    per_layer = [(7, d), (7, CFG["n_heads"], CFG["head_dim"]), (7, CFG["n_heads"] * CFG["head_dim"]), (7, d), (7, f)]
    assert [s for s, _ in calls] == per_layer * L + [(7, d)]


def test_mirror_equals_a_hand_composition_that_rounds_those_sites_only():
    for n_layers in (1, 2):
        cfg = dict(CFG, n_layers=n_layers)
        W = synth.make_weights(cfg, seed=23, std=0.2, gain_jitter=0.3)
        toks = synth.make_prompt(19, cfg["vocab"], 8)
        kv = O.KVCache(cfg, 1, 32)
        got, i = [], 0
        for chunk in (6, 1, 9, 3):
            got.append(O.forward(W, cfg, kv, [0], [toks[i:i + chunk]], mirror_bf16=True)[0])
            kv.ctx[0] += chunk
            i += chunk
        got = torch.cat(got)
        want = _hand_mirror_forward(W, cfg, toks)
        assert (got - want).abs().max() < 1e-9
        # the rounding is really there (a mirror that rounds nothing would equal the exact forward),
        # it is small, and a composition with one site fewer or one more is told apart
        exact = _hand_mirror_forward(W, cfg, toks, round_sites=False)
        gap = float((want - exact).abs().max())
        assert 1e-4 < gap < 0.2
        kv2 = O.KVCache(cfg, 1, 32)
        ex2 = O.forward(W, cfg, kv2, [0], [toks])[0]
        assert (ex2 - exact).abs().max() < 1e-9
        assert (got - _hand_mirror_forward(W, cfg, toks, extra_site=True)).abs().max() > 1e-5
        assert (got - _hand_mirror_forward(W, cfg, toks, skip_site=3)).abs().max() > 1e-5


def test_mirror_stays_within_the_logit_tolerance_on_the_tiny_shape():
    cfg = synth.model_cfg("tiny")
    W = synth.make_weights(cfg, seed=0)
    toks = synth.make_prompt(24, cfg["vocab"], 2000)
    a = O.forward(W, cfg, O.KVCache(cfg, 1, 32), [0], [toks])[0]
    b = O.forward(W, cfg, O.KVCache(cfg, 1, 32), [0], [toks], mirror_bf16=True)[0]
    err = float((a - b).abs().max())
    assert 0 < err < 2e-2


def test_hidden_out_observes_the_residual_stream_without_changing_the_result():
    W = synth.make_weights(CFG, seed=24, std=0.2)
    toks = synth.make_prompt(5, CFG["vocab"], 9)
    hs = []
    a = O.forward(W, CFG, O.KVCache(CFG, 1, 8), [0], [toks], hidden_out=hs)[0]
    b = O.forward(W, CFG, O.KVCache(CFG, 1, 8), [0], [toks])[0]
    assert torch.equal(a, b) and len(hs) == CFG["n_layers"] + 1
    assert torch.equal(hs[0], W["tok_emb"].double()[torch.as_tensor(toks, dtype=torch.long)])
    last = O.rmsnorm(hs[-1], W["final_norm"].double(), CFG["rms_eps"]) @ W["lm_head"].double().T
    assert (last - a).abs().max() < 1e-12


def test_split_rounding_keeps_sixteen_bits():
    """The hi + lo form of the yardstick's rounding: exact on bf16 values, within 2^-16 relative elsewhere,
    and never worse than the plain bf16 rounding."""
    g = torch.Generator().manual_seed(3)
    x = torch.randn(10000, generator=g, dtype=torch.float64) * 37.0
    r1, r2 = O._r(x, True), O._r(x, 2)
    assert ((r2 - x).abs() <= 2.0 ** -16 * x.abs()).all()
    assert ((r2 - x).abs() <= (r1 - x).abs()).all() and ((r1 - x).abs() <= 2.0 ** -8 * x.abs()).all()
    b = x.to(torch.bfloat16).to(torch.float64)
    assert torch.equal(O._r(b, 2), b) and torch.equal(O._r(b, True), b) and torch.equal(O._r(x, False), x)
