"""Seeded synthetic inputs: model shapes, weights, prompts, pools, queries, logits.

These generators stand in for the public recommendation datasets and trained
language models the paper measures on (Section 4.1); none of those is
available offline.  The module holds no step of the decoding method itself:
it only draws numbers.  Both the CPU oracle's tests and the CUDA path's tests
feed from here so that they see identical bits.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np
import torch

SENTINEL = -1  # document separator inside a pool's token array

# Llama-style decoder shapes.  "tiny" is the small end-to-end case; "7b" and
# "13b" follow the Llama-2 dimensions.
MODEL_SHAPES: Dict[str, Dict] = {
    "tiny": dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64,
                 d_ffn=688, vocab=4096),
    "7b": dict(n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32, head_dim=128,
               d_ffn=11008, vocab=32000),
    "13b": dict(n_layers=40, d_model=5120, n_heads=40, n_kv_heads=40, head_dim=128,
                d_ffn=13824, vocab=32000),
}


def model_cfg(name: str, **over) -> Dict:
    cfg = dict(MODEL_SHAPES[name])
    cfg.update(rms_eps=1e-5, rope_theta=10000.0, page_size=16, max_draft=8)
    cfg.update(over)
    return cfg


def make_weights(cfg: Dict, seed: int = 0, device: str = "cpu", std: float = 0.02,
                 gain_jitter: float = 0.0) -> Dict:
    """Random-init weights, N(0, std) rounded to bf16, norm gains 1 (+ jitter).

    Q/K/V of a layer are slices of one [3*d, d] tensor and gate/up slices of
    one [2*f, d] tensor, so a consumer may treat each group as a single matrix.
    All matrices are row-major [out_features, in_features].
    """
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    d, f, V, L = cfg["d_model"], cfg["d_ffn"], cfg["vocab"], cfg["n_layers"]
    dq = cfg["n_heads"] * cfg["head_dim"]
    dkv = cfg["n_kv_heads"] * cfg["head_dim"]

    def mat(rows, cols):
        w = torch.empty(rows, cols, dtype=torch.float32, device=device)
        w.normal_(0.0, std, generator=g)
        return w.to(torch.bfloat16)

    def gain(n):
        w = torch.ones(n, dtype=torch.float32, device=device)
        if gain_jitter > 0:
            w += gain_jitter * torch.randn(n, generator=g, device=device)
        return w.to(torch.bfloat16)

    W = dict(tok_emb=mat(V, d), lm_head=mat(V, d), final_norm=gain(d), layers=[])
    for _ in range(L):
        wqkv = mat(dq + 2 * dkv, d)
        wgu = mat(2 * f, d)
        W["layers"].append(dict(
            wqkv=wqkv, wq=wqkv[:dq], wk=wqkv[dq:dq + dkv], wv=wqkv[dq + dkv:],
            wo=mat(d, dq), wgu=wgu, w_gate=wgu[:f], w_up=wgu[f:], w_down=mat(d, f),
            attn_norm=gain(d), ffn_norm=gain(d)))
    return W


def make_prompt(length: int, vocab: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.integers(0, vocab, size=length, dtype=np.int64).astype(np.int32)


def make_prompts(n: int, len_lo: int, len_hi: int, vocab: int, seed_base: int) -> List[np.ndarray]:
    """n prompts of uniform-random tokens, lengths uniform in [len_lo, len_hi]."""
    out = []
    for b in range(n):
        rng = np.random.default_rng(seed_base + b)
        ln = int(rng.integers(len_lo, len_hi + 1))
        out.append(rng.integers(0, vocab, size=ln, dtype=np.int64).astype(np.int32))
    return out


def pool_from_documents(groups: Sequence[Sequence[Sequence[int]]]) -> Tuple[np.ndarray, np.ndarray]:
    """Concatenate documents (token lists) per group, separated by SENTINEL."""
    toks: List[int] = []
    offs = [0]
    for docs in groups:
        first = True
        for doc in docs:
            if not first:
                toks.append(SENTINEL)
            toks.extend(int(t) for t in doc)
            first = False
        offs.append(len(toks))
    return np.asarray(toks, dtype=np.int32), np.asarray(offs, dtype=np.int64)


# ---------------------------------------------------------------------------
# Zipf / template pool (draft-retrieval workload)
# ---------------------------------------------------------------------------

def _zipf_cdf(vocab: int, s: float) -> np.ndarray:
    w = 1.0 / np.power(np.arange(1, vocab + 1, dtype=np.float64), s)
    c = np.cumsum(w)
    return c / c[-1]


def zipf_tokens(n: int, vocab: int, s: float, rng: np.random.Generator,
                perm: np.ndarray, cdf: np.ndarray | None = None) -> np.ndarray:
    """n draws from Zipf(s) over ranks 1..vocab; token id = perm[rank-1]."""
    if cdf is None:
        cdf = _zipf_cdf(vocab, s)
    out = np.empty(n, dtype=np.int32)
    step = 1 << 24
    for i in range(0, n, step):
        m = min(step, n - i)
        r = np.searchsorted(cdf, rng.random(m), side="left")
        np.minimum(r, vocab - 1, out=r)
        out[i:i + m] = perm[r]
    return out


def group_sizes_lognormal(n_tokens: int, n_groups: int, rng: np.random.Generator,
                          sigma: float = 1.0, min_size: int = 16) -> np.ndarray:
    """Log-normal sizes, renormalised to sum exactly n_tokens, each >= min_size."""
    raw = rng.lognormal(mean=0.0, sigma=sigma, size=n_groups)
    spare = n_tokens - min_size * n_groups
    if spare < 0:
        raise ValueError("n_tokens too small for n_groups * min_size")
    sizes = np.floor(raw / raw.sum() * spare).astype(np.int64) + min_size
    sizes[: n_tokens - int(sizes.sum())] += 1  # hand out the rounding remainder
    assert sizes.sum() == n_tokens and sizes.min() >= min_size
    return sizes


def make_zipf_pool(n_tokens: int, n_groups: int, vocab: int = 32000, s: float = 1.1,
                   seed: int = 42, template_seed: int = 43, n_templates: int = 200,
                   tmpl_lo: int = 20, tmpl_hi: int = 60, template_frac: float = 0.30
                   ) -> Tuple[np.ndarray, np.ndarray]:
    """Zipf unigram stream with ~template_frac of tokens overwritten by template copies.

    Returns (tokens int32[n_tokens], group_offsets int64[n_groups+1]).  Template
    copies are pasted at uniform positions (later copies overwrite earlier ones,
    so the covered fraction lands slightly below template_frac).  There are no
    sentinels: every group is one document.
    """
    rng = np.random.default_rng(seed)
    trng = np.random.default_rng(template_seed)
    perm = trng.permutation(vocab).astype(np.int32)
    cdf = _zipf_cdf(vocab, s)
    sizes = group_sizes_lognormal(n_tokens, n_groups, rng)
    offs = np.zeros(n_groups + 1, dtype=np.int64)
    np.cumsum(sizes, out=offs[1:])
    toks = zipf_tokens(n_tokens, vocab, s, rng, perm, cdf)

    t_len = trng.integers(tmpl_lo, tmpl_hi + 1, size=n_templates)
    t_off = np.zeros(n_templates + 1, dtype=np.int64)
    np.cumsum(t_len, out=t_off[1:])
    t_tok = zipf_tokens(int(t_off[-1]), vocab, s, trng, perm, cdf)

    mean_len = float(t_len.mean())
    n_copies = int(template_frac * n_tokens / mean_len)
    if n_copies > 0:
        which = rng.integers(0, n_templates, size=n_copies)
        lens = t_len[which]
        start = rng.integers(0, np.maximum(1, n_tokens - tmpl_hi), size=n_copies)
        rep = np.repeat(np.arange(n_copies), lens)
        base = np.zeros(n_copies + 1, dtype=np.int64)
        np.cumsum(lens, out=base[1:])
        within = np.arange(int(base[-1]), dtype=np.int64) - base[rep]
        toks[start[rep] + within] = t_tok[t_off[which][rep] + within]
    return toks, offs


def make_queries(tokens: np.ndarray, group_offsets: np.ndarray, n_queries: int,
                 n_tail: int = 4, vocab: int = 32000, s: float = 1.1, seed: int = 44,
                 template_seed: int = 43, from_pool_frac: float = 0.7
                 ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Queries: group drawn in proportion to its size; the tail is n_tail consecutive
    pool tokens of that group (prob. from_pool_frac) or n_tail Zipf draws.

    Returns (tails int32[Q, n_tail], tail_len int32[Q], group_id int32[Q]).
    """
    rng = np.random.default_rng(seed)
    trng = np.random.default_rng(template_seed)
    perm = trng.permutation(vocab).astype(np.int32)
    sizes = np.diff(group_offsets).astype(np.float64)
    gid = rng.choice(len(sizes), size=n_queries, p=sizes / sizes.sum()).astype(np.int32)
    tails = zipf_tokens(n_queries * n_tail, vocab, s, rng, perm).reshape(n_queries, n_tail)
    from_pool = rng.random(n_queries) < from_pool_frac
    u = rng.random(n_queries)
    for q in np.nonzero(from_pool)[0]:
        lo, hi = int(group_offsets[gid[q]]), int(group_offsets[gid[q] + 1])
        if hi - lo < n_tail:
            continue
        st = lo + int(u[q] * (hi - lo - n_tail + 1))
        w = tokens[st:st + n_tail]
        if (w >= 0).all():
            tails[q] = w
    tail_len = np.full(n_queries, n_tail, dtype=np.int32)
    return tails.astype(np.int32), tail_len, gid


# ---------------------------------------------------------------------------
# Verify-step workload helpers
# ---------------------------------------------------------------------------

def make_kv_layer(n_tokens: int, width: int, seed: int, layer: int, device: str = "cpu"
                  ) -> Tuple[torch.Tensor, torch.Tensor]:
    """Synthetic cache contents of one layer: K, V ~ N(0,1) in bf16, [n_tokens, width]."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1000003 + int(layer))
    k = torch.randn(n_tokens, width, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(n_tokens, width, generator=g, device=device, dtype=torch.float32)
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def corrupt_drafts(greedy: np.ndarray, second: np.ndarray, vocab: int, seed: int,
                   p_agree: float = 0.6, p_second: float = 0.2) -> np.ndarray:
    """Drafts that agree with a given greedy continuation with probability p_agree per
    position, equal the runner-up token with probability p_second, else uniform."""
    rng = np.random.default_rng(seed)
    u = rng.random(greedy.shape)
    rnd = rng.integers(0, vocab, size=greedy.shape)
    out = np.where(u < p_agree, greedy, np.where(u < p_agree + p_second, second, rnd))
    return out.astype(np.int32)


def make_accept_case(B: int, K: int, V: int, seed: int, tie_frac: float = 0.15
                     ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Directly synthesised logits that reach every branch of the acceptance rules.

    logits fp32 [B, K+1, V]: N(0,1) with the largest entry of each row boosted so
    that its probability mass is roughly uniform in (0.05, 0.9); a fraction of rows
    get exact ties planted (top-1 == top-2, and rank-2 == rank-3).  tokens int32
    [B, K+1]: column 0 is the pending token, columns 1.. are drafts that are the
    row's rank-1 / rank-2 / rank-3 / a random token.  n_rows int32 [B] in [1, K+1].
    """
    rng = np.random.default_rng(seed)
    logits = rng.standard_normal((B, K + 1, V)).astype(np.float32)
    flat = logits.reshape(-1, V)
    for r in range(flat.shape[0]):
        row = flat[r].astype(np.float64)
        top = int(row.argmax())
        rest = np.exp(np.delete(row, top)).sum()
        mass = rng.uniform(0.05, 0.9)
        flat[r, top] = np.float32(math.log(mass / (1.0 - mass) * rest))
        order = np.argsort(-flat[r], kind="stable")
        c = rng.random()
        if c < tie_frac / 2:
            flat[r, order[1]] = flat[r, order[0]]
        elif c < tie_frac:
            flat[r, order[2]] = flat[r, order[1]]
    tokens = rng.integers(0, V, size=(B, K + 1)).astype(np.int32)
    for b in range(B):
        for i in range(1, K + 1):
            order = np.argsort(-logits[b, i - 1], kind="stable")
            c = rng.random()
            if c < 0.55:
                tokens[b, i] = order[0]
            elif c < 0.80:
                tokens[b, i] = order[1]
            elif c < 0.90:
                tokens[b, i] = order[2]
    n_rows = rng.integers(1, K + 2, size=B).astype(np.int32)
    return logits, tokens, n_rows


def make_embeddings(n: int, dim: int, n_clusters: int, seed: int = 50, spread: float = 0.35
                    ) -> Tuple[np.ndarray, np.ndarray]:
    """Synthetic user / item embeddings for the grouping stand-in: a mixture of n_clusters Gaussians with
    unit-scale centres and standard deviation `spread` per coordinate, cluster sizes log-normal.
    Returns (fp32 [n, dim], the generating component int32[n])."""
    rng = np.random.default_rng(seed)
    centres = rng.standard_normal((n_clusters, dim))
    w = rng.lognormal(0.0, 0.7, n_clusters)
    comp = rng.choice(n_clusters, size=n, p=w / w.sum()).astype(np.int32)
    x = centres[comp] + spread * rng.standard_normal((n, dim))
    return x.astype(np.float32), comp
