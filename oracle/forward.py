"""Verify-forward oracle: q_i = M(x_<=t, x~_<i), i = 1..K+1 (Eq. 3 / Eq. 6).

Test infrastructure only (see the package docstring).

The paper treats the target model M as a black box; the model here is the
Llama-style decoder the workloads name: RMSNorm, rotary position embedding
(rotate-half pairing of feature i with i + head_dim/2), causal attention scaled by
1/sqrt(head_dim), SwiGLU feed-forward, no biases, separate embedding and LM head.
For a chain pseudo-sequence the mask M_t is causal and the position ids P_t are
consecutive: row i of a sequence with ctx cached tokens sits at position ctx + i and
attends to the cache [0, ctx) and to rows 0..i of the same step.  For a token tree
(Section 3.3, `parents` given) row i sits at position ctx + depth(i), attends to the
cache and to its ancestors and itself, and its K and V still go to cache slot ctx + i.

Arithmetic: everything in fp64 except what the data contract fixes - weights are
bf16 values, and K and V are rounded to bf16 (round-to-nearest-even) when they
enter the cache.  Logits come back as fp64; callers round to fp32 where the
interface says fp32.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

F64 = torch.float64


class KVCache:
    """Contiguous per-sequence cache: k, v bf16 [L, n_seqs, capacity, n_kv_heads, head_dim]."""

    def __init__(self, cfg: Dict, n_seqs: int, capacity: int):
        L, Hkv, dh = cfg["n_layers"], cfg["n_kv_heads"], cfg["head_dim"]
        self.k = torch.zeros(L, n_seqs, capacity, Hkv, dh, dtype=torch.bfloat16)
        self.v = torch.zeros(L, n_seqs, capacity, Hkv, dh, dtype=torch.bfloat16)
        self.ctx = np.zeros(n_seqs, dtype=np.int64)
        self.capacity = capacity

    def clone(self) -> "KVCache":
        c = object.__new__(KVCache)
        c.k, c.v, c.ctx, c.capacity = self.k.clone(), self.v.clone(), self.ctx.copy(), self.capacity
        return c


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    return x * torch.rsqrt((x * x).mean(dim=-1, keepdim=True) + eps) * gain


def rope(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """x [R, H, dh]; rotate the pair (i, i + dh/2) by pos * theta^(-2i/dh)."""
    dh = x.shape[-1]
    half = dh // 2
    inv_freq = theta ** (-(torch.arange(half, dtype=F64) * 2.0 / dh))
    ang = pos.to(F64)[:, None] * inv_freq[None, :]
    c, s = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * c - x2 * s, x2 * c + x1 * s], dim=-1)


# The activations a bf16-operand implementation hands to a matrix product (the A operands): per
# layer the attention-norm output, the rotated queries, the attention output, the FFN-norm output
# and the SwiGLU output; after the last layer the final-norm output.
MIRROR_SITES_PER_LAYER = 5
MIRROR_SITES_FINAL = 1


def _r(x: torch.Tensor, mirror) -> torch.Tensor:
    """Yardstick mode: round an activation where a bf16-operand implementation would hand it to a matrix
    product.  mirror = True: to bf16 (nearest-even).  mirror = 2: to a sum of two bf16 values, hi = bf16(x)
    and lo = bf16(x - hi), which is what an implementation gets that feeds the operand as two bf16
    matrices (about 16 significant bits).  False: identity."""
    if not mirror:
        return x
    hi = x.to(torch.bfloat16).to(F64)
    if mirror == 2:
        return hi + (x - hi).to(torch.bfloat16).to(F64)
    return hi


def forward(W: Dict, cfg: Dict, kv: KVCache, seq_ids: Sequence[int],
            tokens: Sequence[np.ndarray], mirror_bf16=False,
            parents: Optional[Sequence[Sequence[int]]] = None,
            hidden_out: Optional[List[torch.Tensor]] = None) -> List[torch.Tensor]:
    """One forward over the new rows of each listed sequence.

    tokens[j] holds the rows of sequence seq_ids[j]: the pending token followed by its
    drafts (or a prompt chunk).  K and V of every row are written to the cache at
    positions ctx .. ctx + rows - 1; kv.ctx itself is not changed (committing is the
    acceptance step's job).  Returns one fp64 logits tensor [rows, vocab] per sequence.
    parents[j][i-1] (optional) = row of row i's parent in sequence j's token tree (row 0 is the
    root); without it the rows are a chain.
    mirror_bf16 = True gives the yardstick of a bf16-operand implementation: the same forward with
    the matrix-product A operands (MIRROR_SITES_PER_LAYER per layer, MIRROR_SITES_FINAL after the
    last) rounded to bf16 and nothing else changed.
    hidden_out (optional list) receives the residual stream [all rows, d_model] entering layer 0
    and leaving every layer (observation only).
    """
    H, Hkv, dh = cfg["n_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    eps, theta = cfg["rms_eps"], cfg["rope_theta"]
    rows = [len(t) for t in tokens]
    starts = np.concatenate([[0], np.cumsum(rows)]).astype(int)
    flat = torch.as_tensor(np.concatenate([np.asarray(t, dtype=np.int64) for t in tokens]))
    anc: List[List[List[int]]] = []      # per sequence, per row: the rows it sees (ancestors and itself)
    dep: List[List[int]] = []
    for j, r in enumerate(rows):
        par = [i - 1 for i in range(1, r)] if parents is None else [int(x) for x in parents[j][:max(r - 1, 0)]]
        d, a = [0] * r, [[0]] * r if r else []
        for i in range(1, r):
            if not 0 <= par[i - 1] < i:
                raise ValueError("a parent must be an earlier row")
            d[i] = d[par[i - 1]] + 1
            a[i] = a[par[i - 1]] + [i]
        dep.append(d)
        anc.append(a)
    pos = torch.cat([torch.as_tensor(dep[j], dtype=torch.int64) + int(kv.ctx[s])
                     for j, s in enumerate(seq_ids)])
    for s, r in zip(seq_ids, rows):
        if kv.ctx[s] + r > kv.capacity:
            raise ValueError("KV capacity exceeded")
    x = W["tok_emb"][flat].to(F64)
    if hidden_out is not None:
        hidden_out.append(x.clone())
    rep = H // Hkv
    for l, lw in enumerate(W["layers"]):
        h = _r(rmsnorm(x, lw["attn_norm"].to(F64), eps), mirror_bf16)
        q = (h @ lw["wq"].to(F64).T).view(-1, H, dh)
        k = (h @ lw["wk"].to(F64).T).view(-1, Hkv, dh)
        v = (h @ lw["wv"].to(F64).T).view(-1, Hkv, dh)
        q = _r(rope(q, pos, theta), mirror_bf16)
        k = rope(k, pos, theta).to(torch.bfloat16)          # cache contract: bf16 K, V
        v = v.to(torch.bfloat16)
        att = torch.empty(x.shape[0], H, dh, dtype=F64)
        for j, s in enumerate(seq_ids):
            a, b, c = starts[j], starts[j + 1], int(kv.ctx[s])
            kv.k[l, s, c:c + rows[j]] = k[a:b]
            kv.v[l, s, c:c + rows[j]] = v[a:b]
            for i in range(rows[j]):                          # row i sees the cache + its ancestors + itself
                see = list(range(c)) + [c + r_ for r_ in anc[j][i]]
                kk = kv.k[l, s, see].to(F64).repeat_interleave(rep, dim=1)   # [n, H, dh]
                vv = kv.v[l, s, see].to(F64).repeat_interleave(rep, dim=1)
                sc = torch.einsum("hd,nhd->hn", q[a + i], kk) / (dh ** 0.5)
                pr = torch.softmax(sc, dim=-1)
                att[a + i] = torch.einsum("hn,nhd->hd", pr, vv)
        x = x + _r(att.reshape(-1, H * dh), mirror_bf16) @ lw["wo"].to(F64).T
        h2 = _r(rmsnorm(x, lw["ffn_norm"].to(F64), eps), mirror_bf16)
        gate = h2 @ lw["w_gate"].to(F64).T
        up = h2 @ lw["w_up"].to(F64).T
        act = _r(gate * torch.sigmoid(gate) * up, mirror_bf16)  # SwiGLU: silu(gate) * up
        x = x + act @ lw["w_down"].to(F64).T
        if hidden_out is not None:
            hidden_out.append(x.clone())
    hn = _r(rmsnorm(x, W["final_norm"].to(F64), eps), mirror_bf16)
    logits = hn @ W["lm_head"].to(F64).T
    return [logits[starts[j]:starts[j + 1]] for j in range(len(rows))]
