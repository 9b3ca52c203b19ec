"""Generation-loop oracle: Draft-Then-Verify (Section 2.1, Section 3) and Eq. 1.

Test infrastructure only (see the package docstring).

One decoding step per sequence: take the last n_max tokens as the tail (the
pending, not-yet-cached token is its newest element), retrieve a draft (Eq. 5),
verify [pending token, drafts] in one forward (Eq. 3), accept a prefix (Eq. 4 or
Eq. 8), emit the accepted drafts plus one token from the model, advance the cache
by the number of emitted tokens.  The prompt is prefilled except for its last
token, which is the first pending token.  Generation stops at max_new tokens
(the last step is truncated) or right after the first eos_id.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import accept as acc
from . import forward as fwd
from . import retrieval as ret
from . import tree as tr


def prefill(W: Dict, cfg: Dict, kv: fwd.KVCache, seq: int, prompt: np.ndarray, chunk: int = 64) -> None:
    """Cache all prompt tokens but the last."""
    body = np.asarray(prompt[:-1])
    for i in range(0, len(body), chunk):
        part = body[i:i + chunk]
        fwd.forward(W, cfg, kv, [seq], [part])
        kv.ctx[seq] += len(part)


def generate(W: Dict, cfg: Dict, prompts: Sequence[np.ndarray], group_id: Sequence[int],
             pool: Optional[np.ndarray], group_offsets: Optional[np.ndarray], *,
             K: int, n_min: int, n_max: int, max_new: int, mode: int = acc.STRICT,
             topk: int = 2, p: float = 0.1, min_draft: int = 1, max_occ: int = 0,
             eos_id: int = -1, capacity: Optional[int] = None, temp_branches: bool = False,
             tree: bool = False) -> Dict:
    """Draft-Then-Verify generation.  pool=None (or K=0) gives plain greedy decoding.
    temp_branches: the sequence's prompt and the tokens generated so far are searched as a
    temporary branch beside the pool (Section 3.2).
    tree: draft a token tree of up to K nodes and verify it with tree attention (Section 3.3); the
    accepted path's K and V move from their rows' cache slots to consecutive positions.

    Returns dict(out=[token lists], steps, drafted, accepted, emitted) where the three
    counters are sums over all decoding steps of all sequences, and trace = per sequence
    list of (draft, n_accept, emitted tokens) for each step.
    """
    B = len(prompts)
    cap = capacity or (max(len(p_) for p_ in prompts) + max_new + K + 2)
    kv = fwd.KVCache(cfg, B, cap)
    seqs: List[List[int]] = [list(map(int, p_)) for p_ in prompts]
    out: List[List[int]] = [[] for _ in range(B)]
    trace: List[list] = [[] for _ in range(B)]
    stats = dict(steps=0, drafted=0, accepted=0, emitted=0)
    for b in range(B):
        prefill(W, cfg, kv, b, np.asarray(prompts[b]))
    done = [False] * B
    while not all(done):
        for b in range(B):
            if done[b]:
                continue
            draft: List[int] = []
            par: List[int] = []
            if pool is not None and K > 0:
                g = int(group_id[b])
                hist = np.asarray(seqs[b]) if temp_branches else None
                if tree:
                    draft, par, _ = tr.draft_tree_one(pool, int(group_offsets[g]), int(group_offsets[g + 1]),
                                                      np.asarray(seqs[b][-n_max:]), K, n_min, n_max,
                                                      min_draft, max_occ, hist)
                else:
                    draft, _ = ret.draft_one(pool, int(group_offsets[g]), int(group_offsets[g + 1]),
                                             np.asarray(seqs[b][-n_max:]), K, n_min, n_max,
                                             min_draft, max_occ, hist)
            rows = np.asarray([seqs[b][-1]] + draft, dtype=np.int32)
            if tree:
                logits = fwd.forward(W, cfg, kv, [b], [rows], parents=[par])[0].to(torch.float32).numpy()
                a, em, path = tr.accept_tree(logits, rows, par, len(rows), mode, topk, p)
                c = int(kv.ctx[b])
                for d, row in enumerate(path, 1):       # ascending: a target slot is never a later source
                    kv.k[:, b, c + d] = kv.k[:, b, c + row]
                    kv.v[:, b, c + d] = kv.v[:, b, c + row]
            else:
                logits = fwd.forward(W, cfg, kv, [b], [rows])[0].to(torch.float32).numpy()
                a, em = acc.accept_one(logits, rows, len(rows), mode, topk, p)
            room = max_new - len(out[b])
            em = em[:room]
            if eos_id >= 0 and eos_id in em:
                em = em[:em.index(eos_id) + 1]
                done[b] = True
            kv.ctx[b] += len(em)
            seqs[b].extend(em)
            out[b].extend(em)
            trace[b].append((list(draft), a, list(em)))
            stats["steps"] += 1
            stats["drafted"] += len(draft)
            stats["accepted"] += a
            stats["emitted"] += len(em)
            if len(out[b]) >= max_new:
                done[b] = True
    return dict(out=out, trace=trace, ctx=kv.ctx.copy(), **stats)


def greedy(W: Dict, cfg: Dict, prompts: Sequence[np.ndarray], max_new: int, eos_id: int = -1) -> Dict:
    """Plain autoregressive greedy decoding (Eq. 1 with argmax), one token per forward."""
    return generate(W, cfg, prompts, [0] * len(prompts), None, None, K=0, n_min=1, n_max=1,
                    max_new=max_new, eos_id=eos_id)
