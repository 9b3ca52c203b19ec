"""Retrieval time against pool size, one global pool against customised (per-group) pools.

A synthetic analogue of the paper's pool-size study (Section 3.1, Figure 2) and of the retrieval-time
column of its ablation (Table 3): the same token stream is indexed once as a single group (global pool)
and once as groups of about 5 k tokens (customised pools), at several total sizes.  Reported per
configuration: index build time and bytes, device time of laser_draft for 4096 queries (chain and tree
form), hit rate and mean draft length.

    python -m paper_2408_05676_b200.pool_sweep [--sizes 1,5,20,50]

Prints one JSON line per configuration.  The streams are the Zipf/template recipe of synth.py; real
datasets and embeddings are not available here, so acceptance quality is not part of this sweep.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from . import binding as L
from . import synth


def _time_ms(fn, reps: int = 10) -> float:
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def run(sizes_m, n_queries: int = 4096, K: int = 16) -> None:
    dev = "cuda"
    for size_m in sizes_m:
        n = int(size_m * 1e6)
        g_custom = max(1, n // 5000)
        pool, offs_c = synth.make_zipf_pool(n, g_custom, vocab=32000, seed=42)
        tails, tail_len, gid_c = synth.make_queries(pool, offs_c, n_queries, n_tail=4, seed=44)
        for name, offs, gid in (("customised", offs_c, gid_c),
                                ("global", np.asarray([0, n], np.int64), np.zeros(n_queries, np.int32))):
            t0 = time.time()
            h = L.pool_build(pool, offs, 1, 4)
            torch.cuda.synchronize()
            build_s = time.time() - t0
            info = h.info()
            n_keys, dev_bytes = info["n_keys"], info["device_bytes"]
            prm = L.make_params(K=K, n_min=1, n_max=4, max_occ=64)
            d_t, d_l, d_g = (torch.as_tensor(x, device=dev) for x in (tails, tail_len, gid))
            out = {}

            def chain():
                out["c"] = L.draft(h, d_t, d_l, d_g, prm)

            def tree():
                out["t"] = L.draft_tree(h, d_t, d_l, d_g, prm)

            ms_chain, ms_tree = _time_ms(chain), _time_ms(tree)
            dl = out["c"][1].cpu().numpy()
            rec = dict(pool_tokens=n, pools=name, groups=int(len(offs) - 1), build_s=round(build_s, 3),
                       index_gb=round(dev_bytes / 1e9, 3), keys=int(n_keys),
                       draft_us_per_4096_queries=round(ms_chain * 1e3, 1),
                       tree_draft_us_per_4096_queries=round(ms_tree * 1e3, 1),
                       hit_rate=round(float((dl > 0).mean()), 3), mean_draft=round(float(dl.mean()), 2),
                       mean_tree_nodes=round(float(out["t"][2].float().mean()), 2))
            print(json.dumps(rec), flush=True)
            h.free()


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--sizes", default="1,5,20,50", help="total pool sizes in millions of tokens")
    a = ap.parse_args()
    run([float(x) for x in a.sizes.split(",")])
