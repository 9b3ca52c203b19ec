"""Error-versus-depth curve of the bf16-operand yardstick at the 7B width (CPU only).

Test infrastructure (see the package docstring): calls only the oracle and the seeded input
generators.  For one sequence of the verify-step workload (Llama-2-7B shape, 512 cached tokens of
synthetic N(0,1) K/V in bf16, 1 + 8 rows) it runs the exact fp64 forward and the same forward with
the matrix-product A operands rounded to bf16 (`forward(..., mirror_bf16=True)`), and compares the
logits the two give when the model is cut after L = 1, 2, 4, 8, 16, 32 layers (final norm and LM head
applied to the residual stream leaving layer L).  The table answers: how far can ANY implementation
that feeds bf16 activations to its matrix products be from the exact forward at this width and depth.

    python -m oracle.mirror_depth_curve [--layers 32] [--rows 9] [--write FILE]

With --write the table replaces the block between the markers
`<!-- mirror-depth-curve:begin -->` and `<!-- mirror-depth-curve:end -->` of that file.
"""
from __future__ import annotations

import argparse
import os
import sys
import time

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from oracle import forward as O                      # noqa: E402
from paper_2408_05676_b200 import synth              # noqa: E402

BEGIN, END = "<!-- mirror-depth-curve:begin -->", "<!-- mirror-depth-curve:end -->"


def curve(n_layers: int, rows: int, ctx: int, depths, seed_w: int = 0, seed_kv: int = 7, seed_tok: int = 8):
    cfg = synth.model_cfg("7b", n_layers=n_layers)
    t0 = time.time()
    W = synth.make_weights(cfg, seed=seed_w)
    print("weights: %.0f s" % (time.time() - t0), flush=True)
    width = cfg["n_kv_heads"] * cfg["head_dim"]
    kv = O.KVCache(cfg, 1, ctx + rows)
    for l in range(n_layers):
        k, v = synth.make_kv_layer(ctx, width, seed_kv, l)
        kv.k[l, 0, :ctx] = k.view(ctx, cfg["n_kv_heads"], cfg["head_dim"])
        kv.v[l, 0, :ctx] = v.view(ctx, cfg["n_kv_heads"], cfg["head_dim"])
    kv.ctx[:] = ctx
    tokens = np.random.default_rng(seed_tok).integers(0, cfg["vocab"], size=rows).astype(np.int32)
    hid = {}
    for mirror in (False, True, 2):
        t0 = time.time()
        hs = []
        O.forward(W, cfg, kv.clone(), [0], [tokens], mirror_bf16=mirror, hidden_out=hs)
        hid[mirror] = hs
        print("forward mirror=%s: %.0f s" % (mirror, time.time() - t0), flush=True)
    gain, head = W["final_norm"].to(O.F64), W["lm_head"].to(O.F64)
    out = []
    for L in depths:
        if L > n_layers:
            continue
        exact = O.rmsnorm(hid[False][L], gain, cfg["rms_eps"]) @ head.T
        mirr = O._r(O.rmsnorm(hid[True][L], gain, cfg["rms_eps"]), True) @ head.T
        split = O._r(O.rmsnorm(hid[2][L], gain, cfg["rms_eps"]), 2) @ head.T
        diff = mirr - exact
        out.append(dict(L=L, max_abs=float(diff.abs().max()), rms=float(diff.pow(2).mean().sqrt()),
                        logit_std=float(exact.std()),
                        argmax_agree=float((mirr.argmax(-1) == exact.argmax(-1)).double().mean()),
                        split_max_abs=float((split - exact).abs().max())))
        print(out[-1], flush=True)
    return out


def table(rows_out, rows, ctx) -> str:
    lines = ["Yardstick: fp64 forward with bf16-rounded matrix-product operands against the exact fp64 forward,",
             "7B width, one sequence, %d cached tokens, %d rows x 32000 logits (written by" % (ctx, rows),
             "`python -m oracle.mirror_depth_curve --write <this file>`; CPU only, oracle only).", "",
             "| layers L | max-abs | rms | logit std | arg-max agreement | max-abs with operands as hi + lo bf16 pairs |",
             "|---|---|---|---|---|---|"]
    for r in rows_out:
        lines.append("| %d | %.4f | %.5f | %.3f | %.2f | %.2e |" % (r["L"], r["max_abs"], r["rms"], r["logit_std"], r["argmax_agree"],
                                                                   r["split_max_abs"]))
    return "\n".join(lines)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--rows", type=int, default=9)
    ap.add_argument("--ctx", type=int, default=512)
    ap.add_argument("--write", default=None)
    a = ap.parse_args()
    res = curve(a.layers, a.rows, a.ctx, (1, 2, 4, 8, 16, 32))
    txt = table(res, a.rows, a.ctx)
    print(txt)
    if a.write:
        s = open(a.write).read()
        if BEGIN in s and END in s:
            s = s[:s.index(BEGIN) + len(BEGIN)] + "\n" + txt + "\n" + s[s.index(END):]
        else:
            s = s.rstrip("\n") + "\n\n" + BEGIN + "\n" + txt + "\n" + END + "\n"
        open(a.write, "w").write(s)


if __name__ == "__main__":
    main()
