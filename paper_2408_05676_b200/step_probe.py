"""Device time of laser_verify_step alone for a model shape and step size, with the split into dense
contractions and attention (the library's per-launch event brackets), and of the step with acceptance after
the forward against acceptance fused into the LM head.

    python -m paper_2408_05676_b200.step_probe [--shape 7b|13b|tiny] [--layers L] [--batch B] [--draft K]
                                               [--ctx N] [--steps S] [--precise 1]

Synthetic weights (seed 0) and a synthetic cache of `ctx` tokens per sequence; every sequence carries
K + 1 active rows.  Prints one JSON line.  The tests and bench.py measure the named configurations; this
is the tool for other step sizes (and the command the profiler captures of the large-row kernels run).
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as L
from . import synth


def run(shape: str, layers: int, batch: int, draft: int, ctx: int, steps: int, precise: int = 0) -> dict:
    dev = "cuda"
    cfg = synth.model_cfg(shape, n_layers=layers, max_draft=draft, precise=precise)
    W = synth.make_weights(cfg, seed=0, device=dev)
    model = L.model_create(cfg, W, max_batch=batch)
    pages = (ctx + draft + 1 + 15) // 16 + 1
    kv = L.kv_create(model, batch, batch * pages)
    width = cfg["n_kv_heads"] * cfg["head_dim"]
    for l in range(layers):
        for s in range(batch):
            k, v = synth.make_kv_layer(ctx, width, 7 + 17 * s, l, device=dev)
            L.kv_import(kv, s, l, 0, k, v)
    ids = torch.arange(batch, dtype=torch.int32, device=dev)
    lens = torch.full((batch,), ctx, dtype=torch.int32, device=dev)
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    tokens = torch.randint(0, cfg["vocab"], (batch, draft + 1), dtype=torch.int32, device=dev, generator=g)
    n_rows = torch.full((batch,), draft + 1, dtype=torch.int32, device=dev)
    logits = torch.empty(batch, draft + 1, cfg["vocab"], dtype=torch.float32, device=dev)
    L.kv_set_len_dev(kv, lens)
    for _ in range(3):
        L.verify_step(model, kv, ids, tokens, n_rows, logits)
    torch.cuda.synchronize()
    L.check(model)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        L.verify_step(model, kv, ids, tokens, n_rows, logits)
    e1.record()
    torch.cuda.synchronize()
    # acceptance after the forward (logits stored, two more passes over them) against acceptance fused into the
    # LM head (no logits), strict rule, alternating so that clock drift hits both alike
    prm = L.make_params(K=draft, mode=L.MODE_STRICT)
    outs = (torch.empty(batch, dtype=torch.int32, device=dev), torch.empty(batch, draft + 1, dtype=torch.int32, device=dev),
            torch.empty(batch, dtype=torch.int32, device=dev))

    def two_kernels():
        L.verify_step(model, kv, ids, tokens, n_rows, logits)
        L.accept_commit(None, None, logits, tokens, n_rows, prm, out=outs)

    def fused():
        L.verify_accept(model, kv, ids, tokens, n_rows, prm, commit=False, out=outs)

    ab = {"two": 0.0, "fused": 0.0}
    for rnd in range(4):
        for name, fn in (("two", two_kernels), ("fused", fused)) if rnd % 2 == 0 else (("fused", fused), ("two", two_kernels)):
            fn()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            for _ in range(steps):
                fn()
            a1.record()
            torch.cuda.synchronize()
            ab[name] += a0.elapsed_time(a1) / steps / 4
    L.check(model)
    L.profile_enable(model, True)
    for _ in range(2):
        L.verify_step(model, kv, ids, tokens, n_rows, logits)
    gemm_ms, n_gemm = L.profile_read(model, 0)
    attn_ms, n_attn = L.profile_read(model, 1)
    L.profile_enable(model, False)
    L.check(model)
    d, f, V = cfg["d_model"], cfg["d_ffn"], cfg["vocab"]
    dkv = cfg["n_kv_heads"] * cfg["head_dim"]
    rows = batch * (draft + 1)
    weight_bytes = 2 * (layers * (2 * d * d + 2 * d * dkv + 3 * d * f) + d * V)
    flops = float(rows) * weight_bytes
    kv_bytes = batch * ctx * layers * 2 * dkv * 2
    return dict(shape=shape, precise=precise, layers=layers, batch=batch, rows=rows, ctx=ctx, ms_per_step=e0.elapsed_time(e1) / steps,
                verify_then_accept_ms=ab["two"], verify_accept_fused_ms=ab["fused"],
                contractions_ms=gemm_ms / 2, contraction_launches=n_gemm // 2, attention_ms=attn_ms / 2,
                attention_launches=n_attn // 2, weight_gb=weight_bytes / 1e9, kv_gb=kv_bytes / 1e9,
                contraction_tflops=flops / (gemm_ms / 2) * 1e-9, weight_gbs=weight_bytes / (gemm_ms / 2) * 1e-6,
                kv_gbs=kv_bytes / max(attn_ms / 2, 1e-9) * 1e-6)


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="7b")
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--draft", type=int, default=8)
    ap.add_argument("--ctx", type=int, default=512)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--precise", type=int, default=0, help="1 = operands as hi + lo bf16 pairs, fp32 attention")
    a = ap.parse_args()
    print(json.dumps(run(a.shape, a.layers, a.batch, a.draft, a.ctx, a.steps, a.precise)))
