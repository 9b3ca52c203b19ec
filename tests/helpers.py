"""Shared helpers of the GPU parity tests."""
import numpy as np
import torch

from paper_2408_05676_b200 import synth


def ensure_built():
    from paper_2408_05676_b200 import build
    return build.build()


def weights_to(W, device):
    """Move synth weights to a device, keeping q/k/v and gate/up as slices of one tensor."""
    out = {k: W[k].to(device) for k in ("tok_emb", "lm_head", "final_norm")}
    out["layers"] = []
    for lw in W["layers"]:
        wqkv, wgu = lw["wqkv"].to(device), lw["wgu"].to(device)
        dq, dkv, f = lw["wq"].shape[0], lw["wk"].shape[0], lw["w_gate"].shape[0]
        out["layers"].append(dict(
            wqkv=wqkv, wq=wqkv[:dq], wk=wqkv[dq:dq + dkv], wv=wqkv[dq + dkv:], wo=lw["wo"].to(device),
            wgu=wgu, w_gate=wgu[:f], w_up=wgu[f:], w_down=lw["w_down"].to(device),
            attn_norm=lw["attn_norm"].to(device), ffn_norm=lw["ffn_norm"].to(device)))
    return out


def dev_i32(a):
    return torch.as_tensor(np.ascontiguousarray(a, dtype=np.int32), device="cuda")
