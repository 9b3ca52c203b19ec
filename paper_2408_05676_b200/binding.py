"""Thin ctypes binding of liblaser.so: same names as the C ABI, argument marshalling only.

Device arrays are torch CUDA tensors (torch provides device memory and streams, nothing
else); their data pointers are handed to the library unchanged.  Importing this module
loads the CUDA library and raises if it has not been built - there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblaser.so")
if not os.path.exists(LIB_PATH):
    raise ImportError("%s is missing: run `python -m paper_2408_05676_b200.build` first" % LIB_PATH)
lib = C.CDLL(LIB_PATH)

OK = 0
MODE_STRICT, MODE_RELAXED, MODE_TOPK, MODE_TOPP, MODE_RELAXED_ARGMAX = 0, 1, 2, 3, 4
STATUS = {0: "OK", -1: "INVALID_ARG", -2: "OOM", -3: "CUDA", -4: "CAPACITY", -5: "TIMEOUT", -6: "UNSUPPORTED"}


class LaserError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__("laser: %s (%d): %s" % (STATUS.get(status, "?"), status, msg))
        self.status = status


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim",
                                          "d_ffn", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("page_size", "max_draft", "max_batch", "precise")]


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tok_emb", "lm_head", "final_norm")] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down",
                                                     "attn_norm", "ffn_norm")]


class Params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("K", "n_min", "n_max", "min_draft", "max_occ", "mode", "topk")] + \
               [("p", C.c_float), ("max_new", C.c_int32), ("eos_id", C.c_int32), ("temp_branches", C.c_int32), ("tree", C.c_int32),
                ("fused_accept", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("steps", "drafted", "accepted", "emitted", "launches", "verify_calls")] + \
               [(n, C.c_float) for n in ("ms_prefill", "ms_draft", "ms_verify", "ms_accept", "ms_total")]

    def as_dict(self) -> Dict:
        return {n: getattr(self, n) for n, _ in self._fields_}


EXPORTS = ["laser_version", "laser_last_error", "laser_launch_count", "laser_pool_build", "laser_pool_free",
           "laser_pool_info", "laser_draft", "laser_draft_temp", "laser_draft_tree", "laser_make_rows", "laser_make_rows_tree", "laser_model_create", "laser_model_free",
           "laser_kv_create", "laser_kv_free", "laser_kv_set_page_table", "laser_kv_set_len",
           "laser_kv_get_len", "laser_kv_reset", "laser_kv_set_len_dev", "laser_kv_import", "laser_kv_export",
           "laser_verify_step", "laser_verify_step_tree", "laser_check", "laser_profile_enable", "laser_profile_read", "laser_accept_commit", "laser_accept_commit_noalloc", "laser_accept_tree", "laser_kv_compact_path",
           "laser_verify_accept",
           "laser_selftest_wait", "laser_group_kmeans", "laser_generate"]

lib.laser_version.restype = C.c_char_p
lib.laser_last_error.restype = C.c_char_p
lib.laser_launch_count.restype = C.c_int64
for _n in EXPORTS[3:]:
    getattr(lib, _n).restype = C.c_int32


def _chk(status: int) -> None:
    if status != OK:
        raise LaserError(status, lib.laser_last_error().decode())


def _ptr(t) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensor must be contiguous"
        return C.c_void_p(t.data_ptr())
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return C.c_void_p(t.ctypes.data)
    raise TypeError(type(t))


def _dev(t: torch.Tensor, dtype) -> torch.Tensor:
    assert t.is_cuda and t.dtype == dtype, (t.device, t.dtype, dtype)
    return t


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def make_params(K=8, n_min=1, n_max=4, min_draft=1, max_occ=64, mode=MODE_STRICT, topk=2, p=0.1,
                max_new=0, eos_id=-1, temp_branches=0, tree=0, fused_accept=0) -> Params:
    return Params(K, n_min, n_max, min_draft, max_occ, mode, topk, p, max_new, eos_id, temp_branches, tree, fused_accept)


def version() -> str:
    return lib.laser_version().decode()


def launch_count() -> int:
    return int(lib.laser_launch_count())


# ---- pool ------------------------------------------------------------------------------
class Pool:
    def __init__(self, handle):
        self.handle = handle

    def info(self) -> Dict:
        a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
        _chk(lib.laser_pool_info(self.handle, C.byref(a), C.byref(b), C.byref(c)))
        return dict(n_tokens=a.value, n_keys=b.value, device_bytes=c.value)

    def free(self):
        if self.handle and lib is not None:      # lib is None while the interpreter shuts down
            lib.laser_pool_free(self.handle)
            self.handle = None

    def __del__(self):
        self.free()


def pool_build(tokens, group_offsets: np.ndarray, n_min: int, n_max: int, stream=None) -> Pool:
    """tokens: int32 numpy array (host) or torch CUDA tensor; group_offsets: int64 numpy."""
    if isinstance(tokens, np.ndarray):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    else:
        _dev(tokens, torch.int32)
    offs = np.ascontiguousarray(group_offsets, dtype=np.int64)
    h = C.c_void_p()
    _chk(lib.laser_pool_build(_ptr(tokens), C.c_int64(len(tokens)), _ptr(offs), C.c_int32(len(offs) - 1),
                              C.c_int32(n_min), C.c_int32(n_max), _stream(stream), C.byref(h)))
    return Pool(h)


def draft(pool: Pool, tails, tail_len, group_id, params: Params, draft_out=None, draft_len=None,
          match_n=None, stream=None):
    B = tail_len.shape[0]
    dev = tails.device
    if draft_out is None:
        draft_out = torch.empty(B, params.K, dtype=torch.int32, device=dev)
        draft_len = torch.empty(B, dtype=torch.int32, device=dev)
        match_n = torch.empty(B, dtype=torch.int32, device=dev)
    _chk(lib.laser_draft(pool.handle, _ptr(_dev(tails, torch.int32)), _ptr(_dev(tail_len, torch.int32)),
                         _ptr(_dev(group_id, torch.int32)), C.c_int32(B), C.byref(params),
                         _ptr(draft_out), _ptr(draft_len), _ptr(match_n), _stream(stream)))
    return draft_out, draft_len, match_n


def draft_temp(pool: Pool, tails, tail_len, group_id, hist, hist_len, params: Params, draft_out=None,
               draft_len=None, match_n=None, stream=None):
    """laser_draft_temp: hist int32[B, stride] holds each sequence's own text, hist_len int32[B]."""
    B = tail_len.shape[0]
    dev = tails.device
    if draft_out is None:
        draft_out = torch.empty(B, params.K, dtype=torch.int32, device=dev)
        draft_len = torch.empty(B, dtype=torch.int32, device=dev)
        match_n = torch.empty(B, dtype=torch.int32, device=dev)
    hist = _dev(hist, torch.int32)
    _chk(lib.laser_draft_temp(pool.handle, _ptr(_dev(tails, torch.int32)), _ptr(_dev(tail_len, torch.int32)),
                              _ptr(_dev(group_id, torch.int32)), _ptr(hist), _ptr(_dev(hist_len, torch.int32)),
                              C.c_int64(hist.shape[1] if hist.dim() == 2 else 0), C.c_int32(B), C.byref(params),
                              _ptr(draft_out), _ptr(draft_len), _ptr(match_n), _stream(stream)))
    return draft_out, draft_len, match_n


def draft_tree(pool: Pool, tails, tail_len, group_id, params: Params, hist=None, hist_len=None, stream=None):
    """laser_draft_tree; returns draft, draft_parents, draft_len, match_n (device tensors)."""
    B = tail_len.shape[0]
    dev = tails.device
    draft_out = torch.empty(B, params.K, dtype=torch.int32, device=dev)
    par_out = torch.empty(B, params.K, dtype=torch.int32, device=dev)
    draft_len = torch.empty(B, dtype=torch.int32, device=dev)
    match_n = torch.empty(B, dtype=torch.int32, device=dev)
    stride = 0
    if hist is not None:
        hist, hist_len = _dev(hist, torch.int32), _dev(hist_len, torch.int32)
        stride = hist.shape[1]
    _chk(lib.laser_draft_tree(pool.handle, _ptr(_dev(tails, torch.int32)), _ptr(_dev(tail_len, torch.int32)),
                              _ptr(_dev(group_id, torch.int32)), _ptr(hist), _ptr(hist_len), C.c_int64(stride),
                              C.c_int32(B), C.byref(params), _ptr(draft_out), _ptr(par_out), _ptr(draft_len),
                              _ptr(match_n), _stream(stream)))
    return draft_out, par_out, draft_len, match_n


def make_rows_tree(last_token, draft_t, draft_parents, draft_len, K: int, stream=None):
    B = last_token.shape[0]
    dev = last_token.device
    tokens = torch.empty(B, K + 1, dtype=torch.int32, device=dev)
    parents = torch.empty(B, K + 1, dtype=torch.int32, device=dev)
    n_rows = torch.empty(B, dtype=torch.int32, device=dev)
    _chk(lib.laser_make_rows_tree(_ptr(_dev(last_token, torch.int32)), _ptr(_dev(draft_t, torch.int32)),
                                  _ptr(_dev(draft_parents, torch.int32)), _ptr(_dev(draft_len, torch.int32)),
                                  C.c_int32(B), C.c_int32(K), _ptr(tokens), _ptr(parents), _ptr(n_rows), _stream(stream)))
    return tokens, parents, n_rows


def make_rows(last_token, draft_t, draft_len, K: int, tokens=None, n_rows=None, stream=None):
    B = last_token.shape[0]
    if tokens is None:
        tokens = torch.empty(B, K + 1, dtype=torch.int32, device=last_token.device)
        n_rows = torch.empty(B, dtype=torch.int32, device=last_token.device)
    _chk(lib.laser_make_rows(_ptr(_dev(last_token, torch.int32)), _ptr(_dev(draft_t, torch.int32)),
                             _ptr(_dev(draft_len, torch.int32)), C.c_int32(B), C.c_int32(K),
                             _ptr(tokens), _ptr(n_rows), _stream(stream)))
    return tokens, n_rows


# ---- model / kv --------------------------------------------------------------------------
class Model:
    def __init__(self, handle, cfg: Dict, keep):
        self.handle, self.cfg, self._keep = handle, cfg, keep

    def free(self):
        if self.handle and lib is not None:
            lib.laser_model_free(self.handle)
            self.handle = None

    def __del__(self):
        self.free()


def model_create(cfg: Dict, W: Dict, max_batch: int) -> Model:
    """cfg: dict as synth.model_cfg; W: dict of CUDA bf16 tensors as synth.make_weights."""
    c = ModelCfg(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["n_kv_heads"], cfg["head_dim"],
                 cfg["d_ffn"], cfg["vocab"], cfg["rms_eps"], cfg["rope_theta"], cfg["page_size"],
                 cfg["max_draft"], max_batch, int(cfg.get("precise", 0)))
    L = cfg["n_layers"]

    def arr(name):
        a = (C.c_void_p * max(L, 1))()
        for i, lw in enumerate(W["layers"]):
            t = lw[name]
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
            a[i] = t.data_ptr()
        return a

    arrays = {n: arr(n) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "ffn_norm")}
    for n in ("tok_emb", "lm_head", "final_norm"):
        assert W[n].is_cuda and W[n].dtype == torch.bfloat16 and W[n].is_contiguous()
    w = Weights(W["tok_emb"].data_ptr(), W["lm_head"].data_ptr(), W["final_norm"].data_ptr(),
                *[C.cast(arrays[n], C.POINTER(C.c_void_p)) for n in
                  ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "ffn_norm")])
    h = C.c_void_p()
    _chk(lib.laser_model_create(C.byref(c), C.byref(w), C.byref(h)))
    return Model(h, dict(cfg, max_batch=max_batch), (W, arrays))


class KV:
    def __init__(self, handle, model: Model, max_seqs: int, n_pages: int):
        self.handle, self.model, self.max_seqs, self.n_pages = handle, model, max_seqs, n_pages

    def free(self):
        if self.handle and lib is not None:
            lib.laser_kv_free(self.handle)
            self.handle = None

    def __del__(self):
        self.free()


def kv_create(model: Model, max_seqs: int, n_pages: int) -> KV:
    h = C.c_void_p()
    _chk(lib.laser_kv_create(model.handle, C.c_int32(max_seqs), C.c_int64(n_pages), C.byref(h)))
    return KV(h, model, max_seqs, n_pages)


def kv_set_page_table(kv: KV, table: np.ndarray) -> None:
    t = np.ascontiguousarray(table, dtype=np.int32)
    _chk(lib.laser_kv_set_page_table(kv.handle, _ptr(t)))


def kv_set_len(kv: KV, seq_ids: Sequence[int], lens: Sequence[int], stream=None) -> None:
    s = np.ascontiguousarray(seq_ids, dtype=np.int32)
    l = np.ascontiguousarray(lens, dtype=np.int32)
    _chk(lib.laser_kv_set_len(kv.handle, _ptr(s), _ptr(l), C.c_int32(len(s)), _stream(stream)))


def kv_reset(kv: KV, stream=None) -> None:
    _chk(lib.laser_kv_reset(kv.handle, _stream(stream)))


def kv_set_len_dev(kv: KV, lens_dev: torch.Tensor, stream=None) -> None:
    _chk(lib.laser_kv_set_len_dev(kv.handle, _ptr(_dev(lens_dev, torch.int32)), C.c_int32(lens_dev.numel()),
                                  _stream(stream)))


def kv_get_len(kv: KV, seq_ids: Sequence[int], stream=None) -> np.ndarray:
    s = np.ascontiguousarray(seq_ids, dtype=np.int32)
    out = np.zeros(len(s), dtype=np.int32)
    _chk(lib.laser_kv_get_len(kv.handle, _ptr(s), _ptr(out), C.c_int32(len(s)), _stream(stream)))
    return out


def kv_import(kv: KV, seq: int, layer: int, pos0: int, k: torch.Tensor, v: torch.Tensor, stream=None) -> None:
    _dev(k, torch.bfloat16), _dev(v, torch.bfloat16)
    _chk(lib.laser_kv_import(kv.handle, C.c_int32(seq), C.c_int32(layer), C.c_int32(pos0),
                             C.c_int32(k.shape[0]), _ptr(k), _ptr(v), _stream(stream)))


def kv_export(kv: KV, seq: int, layer: int, pos0: int, n: int, stream=None):
    cfg = kv.model.cfg
    w = cfg["n_kv_heads"] * cfg["head_dim"]
    k = torch.empty(n, w, dtype=torch.bfloat16, device="cuda")
    v = torch.empty(n, w, dtype=torch.bfloat16, device="cuda")
    _chk(lib.laser_kv_export(kv.handle, C.c_int32(seq), C.c_int32(layer), C.c_int32(pos0), C.c_int32(n),
                             _ptr(k), _ptr(v), _stream(stream)))
    return k, v


def verify_step(model: Model, kv: KV, seq_ids, tokens, n_rows, logits=None, stream=None) -> torch.Tensor:
    B = seq_ids.shape[0]
    R = model.cfg["max_draft"] + 1
    assert tokens.shape == (B, R), (tokens.shape, B, R)
    if logits is None:
        logits = torch.empty(B, R, model.cfg["vocab"], dtype=torch.float32, device=tokens.device)
    _chk(lib.laser_verify_step(model.handle, kv.handle, _ptr(_dev(seq_ids, torch.int32)),
                               _ptr(_dev(tokens, torch.int32)), _ptr(_dev(n_rows, torch.int32)),
                               C.c_int32(B), _ptr(_dev(logits, torch.float32)), _stream(stream)))
    return logits


def verify_step_tree(model: Model, kv: KV, seq_ids, tokens, parents, n_rows, logits=None, stream=None) -> torch.Tensor:
    """laser_verify_step_tree: parents int32[B, K+1], parents[b, i] = row of row i's parent."""
    B = seq_ids.shape[0]
    R = model.cfg["max_draft"] + 1
    assert tokens.shape == (B, R) and parents.shape == (B, R), (tokens.shape, parents.shape, B, R)
    if logits is None:
        logits = torch.empty(B, R, model.cfg["vocab"], dtype=torch.float32, device=tokens.device)
    _chk(lib.laser_verify_step_tree(model.handle, kv.handle, _ptr(_dev(seq_ids, torch.int32)),
                                    _ptr(_dev(tokens, torch.int32)), _ptr(_dev(parents, torch.int32)),
                                    _ptr(_dev(n_rows, torch.int32)), C.c_int32(B), _ptr(_dev(logits, torch.float32)),
                                    _stream(stream)))
    return logits


def profile_enable(model: Model, on: bool) -> None:
    _chk(lib.laser_profile_enable(model.handle, C.c_int32(1 if on else 0)))


def profile_read(model: Model, cls: int):
    """Returns (device ms, launches) of class 0 (dense contractions) or 1 (attention)."""
    ms, n = C.c_double(), C.c_int64()
    _chk(lib.laser_profile_read(model.handle, C.c_int32(cls), C.byref(ms), C.byref(n)))
    return ms.value, n.value


def check(model: Model, stream=None) -> None:
    _chk(lib.laser_check(model.handle, _stream(stream)))


def selftest_wait(model: Model, limit_cycles: int, stream=None) -> torch.Tensor:
    report = torch.zeros(4, dtype=torch.int32, device="cuda")
    _chk(lib.laser_selftest_wait(model.handle, C.c_int64(int(limit_cycles)), _ptr(report), _stream(stream)))
    return report


def accept_commit_noalloc(kv: Optional[KV], seq_ids, logits, tokens, n_rows, params: Params, out, stream=None):
    """laser_accept_commit_noalloc: same outputs as accept_commit, no device allocation inside the
    library.  The caller supplies every output tensor: out = (n_accept, out_tokens, n_out)."""
    B, R, V = logits.shape
    n_accept, out_tokens, n_out = out
    _chk(lib.laser_accept_commit_noalloc(kv.handle if kv is not None else C.c_void_p(0),
                                         _ptr(seq_ids) if seq_ids is not None else C.c_void_p(0),
                                         _ptr(_dev(logits, torch.float32)), _ptr(_dev(tokens, torch.int32)),
                                         _ptr(_dev(n_rows, torch.int32)), C.c_int32(B), C.c_int32(V),
                                         C.byref(params), _ptr(n_accept), _ptr(out_tokens), _ptr(n_out),
                                         _stream(stream)))
    return out


def accept_commit(kv: Optional[KV], seq_ids, logits, tokens, n_rows, params: Params, out=None, stream=None):
    B, R, V = logits.shape
    assert R == params.K + 1 and tokens.shape == (B, R)
    if out is None:
        dev = logits.device
        out = (torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, R, dtype=torch.int32, device=dev),
               torch.empty(B, dtype=torch.int32, device=dev))
    n_accept, out_tokens, n_out = out
    _chk(lib.laser_accept_commit(kv.handle if kv is not None else C.c_void_p(0),
                                 _ptr(seq_ids) if seq_ids is not None else C.c_void_p(0),
                                 _ptr(_dev(logits, torch.float32)), _ptr(_dev(tokens, torch.int32)),
                                 _ptr(_dev(n_rows, torch.int32)), C.c_int32(B), C.c_int32(V), C.byref(params),
                                 _ptr(n_accept), _ptr(out_tokens), _ptr(n_out), _stream(stream)))
    return n_accept, out_tokens, n_out


def verify_accept(model: Model, kv: KV, seq_ids, tokens, n_rows, params: Params, commit: bool = True, logits=None, out=None,
                  stream=None):
    """laser_verify_accept: the verify forward with acceptance fused into the LM head; logits (optional, fp32
    [B, K+1, vocab]) are stored only when given.  Returns n_accept, out_tokens, n_out (device tensors)."""
    B = seq_ids.shape[0]
    R = model.cfg["max_draft"] + 1
    assert tokens.shape == (B, R), (tokens.shape, B, R)
    if out is None:
        dev = tokens.device
        out = (torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, R, dtype=torch.int32, device=dev),
               torch.empty(B, dtype=torch.int32, device=dev))
    n_accept, out_tokens, n_out = out
    _chk(lib.laser_verify_accept(model.handle, kv.handle, _ptr(_dev(seq_ids, torch.int32)), _ptr(_dev(tokens, torch.int32)),
                                 _ptr(_dev(n_rows, torch.int32)), C.c_int32(B), C.byref(params), C.c_int32(1 if commit else 0),
                                 _ptr(_dev(logits, torch.float32)) if logits is not None else C.c_void_p(0),
                                 _ptr(n_accept), _ptr(out_tokens), _ptr(n_out), _stream(stream)))
    return n_accept, out_tokens, n_out


def accept_tree(kv: Optional[KV], seq_ids, logits, tokens, parents, n_rows, params: Params, stream=None):
    """laser_accept_tree; returns n_accept, out_tokens, n_out, path_rows (device tensors)."""
    B, R, V = logits.shape
    dev = logits.device
    n_accept = torch.empty(B, dtype=torch.int32, device=dev)
    out_tokens = torch.empty(B, R, dtype=torch.int32, device=dev)
    n_out = torch.empty(B, dtype=torch.int32, device=dev)
    path_rows = torch.empty(B, R, dtype=torch.int32, device=dev)
    _chk(lib.laser_accept_tree(kv.handle if kv is not None else C.c_void_p(0),
                               _ptr(_dev(seq_ids, torch.int32)) if seq_ids is not None else C.c_void_p(0),
                               _ptr(_dev(logits, torch.float32)), _ptr(_dev(tokens, torch.int32)),
                               _ptr(_dev(parents, torch.int32)), _ptr(_dev(n_rows, torch.int32)), C.c_int32(B),
                               C.c_int32(V), C.byref(params), _ptr(n_accept), _ptr(out_tokens), _ptr(n_out),
                               _ptr(path_rows), _stream(stream)))
    return n_accept, out_tokens, n_out, path_rows


def kv_compact_path(kv: KV, seq_ids, path_rows, n_accept, stream=None) -> None:
    """laser_kv_compact_path: path_rows int32[B, stride] as laser_accept_tree writes them."""
    B = n_accept.shape[0]
    _chk(lib.laser_kv_compact_path(kv.handle, _ptr(_dev(seq_ids, torch.int32)), _ptr(_dev(path_rows, torch.int32)),
                                   _ptr(_dev(n_accept, torch.int32)), C.c_int32(B), C.c_int32(path_rows.shape[1]),
                                   _stream(stream)))


def group_kmeans(x: torch.Tensor, centroids: torch.Tensor, iters: int, stream=None):
    """laser_group_kmeans: x fp32 [n, dim], centroids fp32 [k, dim] (updated in place).
    Returns (assign int32[n], counts int32[k])."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 2
    assert centroids.is_cuda and centroids.dtype == torch.float32 and centroids.is_contiguous()
    n, dim = x.shape
    k = centroids.shape[0]
    assign = torch.empty(n, dtype=torch.int32, device=x.device)
    counts = torch.empty(k, dtype=torch.int32, device=x.device)
    _chk(lib.laser_group_kmeans(_ptr(x), C.c_int64(n), C.c_int32(dim), C.c_int32(k), C.c_int32(iters),
                                _ptr(centroids), _ptr(assign), _ptr(counts), _stream(stream)))
    return assign, counts


def generate(model: Model, kv: KV, pool: Optional[Pool], prompts: Sequence[np.ndarray], group_id: Sequence[int],
             params: Params, stream=None) -> Dict:
    B = len(prompts)
    flat = np.ascontiguousarray(np.concatenate([np.asarray(p_, dtype=np.int32) for p_ in prompts]))
    offs = np.zeros(B + 1, dtype=np.int64)
    np.cumsum([len(p_) for p_ in prompts], out=offs[1:])
    gid = np.ascontiguousarray(group_id, dtype=np.int32)
    out = np.full((B, params.max_new), -1, dtype=np.int32)
    out_len = np.zeros(B, dtype=np.int32)
    st = Stats()
    _chk(lib.laser_generate(model.handle, kv.handle, pool.handle if pool is not None else C.c_void_p(0),
                            _ptr(flat), _ptr(offs), _ptr(gid), C.c_int32(B), C.byref(params), _ptr(out),
                            _ptr(out_len), C.byref(st), _stream(stream)))
    return dict(out=[out[b, :out_len[b]].tolist() for b in range(B)], out_len=out_len, **st.as_dict())
