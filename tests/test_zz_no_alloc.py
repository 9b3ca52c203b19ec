"""laser_accept_commit_noalloc against laser_accept_commit.

Some programs embedding this library cannot allocate device memory while decoding: an engine
that took all of HBM for its own pools at start-up leaves nothing for cudaMalloc, and an
allocation inside a step would stall the whole device.  For them the library offers an
acceptance call whose scratch is a fixed array inside the library image.  This test drives that
call through the C ABI twice in a row (the array keeps the first call's contents, so the second
call proves the counters are cleared) and requires the very same outputs as the ordinary call -
acceptance is integer work, so the tolerance is exact equality.  It also checks that a call
beyond the fixed capacity is refused instead of overrunning the array.  The file sorts last so
that a stop-at-first-failure run has already covered every other test.
"""
import numpy as np
import pytest
import torch

from helpers import dev_i32, ensure_built
from paper_2408_05676_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def _outs(B, R):
    return (torch.full((B,), -7, dtype=torch.int32, device="cuda"),
            torch.full((B, R), -7, dtype=torch.int32, device="cuda"),
            torch.full((B,), -7, dtype=torch.int32, device="cuda"))


def test_two_calls_in_a_row_match_the_allocating_entry_point(L):
    for (B, K, V, seed, mode) in [(16, 8, 4096, 21, L.MODE_RELAXED), (5, 3, 1001, 22, L.MODE_STRICT)]:
        logits, tokens, n_rows = synth.make_accept_case(B, K, V, seed)
        n_rows[1] = 0
        dl, dt, dn = torch.as_tensor(logits, device="cuda"), dev_i32(tokens), dev_i32(n_rows)
        prm = L.make_params(K=K, mode=mode, topk=2, p=0.1)
        want = [t.cpu().numpy() for t in L.accept_commit(None, None, dl, dt, dn, prm)]
        for call in range(2):
            got = L.accept_commit_noalloc(None, None, dl, dt, dn, prm, _outs(B, K + 1))
            torch.cuda.synchronize()
            for g, w in zip(got, want):
                assert (g.cpu().numpy() == w).all(), (B, K, V, call)
        # a different shape right after reuses the same array
        logits2, tokens2, n_rows2 = synth.make_accept_case(B + 3, K, V, seed + 100)
        dl2, dt2, dn2 = torch.as_tensor(logits2, device="cuda"), dev_i32(tokens2), dev_i32(n_rows2)
        want2 = [t.cpu().numpy() for t in L.accept_commit(None, None, dl2, dt2, dn2, prm)]
        got2 = L.accept_commit_noalloc(None, None, dl2, dt2, dn2, prm, _outs(B + 3, K + 1))
        for g, w in zip(got2, want2):
            assert (g.cpu().numpy() == w).all()


def test_sizes_beyond_the_fixed_array_are_refused(L):
    B, K, V = 1025, 0, 8
    logits = torch.zeros(B, K + 1, V, device="cuda")
    tokens = torch.zeros(B, K + 1, dtype=torch.int32, device="cuda")
    n_rows = torch.ones(B, dtype=torch.int32, device="cuda")
    outs = _outs(B, K + 1)
    with pytest.raises(L.LaserError) as e:
        L.accept_commit_noalloc(None, None, logits, tokens, n_rows, L.make_params(K=K), outs)
    assert e.value.status == -4 and "at most" in str(e.value)
    assert int(outs[0][0]) == -7                      # nothing was launched
    B, K = 600, 31                                     # 19200 rows > 16384
    with pytest.raises(L.LaserError):
        L.accept_commit_noalloc(None, None, torch.zeros(B, K + 1, V, device="cuda"),
                                torch.zeros(B, K + 1, dtype=torch.int32, device="cuda"),
                                torch.ones(B, dtype=torch.int32, device="cuda"), L.make_params(K=K), _outs(B, K + 1))


def test_commit_and_exact_limits(L):
    """With a cache handle the call also advances the committed lengths, exactly as the allocating call
    does; and the two stated limits themselves (1024 sequences; 16384 rows) are accepted."""
    cfg = synth.model_cfg("tiny")
    from helpers import weights_to
    m = L.model_create(cfg, weights_to(synth.make_weights(cfg, seed=0), "cuda"), max_batch=8)
    kv = L.kv_create(m, 8, 8 * 8)
    B, K, V = 8, 8, cfg["vocab"]
    logits, tokens, n_rows = synth.make_accept_case(B, K, V, 31)
    dl, dt, dn = torch.as_tensor(logits, device="cuda"), dev_i32(tokens), dev_i32(n_rows)
    ids = torch.arange(B, dtype=torch.int32, device="cuda")
    prm = L.make_params(K=K, mode=L.MODE_STRICT)
    L.kv_set_len(kv, list(range(B)), [5] * B)
    want = [t.cpu().numpy() for t in L.accept_commit(kv, ids, dl, dt, dn, prm)]
    want_len = L.kv_get_len(kv, list(range(B)))
    for call in range(2):
        L.kv_set_len(kv, list(range(B)), [5] * B)
        got = L.accept_commit_noalloc(kv, ids, dl, dt, dn, prm, _outs(B, K + 1))
        torch.cuda.synchronize()
        for g, w in zip(got, want):
            assert (g.cpu().numpy() == w).all()
        assert (L.kv_get_len(kv, list(range(B))) == want_len).all() and (want_len == 5 + want[2]).all()
    for (B, K) in ((1024, 0), (1024, 15)):              # 1024 sequences; 1024 * 16 = 16384 rows
        V = 64
        logits, tokens, n_rows = synth.make_accept_case(B, K, V, 40 + K)
        dl, dt, dn = torch.as_tensor(logits, device="cuda"), dev_i32(tokens), dev_i32(n_rows)
        prm = L.make_params(K=K, mode=L.MODE_RELAXED, topk=2, p=0.05)
        want = [t.cpu().numpy() for t in L.accept_commit(None, None, dl, dt, dn, prm)]
        got = L.accept_commit_noalloc(None, None, dl, dt, dn, prm, _outs(B, K + 1))
        for g, w in zip(got, want):
            assert (g.cpu().numpy() == w).all()
