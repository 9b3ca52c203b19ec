"""laser_accept_commit against the acceptance oracle: bit-exact on synthesised logits that
reach every branch of Eq. 4 / Eq. 7 / Eq. 8, ties and ragged row counts included."""
import numpy as np
import pytest
import torch

from helpers import dev_i32, ensure_built
from oracle import accept as A
from paper_2408_05676_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def _run(L, logits, tokens, n_rows, mode, k, p):
    prm = L.make_params(K=logits.shape[1] - 1, mode=mode, topk=k, p=p)
    out = L.accept_commit(None, None, torch.as_tensor(logits, device="cuda"), dev_i32(tokens), dev_i32(n_rows), prm)
    torch.cuda.synchronize()
    return [o.cpu().numpy() for o in out], float(np.float32(p))


@pytest.mark.parametrize("B,K,V,seed", [(24, 8, 4096, 3), (7, 16, 32000, 4), (5, 3, 1001, 5), (64, 1, 257, 6), (3, 0, 64, 7)])
def test_matches_oracle_all_modes(L, B, K, V, seed):
    logits, tokens, n_rows = synth.make_accept_case(B, K, V, seed)
    n_rows[0] = 0 if B > 3 else n_rows[0]
    n_threshold_ties = 0
    for mode, k, p in [(A.STRICT, 1, 0.0), (A.RELAXED, 2, 0.1), (A.RELAXED, 3, 0.3), (A.RELAXED, 1, 0.0),
                       (A.TOPK, 2, 0.0), (A.TOPP, 1, 0.1), (A.RELAXED, 2, 1.0), (A.RELAXED_ARGMAX, 2, 0.1),
                       (A.RELAXED_ARGMAX, 3, 0.3)]:
        got, p32 = _run(L, logits, tokens, n_rows, mode, k, p)
        want = A.accept_batch(logits, tokens, n_rows, mode, k, p32)
        for g, w, name in zip(got, want, ("n_accept", "out_tokens", "n_out")):
            if not (g == w).all():
                # only a probability within 1e-9 (relative) of p may differ: fp64 summation order
                bad = np.nonzero((got[0] != want[0]))[0]
                for b in bad:
                    a = min(got[0][b], want[0][b])
                    q = A.prob_of(logits[b, a], int(tokens[b, a + 1]))
                    assert abs(q - p32) <= 1e-9 * p32, (name, mode, k, p, b)
                    n_threshold_ties += 1
                break
    assert n_threshold_ties == 0


def test_commit_advances_cache_length_and_calls_repeat(L):
    # a tiny model only to own a cache; acceptance itself needs none
    cfg = synth.model_cfg("tiny", n_layers=1, d_model=64, n_heads=2, n_kv_heads=2, head_dim=32, d_ffn=64,
                          vocab=512, max_draft=4)
    from helpers import weights_to
    W = weights_to(synth.make_weights(cfg, 1), "cuda")
    m = L.model_create(cfg, W, max_batch=8)
    kv = L.kv_create(m, 8, 64)
    logits, tokens, n_rows = synth.make_accept_case(6, 4, 512, 11)
    seq_ids = np.asarray([5, 0, 3, 1, 7, 2], np.int32)
    L.kv_set_len(kv, list(range(8)), [10, 11, 12, 13, 14, 15, 16, 17])
    prm = L.make_params(K=4, mode=A.RELAXED, topk=2, p=0.1)
    want = A.accept_batch(logits, tokens, n_rows, A.RELAXED, 2, float(np.float32(0.1)))
    dl, dt, dn, ds = torch.as_tensor(logits, device="cuda"), dev_i32(tokens), dev_i32(n_rows), dev_i32(seq_ids)
    for rep in range(3):      # scratch counters must return to zero between calls
        got = L.accept_commit(kv, ds, dl, dt, dn, prm)
        for g, w in zip(got, want):
            assert (g.cpu().numpy() == w).all()
    lens = L.kv_get_len(kv, list(range(8)))
    exp = np.asarray([10, 11, 12, 13, 14, 15, 16, 17])
    exp[seq_ids] += 3 * want[2]
    assert (lens == exp).all()
    L.kv_reset(kv)                      # every committed length back to zero
    assert (L.kv_get_len(kv, list(range(8))) == 0).all()


def test_rejects_bad_arguments(L):
    logits, tokens, n_rows = synth.make_accept_case(2, 2, 16, 1)
    with pytest.raises(L.LaserError) as e:
        L.accept_commit(None, None, torch.as_tensor(logits, device="cuda"), dev_i32(tokens), dev_i32(n_rows),
                        L.make_params(K=2, mode=9))
    assert e.value.status == -1
