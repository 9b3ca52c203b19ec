"""Failure detection on the device without faulting or hanging anything: a bounded wait is made to run
out on purpose (a barrier nobody arrives on, 2e6 cycles = about a millisecond), the status word must
report LASER_ERR_TIMEOUT through laser_check exactly once, the producer role must have drained its copy,
and the same model must then run a normal verify step with the same result as before."""
import numpy as np
import pytest
import torch

from helpers import dev_i32, ensure_built, weights_to
from paper_2408_05676_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def test_a_wait_that_runs_out_is_reported_and_the_library_keeps_working(L):
    cfg = synth.model_cfg("tiny")
    m = L.model_create(cfg, weights_to(synth.make_weights(cfg, seed=0), "cuda"), max_batch=4)
    kv = L.kv_create(m, 4, 4 * 8)
    ids = torch.arange(4, dtype=torch.int32, device="cuda")
    tokens = dev_i32(np.random.default_rng(1).integers(0, cfg["vocab"], size=(4, 9)))
    n_rows = dev_i32([9, 3, 0, 9])
    before = L.verify_step(m, kv, ids, tokens, n_rows).clone()
    L.check(m)
    limit = 2_000_000
    report = L.selftest_wait(m, limit).cpu().numpy()
    assert report[0] == 1, "the starved wait must give up"
    assert report[1] == 1, "the abort flag must reach the producer role"
    assert report[2] == 1, "the producer must see its copy land before the CTA exits"
    assert limit <= report[3] < 50 * limit, report[3]
    with pytest.raises(L.LaserError) as e:
        L.check(m)
    assert e.value.status == -5 and "wait ran out" in str(e.value)
    L.check(m)                                    # reported once, then clear
    after = L.verify_step(m, kv, ids, tokens, n_rows)
    L.check(m)
    assert torch.equal(before[0], after[0]) and torch.equal(before[3], after[3]) and torch.equal(before[1, :3], after[1, :3])
    with pytest.raises(L.LaserError):
        L.selftest_wait(m, 10)                    # limits outside [1e3, 2e9] are refused on the host
