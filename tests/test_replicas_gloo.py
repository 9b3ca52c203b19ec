"""The N > 1 path of the benchmark on CPU: two gloo ranks, per-rank figures reduced to the
whole-job time (max) and token count (sum); group sharding covers every group once."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2408_05676_b200 import replicas
    dist, r, w = replicas.init("gloo")
    assert (r, w) == (rank, world)
    replicas.barrier(dist)
    ms, tokens = replicas.reduce_step(dist, 5.0 + 2.0 * rank, 56 + rank)
    groups = list(replicas.shard_groups(11, r, w))
    out.put((rank, ms, tokens, groups))
    replicas.barrier(dist)
    dist.destroy_process_group()


def test_two_ranks_reduce_and_shard():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [7.0, 7.0]            # max over ranks
    assert [r[2] for r in res] == [113, 113]            # sum over ranks
    assert sorted(res[0][3] + res[1][3]) == list(range(11)) and abs(len(res[0][3]) - len(res[1][3])) <= 1


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    os.environ.pop("WORLD_SIZE", None)
    from paper_2408_05676_b200 import replicas
    dist, r, w = replicas.init()
    assert dist is None and (r, w) == (0, 1)
    assert replicas.reduce_step(None, 3.5, 9) == (3.5, 9)
    assert list(replicas.shard_groups(5, 0, 1)) == [0, 1, 2, 3, 4]


def test_launcher_starts_n_ranks_and_reports_failures():
    """The spawn path behind `bench.py --gpus N`: two ranks of a stub workload on CPU (gloo)."""
    import json
    import subprocess
    code = ("import sys; sys.path.insert(0, %r); from paper_2408_05676_b200 import replicas; "
            "sys.exit(replicas.launch_local([sys.executable, '-m', 'paper_2408_05676_b200.replicas', '--stub-workload'] + sys.argv[1:], 2, timeout=120))" % ROOT)
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, cwd=ROOT, timeout=180)
    assert r.returncode == 0, r.stderr
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["ranks_seen"] == 2 and line["ms"] == 4.0 and line["tokens"] == 100
    assert line["groups_rank0"] == [0, 1, 2, 3, 4]
    # a rank that exits with an error ends the job with a non-zero code instead of leaving the other waiting
    r = subprocess.run([sys.executable, "-c", code, "--fail-rank", "1"], capture_output=True, text=True, cwd=ROOT, timeout=180)
    assert r.returncode != 0
