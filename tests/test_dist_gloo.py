"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks shard the batch
without overlap, and the job time is the slowest rank's."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, sys
    sys.path.insert(0, %r)
    from paper_2511_22972_b200 import dist as D
    r = D.init_from_env("gloo")
    D.barrier(r)
    shard = D.shard_sequences(37, r)
    slow = D.max_over_ranks(r, 10.0 + 5.0 * r.rank)
    total = D.sum_over_ranks(r, len(shard))
    D.barrier(r)
    print(json.dumps({"rank": r.rank, "world": r.world, "lo": shard.start, "hi": shard.stop,
                      "slow": slow, "total": total, "main": r.is_main}))
    D.finalize(r)
""") % ROOT


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_shard_and_reduce():
    import json
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert [d["world"] for d in outs] == [2, 2]
    assert (outs[0]["lo"], outs[0]["hi"], outs[1]["lo"], outs[1]["hi"]) == (0, 19, 19, 37)
    assert all(d["slow"] == 15.0 for d in outs)         # max over ranks, seen by every rank
    assert all(d["total"] == 37.0 for d in outs)
    assert outs[0]["main"] and not outs[1]["main"]


def test_single_rank_needs_no_process_group():
    from paper_2511_22972_b200 import dist as D
    env = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        r = D.init_from_env("nccl")
        assert (r.rank, r.world, r.backend) == (0, 1, "")
        assert D.max_over_ranks(r, 3.5) == 3.5 and list(D.shard_sequences(5, r)) == [0, 1, 2, 3, 4]
        D.barrier(r)
        D.finalize(r)
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v
