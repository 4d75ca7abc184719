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
    # vocabulary-parallel plumbing: slice of the vocabulary, all-gather of the per-row partial states
    import torch
    off, width = D.shard_vocab(128256, r)
    mine = torch.full((5, 4), float(r.rank + 1))
    mine[:, 3] = off
    gathered = D.all_gather_partials(r, mine)
    D.barrier(r)
    print(json.dumps({"rank": r.rank, "world": r.world, "lo": shard.start, "hi": shard.stop,
                      "slow": slow, "total": total, "main": r.is_main, "voff": off, "vwidth": width,
                      "gshape": list(gathered.shape), "g0": gathered[0, 0].tolist(), "g1": gathered[1, 4].tolist()}))
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
    assert [(d["voff"], d["vwidth"]) for d in outs] == [(0, 64128), (64128, 64128)]
    for d in outs:                                      # every rank holds every rank's states, in rank order
        assert d["gshape"] == [2, 5, 4] and d["g0"] == [1.0, 1.0, 1.0, 0.0] and d["g1"] == [2.0, 2.0, 2.0, 64128.0]


def test_single_rank_needs_no_process_group():
    from paper_2511_22972_b200 import dist as D
    env = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        r = D.init_from_env("nccl")
        assert (r.rank, r.world, r.backend) == (0, 1, "")
        assert D.max_over_ranks(r, 3.5) == 3.5 and list(D.shard_sequences(5, r)) == [0, 1, 2, 3, 4]
        assert D.shard_vocab(50257, r) == (0, 50257)
        assert [D.shard_vocab(50257, D.Ranks(k, 7, 0, "")) for k in (0, 6)] == [(0, 7184), (43104, 7153)]
        D.barrier(r)
        D.finalize(r)
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v
