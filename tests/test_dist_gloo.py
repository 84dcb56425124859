"""The multi-GPU plumbing (frame sharding, barrier, max-over-ranks timing) on CPU: two gloo
ranks started as child processes.  The forward itself has no collective, so this is all the
N > 1 path adds."""
import os
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch
    from paper_1706_09453_b200 import dist as D, workloads as wl
    rank, world, _ = D.env_world()
    dist = D.init("gloo")
    assert dist is not None and dist.get_world_size() == 2
    cfg = wl.CONFIGS["tiny"]
    X = wl.make_frames(cfg, 8, seed=D.frames_seed(cfg.seed, rank))
    D.barrier(dist)
    ms = D.max_over_ranks(dist, 10.0 + 5.0 * rank)          # rank 1 is the slow one
    # gather a fingerprint of every rank's batch to check the shards differ
    fp = torch.tensor([float(X.sum())], dtype=torch.float64)
    fps = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(fps, fp)
    lo, hi = D.shard_bounds(101, rank, world)
    print(json.dumps({"rank": rank, "ms": ms, "fps": [float(f) for f in fps], "lo": lo, "hi": hi,
                      "rate": D.aggregate_rate(8, world, 3, ms)}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks():
    import json
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda r: r["rank"])
    assert outs[0]["ms"] == outs[1]["ms"] == 15.0                      # MAX over ranks
    assert outs[0]["fps"] == outs[1]["fps"] and outs[0]["fps"][0] != outs[0]["fps"][1]   # distinct batches
    assert (outs[0]["lo"], outs[0]["hi"], outs[1]["lo"], outs[1]["hi"]) == (0, 51, 51, 101)
    assert np.isclose(outs[0]["rate"], 2 * 8 * 3 / 15e-3)


def test_shard_bounds_cover_everything_once():
    from paper_1706_09453_b200 import dist as D
    for total in (1, 7, 8192, 65537):
        for world in (1, 2, 3, 8):
            b = [D.shard_bounds(total, r, world) for r in range(world)]
            assert b[0][0] == 0 and b[-1][1] == total
            assert all(b[i][1] == b[i + 1][0] for i in range(world - 1))
            assert max(h - l for l, h in b) - min(h - l for l, h in b) <= 1
