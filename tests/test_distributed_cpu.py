"""The N>1 host logic on CPU: two gloo ranks shard frames, decode nothing, and agree on max-time / sum-work."""
import os
import socket
import subprocess
import sys

import pytest

from paper_2609_16874_b200 import distributed as D

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
from paper_2609_16874_b200 import distributed as D
import numpy as np
from paper_2609_16874_b200 import workloads as wl
import oracle
rank, local, world = D.env_world()
D.init("gloo")
frames = D.frames_for_rank(rank, world, 2)
cfg = wl.scaled(wl.CONFIGS["c1"], H=32, W=32, K=2)
px = 0
sums = []
for f in frames:                      # every rank works on its own frames; nothing is exchanged on the data path
    fr = wl.make_frame(cfg, f)
    res = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, T_v=4, K_max=8)
    px += cfg.pixels
    sums.append(int(res["labels"].sum()))
D.barrier()
t, u = D.reduce_measurement(10.0 * (rank + 1), px)
allf = D.gather_objects({"rank": rank, "frames": frames, "sums": sums})
D.barrier()
if rank == 0:
    print(json.dumps({"t": t, "u": u, "all": allf}))
D.shutdown()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_frames_for_rank_partitions():
    seen = []
    for r in range(4):
        seen += D.frames_for_rank(r, 4, 3)
    assert sorted(seen) == list(range(12))
    with pytest.raises(ValueError):
        D.frames_for_rank(4, 4, 1)


def test_single_process_is_a_no_op():
    assert D.env_world() == (0, 0, 1) or "RANK" in os.environ
    assert D.reduce_measurement(3.0, 7.0) == (3.0, 7.0)
    assert D.gather_objects("x") == ["x"]


def test_two_gloo_ranks_agree_on_max_time_and_total_work(tmp_path):
    port = _free_port()
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["t"] == 20.0                      # max over ranks
    assert res["u"] == 2 * 2 * 32 * 32           # sum over ranks of the pixels processed
    frames = sorted(f for r in res["all"] for f in r["frames"])
    assert frames == [0, 1, 2, 3]
    assert [r["rank"] for r in res["all"]] == [0, 1]
