"""The N>1 host logic on two CPU processes (gloo): sharding of histories, slowest-rank time, job throughput."""
import os
import subprocess
import sys

import numpy as np

from paper_2204_04179_b200 import dist as gdist
from paper_2204_04179_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import numpy as np
import torch.distributed as dist
from paper_2204_04179_b200 import dist as gdist, synth
from oracle import gram_oracle as orc
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%s" %% os.environ["PORT"], rank=int(os.environ["RANK"]), world_size=2)
rank = dist.get_rank()
shape = synth.config("tiny").replace(B=5, L=6)
ids, lab = synth.batch(shape, 3)                      # one global batch, split by histories
my_ids, my_lab = gdist.shard_batch(ids, lab, rank, 2)
# each rank dedups its own shard: local unique counts, no exchange
U = len(orc.unique_inverse(my_ids)[0])
ms = 10.0 + 5.0 * rank                                # rank 1 is the slow one
out = dict(rank=rank, rows=int(my_ids.shape[0]), U=U, ids=my_ids.tolist(),
           ms_max=gdist.max_over_ranks(ms, dist), total=gdist.sum_over_ranks(my_ids.size, dist),
           thr=gdist.job_throughput(my_ids.size, ms, dist),
           seed=gdist.rank_seed(3, rank))
print("RESULT " + json.dumps(out), flush=True)
dist.barrier()
dist.destroy_process_group()
""" % ROOT


def test_history_shards_cover_the_batch_once():
    for n in (1, 2, 5, 256, 257):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                s = gdist.history_shard(n, r, world)
                got += list(range(n))[s]
            assert got == list(range(n))
            sizes = [len(range(n)[gdist.history_shard(n, r, world)]) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_over_gloo():
    import json
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), PORT=str(port), OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    res = {}
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        line = [l for l in out.splitlines() if l.startswith("RESULT ")][0]
        d = json.loads(line[7:])
        res[d["rank"]] = d
    shape = synth.config("tiny").replace(B=5, L=6)
    ids, _ = synth.batch(shape, 3)
    assert res[0]["rows"] == 3 and res[1]["rows"] == 2
    assert np.array_equal(np.array(res[0]["ids"] + res[1]["ids"]), ids)          # disjoint, complete, in order
    for r in (0, 1):
        assert res[r]["ms_max"] == 15.0 and res[r]["total"] == 30.0
        assert abs(res[r]["thr"] - 30.0 / 0.015) < 1e-9
    assert res[0]["seed"] != res[1]["seed"]
    assert res[0]["U"] == len(np.unique(ids[:3])) and res[1]["U"] == len(np.unique(ids[3:]))
