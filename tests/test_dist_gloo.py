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
# data-parallel gradients: every rank differentiates the loss of ITS histories (a mean over its own predictions);
# after the weighted all-reduce both hold the gradient of the whole batch
import torch
shape2 = synth.GramShape(name="s", n_items=9, l_t=4, vocab=20, d=16, n_heads=2, d_ff=32, n_layers=1, pooling="cls", task="kt",
                         task_layers=1, task_heads=2, task_d_ff=32, task_attn_only=False, B=5, L=6, zipf_s=1.1)
ce = synth.encoder_params(shape2, 3, sigma=0.3, plain=False); tk = synth.task_params(shape2, 3, sigma=0.3, plain=False)
toks = synth.item_tokens(3, shape2.n_items, shape2.l_t, shape2.vocab)
ids2, lab2 = synth.batch(shape2, 3)
lab2 = lab2.copy(); lab2[4, 3:] = -1                  # the last history ends in padding: 3 predictions instead of 6
s_ids, s_lab = gdist.shard_batch(ids2, lab2, rank, 2) # 3 histories on rank 0 (18 predictions), 2 on rank 1 (9 predictions)
r = orc.e2e_step(shape2.replace(B=s_ids.shape[0]), ce, tk, toks, s_ids, s_lab)
grads = [torch.tensor(v) for v in list(r["grad_ce"].values()) + list(r["grad_task"].values())]
n_pred = gdist.n_predictions(shape2, s_lab)
total = gdist.allreduce_weighted_mean(grads, n_pred, dist)
names = list(r["grad_ce"]) + list(r["grad_task"])
out["n_pred"] = n_pred; out["total_pred"] = total
out["grads"] = {n: t.numpy().tolist() for n, t in zip(names, grads) if n in ("l0.w1", "head_w", "pos", "tok_emb")}
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
    # the averaged gradients equal end-to-end training on the whole batch (Eq. 8's mean runs over all predictions)
    from oracle import gram_oracle as orc
    shape2 = synth.GramShape(name="s", n_items=9, l_t=4, vocab=20, d=16, n_heads=2, d_ff=32, n_layers=1, pooling="cls", task="kt",
                             task_layers=1, task_heads=2, task_d_ff=32, task_attn_only=False, B=5, L=6, zipf_s=1.1)
    ce = synth.encoder_params(shape2, 3, sigma=0.3, plain=False); tk = synth.task_params(shape2, 3, sigma=0.3, plain=False)
    toks = synth.item_tokens(3, shape2.n_items, shape2.l_t, shape2.vocab)
    ids2, lab2 = synth.batch(shape2, 3)
    lab2 = lab2.copy(); lab2[4, 3:] = -1
    whole = orc.e2e_step(shape2, ce, tk, toks, ids2, lab2)
    assert (res[0]["n_pred"], res[1]["n_pred"]) == (18, 9) and res[0]["total_pred"] == 27.0
    for r in (0, 1):
        for name, got in res[r]["grads"].items():
            want = whole["grad_ce"][name] if name in whole["grad_ce"] else whole["grad_task"][name]
            assert np.abs(np.array(got) - want).max() <= 1e-12 * max(1.0, np.abs(want).max()), (r, name)
    # an unweighted mean of the two ranks' gradients would be wrong here: the shards hold 18 and 9 predictions
    plain = orc.e2e_step(shape2.replace(B=3), ce, tk, toks, ids2[:3], lab2[:3])
    other = orc.e2e_step(shape2.replace(B=2), ce, tk, toks, ids2[3:], lab2[3:])
    naive = 0.5 * (plain["grad_task"]["head_w"] + other["grad_task"]["head_w"])
    assert np.abs(naive - whole["grad_task"]["head_w"]).max() > 1e-6
