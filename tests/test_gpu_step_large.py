"""Full-size models (BERT-base-shaped encoder, bf16) on a sub-batch the oracle finishes in about a minute."""
import time

import numpy as np
import pytest
import torch

from oracle import gram_oracle as orc
from paper_2204_04179_b200 import binding, synth
from tests import gram_helpers as gh

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,B,L,n_items", [("kt", 2, 20, 24), ("nr", 2, 15, 20)])
def test_bert_base_shape_sub_batch(name, B, L, n_items):
    # the named configuration with its own initialisation (weights N(0, 0.02^2), biases 0, LayerNorm 1/0),
    # a smaller item pool and batch so that the per-occurrence oracle stays affordable
    shape = synth.config(name).replace(B=B, L=L, n_items=n_items, vocab=2000)
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=17, sigma=0.02, plain=True)
    t0 = time.time()
    torch.set_num_threads(max(1, torch.get_num_threads()))
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    t_oracle = time.time() - t0
    rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab)
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    errs = sorted((gh.rel_err(gce[k], want["grad_ce"][k]) for k in gce if np.abs(want["grad_ce"][k]).max() > 0))
    print(f"{name}: P={ids.size} U={rep.n_unique} oracle {t_oracle:.1f}s loss gpu {rep.loss:.5f} oracle {want['loss']:.5f}; "
          f"worst CE {e1:.4f} ({n1}) median {errs[len(errs)//2]:.4f}; worst task {e2:.4f} ({n2})")
    assert abs(rep.loss - want["loss"]) <= 2e-2 * abs(want["loss"])
    assert e1 <= 2e-2, (n1, e1)
    assert e2 <= 2e-2, (n2, e2)
