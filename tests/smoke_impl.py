"""One tiny Single-step GRAM step on cuda:0 through the C ABI, checked against the CPU oracle."""
import numpy as np


def run_smoke():
    import torch
    from oracle import gram_oracle as orc
    from paper_2204_04179_b200 import synth
    from tests import gram_helpers as gh

    assert torch.cuda.is_available(), "smoke() needs a CUDA device"
    shape = synth.config("tiny")
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=0)
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab)
    U = len(np.unique(ids))
    assert rep.n_unique == U and rep.n_positions == ids.size
    assert abs(rep.loss - want["loss"]) <= 1e-4 * abs(want["loss"]), (rep.loss, want["loss"])
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    assert e1 <= 1e-3 and e2 <= 1e-3, (e1, n1, e2, n2)
    print(f"smoke ok: loss {rep.loss:.6f} (oracle {want['loss']:.6f}), U={U}, R={rep.boost_ratio:.2f}, "
          f"worst relative gradient error CE {e1:.2e} ({n1}), task {e2:.2e} ({n2})")
    # the same step with bf16 operands: the tensor-core matrix products and attention kernels
    shape16 = shape.replace(dtype="bf16")
    rep, gce, gtk = gh.gpu_single_step(shape16, ce, tk, toks, ids, lab)
    assert abs(rep.loss - want["loss"]) <= 2e-2 * abs(want["loss"]), (rep.loss, want["loss"])
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    assert e1 <= 2e-2 and e2 <= 2e-2, (e1, n1, e2, n2)
    print(f"smoke ok (bf16 operands): loss {rep.loss:.6f}, worst relative gradient error CE {e1:.2e} ({n1}), task {e2:.2e} ({n2})")
