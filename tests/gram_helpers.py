"""Shared helpers of the GPU parity tests: run the CUDA library on seeded inputs and compare with the oracle."""
from collections import OrderedDict

import numpy as np
import torch

from paper_2204_04179_b200 import binding, synth

DEV = "cuda:0"


def make_inputs(shape, seed=0, sigma=0.1, plain=False):
    ce = synth.encoder_params(shape, seed, sigma=sigma, plain=plain)
    tk = synth.task_params(shape, seed, sigma=sigma, plain=plain)
    toks = synth.item_tokens(seed, shape.n_items, shape.l_t, shape.vocab)
    ids, lab = synth.batch(shape, seed)
    return ce, tk, toks, ids, lab


def make_ctx(shape, ce, tk, toks, **over):
    g = binding.Gram(binding.config_from_shape(shape, **over))
    g.set_params(binding.GRAM_MODULE_CE, synth.flatten(ce))
    g.set_params(binding.GRAM_MODULE_TASK, synth.flatten(tk))
    g.set_item_tokens(toks)
    return g


def gpu_grads(g, shape):
    gce = synth.unflatten(g.get_grads(binding.GRAM_MODULE_CE), synth.encoder_param_spec(shape))
    gtk = synth.unflatten(g.get_grads(binding.GRAM_MODULE_TASK), synth.task_param_spec(shape))
    return gce, gtk


def gpu_single_step(shape, ce, tk, toks, ids, lab, host=False, **over):
    g = make_ctx(shape, ce, tk, toks, **over)
    if host:
        rep = g.step_host(np.ascontiguousarray(ids, np.int32), np.ascontiguousarray(lab, np.int32), ids.shape[0])
    else:
        rep = g.step(torch.from_numpy(np.ascontiguousarray(ids, np.int32)).to(DEV),
                     torch.from_numpy(np.ascontiguousarray(lab, np.int32)).to(DEV), ids.shape[0])
    gce, gtk = gpu_grads(g, shape)
    g.close()
    return rep, gce, gtk


def rel_err(got, want):
    """max |got - want| / max |want| over one parameter tensor."""
    want = np.asarray(want, np.float64)
    return float(np.abs(np.asarray(got, np.float64) - want).max() / (np.abs(want).max() + 1e-30))


def worst_rel_err(got: dict, want: dict):
    worst, name = 0.0, None
    for k in want:
        if np.abs(want[k]).max() == 0:
            assert np.abs(got[k]).max() < 1e-6, k
            continue
        e = rel_err(got[k], want[k])
        if e > worst:
            worst, name = e, k
    return worst, name
