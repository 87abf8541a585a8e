"""Runs a few Single-step GRAM steps of a cut-down knowledge-tracing workload: a small case for kernel profilers.

    python -m paper_2204_04179_b200.step_probe [--layers 1] [--batch 16] [--items 2000] [--steps 2]

The encoder keeps the BERT-base layer shape (d = 768, 12 heads, 64-token texts) with `--layers` layers; the batch has
`--batch` histories of 100 positions over `--items` items, so that a step launches every kernel of the full workload
on a few hundred megabytes.  Prints the step report of the last step as one JSON line.
"""
import argparse
import json

import torch

from paper_2204_04179_b200 import binding, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=1)
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--items", type=int, default=2000)
    ap.add_argument("--steps", type=int, default=2)
    ap.add_argument("--seed", type=int, default=0)
    a = ap.parse_args()
    shape = synth.config("kt").replace(n_layers=a.layers, B=a.batch, n_items=a.items)
    ce = synth.encoder_params(shape, a.seed)
    tk = synth.task_params(shape, a.seed)
    toks = synth.item_tokens(a.seed, shape.n_items, shape.l_t, shape.vocab)
    g = binding.Gram(binding.config_from_shape(shape))
    g.set_params(binding.GRAM_MODULE_CE, synth.flatten(ce))
    g.set_params(binding.GRAM_MODULE_TASK, synth.flatten(tk))
    g.set_item_tokens(toks)
    ids, lab = synth.batch(shape, a.seed)
    ids_d, lab_d = torch.from_numpy(ids).to("cuda:0"), torch.from_numpy(lab).to("cuda:0")
    rep = None
    for _ in range(a.steps):
        rep = g.step(ids_d, lab_d, shape.B)
    print(json.dumps(rep.as_dict()))
    g.close()


if __name__ == "__main__":
    main()
