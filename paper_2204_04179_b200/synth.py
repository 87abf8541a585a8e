"""Seeded synthetic inputs for the GRAM training step.

This module holds no arithmetic of the method: it only draws random inputs
(item IDs, item texts, labels, parameter values) and names the shapes of the
workloads.  Both the CPU oracle's tests and the CUDA path's tests call it so
that they see identical inputs.  Everything comes from numpy's Philox
counter-based generator keyed by (seed, stream), so a value depends only on
its seed, stream and index, never on call order.

The inputs stand in for the paper's datasets (Table 3: item pools of 2.6k to
104k, item texts of 5 to 271 tokens, heavy item reuse), which are not
available here.
"""
from __future__ import annotations

from collections import OrderedDict
from dataclasses import dataclass, field, asdict
from typing import Dict

import numpy as np

# stream numbers, one per kind of draw
_S_IDS, _S_PERM, _S_TOKENS, _S_LABELS, _S_PARAMS_CE, _S_PARAMS_TASK, _S_GRAD = 1, 2, 3, 4, 5, 6, 7


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


@dataclass
class GramShape:
    """Shapes of one workload: encoder (CE), task module (CF) and batch."""
    name: str = "tiny"
    dtype: str = "f32"            # arithmetic type of the CUDA path: "f32" or "bf16"
    # item pool and texts
    n_items: int = 200
    l_t: int = 16
    vocab: int = 1000
    zipf_s: float = 1.1
    # content encoder
    d: int = 64
    n_heads: int = 2
    d_ff: int = 256
    n_layers: int = 2
    pooling: str = "mean"         # "mean", "cls" (token 0) or "additive" (additive attention of width d_a over the tokens)
    # task module
    task: str = "kt"              # "kt" (causal attention over a history) or "nr" (additive attention)
    task_layers: int = 1
    task_heads: int = 2
    task_d_ff: int = 256
    task_attn_only: bool = True   # kt: y = x + MHA_causal(x) without LayerNorm/FFN
    d_a: int = 256                # nr: width of the additive-attention query space
    n_cand: int = 0               # nr: candidates per user (first one is the positive)
    # batch
    B: int = 8
    L: int = 20                   # positions per history (nr: history + candidates)
    p_label: float = 0.6
    # multi-step
    K: int = 1

    @property
    def P(self) -> int:
        return self.B * self.L

    def replace(self, **kw) -> "GramShape":
        d = asdict(self)
        d.update(kw)
        return GramShape(**d)


def config(name: str) -> GramShape:
    """The named workloads (seed-generated stand-ins for the paper's tasks)."""
    if name == "tiny":            # tiny Single-step check, fp32
        return GramShape()
    if name == "kt":              # knowledge-tracing shape, BERT-base-shaped encoder, bf16
        return GramShape(name="kt", dtype="bf16", n_items=10_000, l_t=64, vocab=30_522, zipf_s=1.0,
                         d=768, n_heads=12, d_ff=3072, n_layers=12, pooling="cls",
                         task="kt", task_layers=2, task_heads=12, task_d_ff=3072, task_attn_only=False,
                         B=256, L=100, p_label=0.65)
    if name == "nr":              # news-recommendation shape
        return GramShape(name="nr", dtype="bf16", n_items=100_000, l_t=32, vocab=30_522, zipf_s=1.1,
                         d=768, n_heads=12, d_ff=3072, n_layers=12, pooling="cls",
                         task="nr", task_layers=0, d_a=256, n_cand=5, B=64, L=55)
    if name == "kt_multistep":    # Multi-step GRAM on the knowledge-tracing shape
        return config("kt").replace(name="kt_multistep", K=8)
    if name == "nr_additive":     # news recommendation with the paper's item pooling (additive attention over the title tokens)
        return config("nr").replace(name="nr_additive", pooling="additive")
    if name == "nr_mhsa":         # news recommendation with one self-attention layer over the clicked items (Appendix D)
        return config("nr").replace(name="nr_mhsa", task_layers=1, task_heads=12, task_attn_only=True)
    if name == "kt_6l":           # the same with the paper's own encoder depth (Appendix D: a 6-layer, 768-wide model)
        return config("kt").replace(name="kt_6l", n_layers=6)
    raise KeyError(name)


# ---------------------------------------------------------------------------
# item IDs, texts, labels
# ---------------------------------------------------------------------------

def zipf_ids(seed: int, n_items: int, s: float, size: int, step: int = 0) -> np.ndarray:
    """`size` item IDs in [0, n_items): rank r has probability proportional to
    (r+1)^-s; ranks map to IDs through a seeded permutation so the popular
    IDs are not the numerically smallest.  `step` selects an independent batch."""
    w = (np.arange(1, n_items + 1, dtype=np.float64)) ** (-float(s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = _rng(seed, _S_IDS + 1000 * step).random(size)
    ranks = np.minimum(np.searchsorted(cdf, u, side="right"), n_items - 1)
    perm = _rng(seed, _S_PERM).permutation(n_items)
    return perm[ranks].astype(np.int32)


def item_tokens(seed: int, n_items: int, l_t: int, vocab: int) -> np.ndarray:
    """Token IDs of every item's text, uniform over the vocabulary: int32 [n_items, l_t]."""
    return _rng(seed, _S_TOKENS).integers(0, vocab, size=(n_items, l_t), dtype=np.int32)


def item_lengths(seed: int, n_items: int, l_t: int, shortest: int = 1) -> np.ndarray:
    """Text lengths for variable-length items, uniform over shortest..l_t: int32 [n_items] (the paper's texts run
    from 5 to 271 tokens, Table 3); at least one item gets the full l_t and one the shortest length."""
    n = _rng(seed, _S_TOKENS + 7).integers(shortest, l_t + 1, size=n_items, dtype=np.int32)
    n[0] = l_t
    if n_items > 1:
        n[1] = shortest
    return n


def ragged(tokens: np.ndarray, lengths: np.ndarray):
    """The texts without their padding: a list of int32 arrays, item i holding its first lengths[i] tokens."""
    return [np.asarray(tokens[i, :int(lengths[i])]) for i in range(tokens.shape[0])]


def labels(seed: int, B: int, L: int, p: float, step: int = 0) -> np.ndarray:
    """Bernoulli(p) responses, int32 [B, L]."""
    return (_rng(seed, _S_LABELS + 1000 * step).random((B, L)) < p).astype(np.int32)


def position_gradients(seed: int, P: int, d: int) -> np.ndarray:
    """uniform(-1, 1) fp32 [P, d]: stand-in for dL/dE in the kernel sweeps."""
    return _rng(seed, _S_GRAD).uniform(-1.0, 1.0, size=(P, d)).astype(np.float32)


def batch(shape: GramShape, seed: int, step: int = 0):
    """(ids int32 [B, L], labels int32 [B, L]) of one mini-batch."""
    ids = zipf_ids(seed, shape.n_items, shape.zipf_s, shape.P, step).reshape(shape.B, shape.L)
    lab = labels(seed, shape.B, shape.L, shape.p_label, step)
    return ids, lab


# ---------------------------------------------------------------------------
# parameters: ordered name -> fp32 array; the flat layout is the concatenation
# in this order (row-major), which is what the C library's set/get calls use
# ---------------------------------------------------------------------------

def _layer_spec(prefix: str, d: int, d_ff: int, attn_only: bool):
    spec = [(prefix + "wqkv", (3 * d, d)), (prefix + "bqkv", (3 * d,)),
            (prefix + "wo", (d, d)), (prefix + "bo", (d,))]
    if not attn_only:
        spec += [(prefix + "ln1_g", (d,)), (prefix + "ln1_b", (d,)),
                 (prefix + "w1", (d_ff, d)), (prefix + "b1", (d_ff,)),
                 (prefix + "w2", (d, d_ff)), (prefix + "b2", (d,)),
                 (prefix + "ln2_g", (d,)), (prefix + "ln2_b", (d,))]
    return spec


def encoder_param_spec(s: GramShape):
    spec = [("tok_emb", (s.vocab, s.d)), ("pos_emb", (s.l_t, s.d)),
            ("emb_ln_g", (s.d,)), ("emb_ln_b", (s.d,))]
    for l in range(s.n_layers):
        spec += _layer_spec(f"l{l}.", s.d, s.d_ff, False)
    if s.pooling == "additive":          # additive-attention pooling over an item's tokens (width d_a)
        spec += [("pool_wa", (s.d_a, s.d)), ("pool_ba", (s.d_a,)), ("pool_qa", (s.d_a,))]
    return spec


def task_param_spec(s: GramShape):
    if s.task == "kt":
        spec = [("pos", (s.L, s.d)), ("resp", (3, s.d))]
        for l in range(s.task_layers):
            spec += _layer_spec(f"t{l}.", s.d, s.task_d_ff, s.task_attn_only)
        spec += [("head_w", (s.d,)), ("head_b", (1,))]
        return spec
    if s.task == "nr":
        spec = []
        for l in range(s.task_layers):       # self-attention layers over the clicked items, ahead of the additive attention
            spec += _layer_spec(f"t{l}.", s.d, s.task_d_ff, s.task_attn_only)
        return spec + [("wa", (s.d_a, s.d)), ("ba", (s.d_a,)), ("qa", (s.d_a,))]
    raise KeyError(s.task)


def _draw_params(spec, rng, sigma: float, plain: bool) -> "OrderedDict[str, np.ndarray]":
    out: "OrderedDict[str, np.ndarray]" = OrderedDict()
    for name, shp in spec:
        base = name.split(".")[-1]
        z = rng.standard_normal(shp)
        if base.endswith("_g"):                      # LayerNorm gain
            v = np.ones(shp) if plain else 1.0 + 0.1 * z
        elif base.endswith("_b") or base[0] == "b" or base == "head_b":   # LayerNorm shift, biases
            v = np.zeros(shp) if plain else sigma * z
        else:                                        # weights, embeddings
            v = sigma * z
        out[name] = v.astype(np.float32)
    return out


def encoder_params(s: GramShape, seed: int, sigma: float = 0.02, plain: bool = True):
    """Random-init encoder parameters.  plain=True: weights N(0, sigma^2), biases 0,
    LayerNorm gain 1 / shift 0.  plain=False also randomises biases and LayerNorm
    parameters, so that a test exercises every term."""
    return _draw_params(encoder_param_spec(s), _rng(seed, _S_PARAMS_CE), sigma, plain)


def task_params(s: GramShape, seed: int, sigma: float = 0.02, plain: bool = True):
    return _draw_params(task_param_spec(s), _rng(seed, _S_PARAMS_TASK), sigma, plain)


def flatten(params: Dict[str, np.ndarray]) -> np.ndarray:
    return np.concatenate([np.asarray(v, dtype=np.float32).ravel() for v in params.values()])


def unflatten(flat: np.ndarray, spec) -> "OrderedDict[str, np.ndarray]":
    out: "OrderedDict[str, np.ndarray]" = OrderedDict()
    o = 0
    for name, shp in spec:
        n = int(np.prod(shp))
        out[name] = np.asarray(flat[o:o + n]).reshape(shp)
        o += n
    assert o == flat.size, (o, flat.size)
    return out
