"""CPU oracle for the GRAM training step.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA library must compute.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
it; the product path never does, and it shares no code with the CUDA sources.

What it states, and from where in the paper:

* `e2e_step`: standard end-to-end training (Section 3.3): the content encoder
  CE runs once per *interaction* (every occurrence of an item, duplicates
  included), the task module CF consumes the encodings, and the loss is
  back-propagated through every one of those encoder calls; parameter gradients
  sum over occurrences.  Single-step GRAM reaches exactly this gradient by a
  cheaper route (Proposition, Section 4.1), so this definition is its oracle.
* `gram_single_step`: the route itself (Algorithm 1 with N = 1): encode the
  unique items once (Eq. 4), task forward/backward (Eq. 5), sum dL/dh over the
  occurrences of each item (Eq. 6 with SGD of learning rate 1 makes
  h - h~ equal to that sum), and one encoder VJP per unique item (Eq. 7).
  It exists to check the Proposition on the oracle itself.
* `multistep_window`: Algorithm 1 with N = K > 1, step by step.  The paper
  states that this is not equivalent to end-to-end training, so there is no
  plain definition to reduce to; the readings taken where the algorithm is
  silent are listed in the function's docstring.
* `multistep_window_pseudo_target`: the same window under the trainable-embedding
  reading of Section 4.3 (the task module keeps using the modified embedding
  h~, the encoder regresses towards it with the pseudo-loss of Eq. 9).
* `unique_inverse_bruteforce`, `unique_inverse`, `segment_sum`,
  `table_accumulate`: the index work and the per-item sums on their own.
* `boost_ratio`: the speed-boost ratio R (Section 4.4).
* `noam_rate`, `adam_update`, `train_steps_adam`: the optimiser of Appendix D
  (experiment details): Adam with the Noam learning-rate scheme, written
  from the two published definitions; `train_steps_adam` applies it to the
  end-to-end gradients of successive batches.

Arithmetic is float64 throughout unless a caller passes another dtype: the
paper never fixes a precision.  Derivatives of the end-to-end definition come
from torch's autograd over the plain forward written here; the tests pin that
combination with central finite differences and closed forms.

Pins (tests/test_oracle_*.py): brute force on tiny inputs, the worked count
of Fig. 1, finite differences on a 1-layer encoder, closed forms of softmax /
LayerNorm / GELU, the task module's pieces one by one (`kt_logits`: no label
leak and the one-position closed form; `bce_with_logits_sum` and
`softmax_ce_first`: the library losses at random logits; `nr_user_vector`:
mean at q = 0, a one-click history, the library softmax; each with planted
mistakes that must fail), the Proposition (e2e == single-step), the pseudo-loss
identity (Eqs. 1-3), K = 1 reducing to single-step, and conservation of
column sums; for the trainable-embedding window, torch.optim.SGD(lr=1) on an
embedding parameter, finite differences of the pseudo-loss with a stale cache,
and K = 1 with a fresh cache reducing to end-to-end training; for the optimiser, torch.optim.Adam at a constant rate, the closed
form of the first step, and the closed-form values of the Noam curve.  The
Multi-step *trajectory* beyond those is pinned only by the readings below:
parity unpinned by the paper for that part.
"""
from __future__ import annotations

import math
from collections import OrderedDict
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

LN_EPS = 1e-5


# ---------------------------------------------------------------------------
# index work: the unique-item set B_I of a mini-batch (Table 1) and the map
# from occurrences to items that Fig. 1 draws
# ---------------------------------------------------------------------------

def unique_inverse_bruteforce(ids) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """O(P*U) scan, for tiny inputs.  Returns
    unique   ascending distinct IDs                                  [U]
    inverse  unique[inverse[p]] == ids[p]                            [P]
    perm     positions grouped by item, ascending inside each group  [P]
    seg_off  group u is perm[seg_off[u]:seg_off[u+1]]                [U+1]
    """
    ids = [int(v) for v in np.asarray(ids).ravel()]
    unique: List[int] = []
    for v in ids:
        if v not in unique:
            unique.append(v)
    # ascending order by repeated minimum selection
    ordered: List[int] = []
    rest = list(unique)
    while rest:
        m = min(rest)
        ordered.append(m)
        rest.remove(m)
    inverse = [ordered.index(v) for v in ids]
    perm: List[int] = []
    seg_off = [0]
    for u in range(len(ordered)):
        for p, v in enumerate(ids):
            if v == ordered[u]:
                perm.append(p)
        seg_off.append(len(perm))
    i32 = np.int32
    return (np.array(ordered, i32), np.array(inverse, i32), np.array(perm, i32), np.array(seg_off, i32))


def unique_inverse(ids) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Same result at any size: a library stable sort, then one scan."""
    ids = np.asarray(ids).ravel().astype(np.int64)
    P = ids.size
    perm = np.argsort(ids, kind="stable")
    sk = ids[perm]
    head = np.ones(P, dtype=bool)
    head[1:] = sk[1:] != sk[:-1]
    starts = np.nonzero(head)[0]
    unique = sk[starts]
    seg_off = np.concatenate([starts, [P]])
    seg_of_sorted = np.cumsum(head) - 1
    inverse = np.empty(P, dtype=np.int64)
    inverse[perm] = seg_of_sorted
    i32 = np.int32
    return unique.astype(i32), inverse.astype(i32), perm.astype(i32), seg_off.astype(i32)


def boost_ratio(n_interactions: int, n_items: int) -> float:
    """R = #interactions / #items (Section 4.4)."""
    return float(n_interactions) / float(n_items)


def segment_sum(dE, perm, seg_off) -> np.ndarray:
    """G[u, :] = sum of dE[perm[j], :] over j in [seg_off[u], seg_off[u+1]), in
    float64, rows added in ascending j (Eq. 6: every occurrence of item u
    contributes its gradient to the one pseudo-target of u)."""
    dE = np.asarray(dE, dtype=np.float64)
    U = len(seg_off) - 1
    G = np.zeros((U, dE.shape[1]), dtype=np.float64)
    for u in range(U):
        for j in range(int(seg_off[u]), int(seg_off[u + 1])):
            G[u, :] += dE[int(perm[j]), :]
    return G


def table_accumulate(table, touched, dE, ids) -> None:
    """Multi-step accumulation in place: table[ids[p], :] += dE[p, :] for p in
    ascending order, touched[ids[p]] = True (Section 4.2: gradient buffers are
    kept per item across several mini-batches)."""
    dE = np.asarray(dE, dtype=np.float64)
    for p, i in enumerate(np.asarray(ids).ravel()):
        table[int(i), :] += dE[p, :]
        touched[int(i)] = True


# ---------------------------------------------------------------------------
# the two modules.  CE: a BERT-shaped post-LayerNorm transformer over one
# item's tokens (Appendix D: MHSA layers of width 768; mean pooling for KT).
# CF: the task module over a history of encodings (Section 3.1).
# ---------------------------------------------------------------------------

def layer_norm(x: torch.Tensor, g: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    mu = x.mean(dim=-1, keepdim=True)
    var = ((x - mu) ** 2).mean(dim=-1, keepdim=True)
    return (x - mu) / torch.sqrt(var + LN_EPS) * g + b


def gelu(x: torch.Tensor) -> torch.Tensor:
    return 0.5 * x * (1.0 + torch.erf(x / math.sqrt(2.0)))


def softmax_rows(s: torch.Tensor) -> torch.Tensor:
    e = torch.exp(s - s.max(dim=-1, keepdim=True).values)
    return e / e.sum(dim=-1, keepdim=True)


def attention(x: torch.Tensor, th: Dict[str, torch.Tensor], pre: str, n_heads: int, causal: bool) -> torch.Tensor:
    """Multi-head self-attention over one sequence x [S, d], output projection
    included.  Rows 0..d-1 of wqkv give Q, d..2d-1 K, 2d..3d-1 V; head h owns
    columns h*d_h..(h+1)*d_h of each."""
    S, d = x.shape
    dh = d // n_heads
    qkv = x @ th[pre + "wqkv"].T + th[pre + "bqkv"]
    q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
    heads = []
    for h in range(n_heads):
        sl = slice(h * dh, (h + 1) * dh)
        s = (q[:, sl] @ k[:, sl].T) / math.sqrt(dh)
        if causal:
            mask = torch.ones(S, S, dtype=torch.bool).tril()
            s = torch.where(mask, s, torch.full_like(s, -float("inf")))
        heads.append(softmax_rows(s) @ v[:, sl])
    ctx = torch.cat(heads, dim=1)
    return ctx @ th[pre + "wo"].T + th[pre + "bo"]


def transformer_layer(x, th, pre, n_heads, causal, attn_only=False):
    a = attention(x, th, pre, n_heads, causal)
    if attn_only:
        return x + a
    h1 = layer_norm(x + a, th[pre + "ln1_g"], th[pre + "ln1_b"])
    f = gelu(h1 @ th[pre + "w1"].T + th[pre + "b1"]) @ th[pre + "w2"].T + th[pre + "b2"]
    return layer_norm(h1 + f, th[pre + "ln2_g"], th[pre + "ln2_b"])


def ce_forward(th: Dict[str, torch.Tensor], tokens, shape) -> torch.Tensor:
    """h = CE(c; theta_CE) for ONE item: tokens [n] -> encoding [d], n <= l_t.  A text shorter than l_t is simply a
    shorter sequence (positions 0..n-1): no padding exists on this side, so attention and pooling range over the
    text alone (Section 3.2: c_i is the item's own token sequence; Table 3: lengths vary from item to item)."""
    tok = torch.as_tensor(np.asarray(tokens), dtype=torch.long)
    x = th["tok_emb"][tok] + th["pos_emb"][:tok.shape[0]]
    x = layer_norm(x, th["emb_ln_g"], th["emb_ln_b"])
    for l in range(shape.n_layers):
        x = transformer_layer(x, th, f"l{l}.", shape.n_heads, causal=False)
    if shape.pooling == "mean":
        return x.mean(dim=0)
    if shape.pooling == "cls":
        return x[0]
    if shape.pooling == "additive":
        # additive attention over the item's tokens (Appendix D: the news encoder pools its token outputs with
        # additive attention): a_s = q . tanh(W x_s + b), alpha = softmax(a), h = sum_s alpha_s x_s
        a = torch.tanh(x @ th["pool_wa"].T + th["pool_ba"]) @ th["pool_qa"]
        alpha = softmax_rows(a[None, :])[0]
        return alpha @ x
    raise KeyError(shape.pooling)


def kt_logits(th: Dict[str, torch.Tensor], E_hist: torch.Tensor, labels_hist, shape) -> torch.Tensor:
    """Logits of ONE knowledge-tracing history: E_hist [n, d] (encodings of its n items), labels_hist [n]
    (responses r_0..r_{n-1}) -> z [n].  Prediction n sees interactions (e_m, r_m) for m < n and the item e_n
    (Section 3.1), never r_n itself: x_n = E_hist[n] + pos[n] + resp[r_{n-1}], with resp row 2 standing for
    "no previous response" at n = 0; causal layers; z_n = head_w . y_n + head_b."""
    n = E_hist.shape[0]
    lab = torch.as_tensor(np.asarray(labels_hist), dtype=torch.long)
    prev = torch.cat([torch.full((1,), 2, dtype=torch.long), lab[:n - 1]])
    x = E_hist + th["pos"][:n] + th["resp"][prev]
    for l in range(shape.task_layers):
        x = transformer_layer(x, th, f"t{l}.", shape.task_heads, causal=True, attn_only=shape.task_attn_only)
    return x @ th["head_w"] + th["head_b"]


def bce_with_logits_sum(z: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    """Sum over predictions of -[y log sigma(z) + (1 - y) log(1 - sigma(z))] = softplus(z) - y z, the binary
    cross-entropy of Eq. 8 for correctness labels y in {0, 1}, written with a stable softplus."""
    return (torch.clamp(z, min=0) + torch.log1p(torch.exp(-z.abs())) - y * z).sum()


def nr_user_vector(th: Dict[str, torch.Tensor], clicked: torch.Tensor) -> torch.Tensor:
    """User vector from the encodings of the clicked items [m, d]: additive attention (Appendix D),
    a_n = qa . tanh(wa h_n + ba), alpha = softmax(a), u = sum_n alpha_n h_n."""
    a = torch.tanh(clicked @ th["wa"].T + th["ba"]) @ th["qa"]
    alpha = softmax_rows(a[None, :])[0]
    return alpha @ clicked


def nr_scores(th: Dict[str, torch.Tensor], clicked: torch.Tensor, cand: torch.Tensor, shape) -> torch.Tensor:
    """Scores of ONE user's candidates: s_j = u . c_j, u the user vector of the clicked items (which first pass
    through `task_layers` non-causal self-attention layers over the clicked items when the shape has any:
    Appendix D, a single MHSA layer in the news task)."""
    x = clicked
    for l in range(shape.task_layers):
        x = transformer_layer(x, th, f"t{l}.", shape.task_heads, causal=False, attn_only=shape.task_attn_only)
    return cand @ nr_user_vector(th, x)


def softmax_ce_first(s: torch.Tensor) -> torch.Tensor:
    """-log softmax(s)[0]: the clicked candidate is listed first, the sampled negatives follow."""
    m = s.max()
    return -(s[0] - m - torch.log(torch.exp(s - m).sum()))


def task_loss(th: Dict[str, torch.Tensor], E: torch.Tensor, labels, shape) -> torch.Tensor:
    """The CF objective (Eq. 8) over a mini-batch: E [B, L, d] -> scalar.

    kt: `kt_logits` per history, binary cross-entropy, averaged over all B*L
        predictions (over the real ones when histories end in padding, label -1).
    nr: `nr_scores` per user over the first L - n_cand encodings (the click
        history) and the n_cand candidate encodings, loss = -log softmax(scores)[0],
        averaged over the B users.  History slots with label -1 hold no click
        (a user with fewer clicks than slots) and take no part.
    """
    B, L, d = E.shape
    lab = torch.as_tensor(np.asarray(labels), dtype=torch.long)
    if shape.task == "kt":
        # A history shorter than L ends in padding, marked by label -1 (Appendix D: sequences are cut or padded to a
        # maximum length).  Padding is simply absent here: history b is the sequence of its first n_b positions,
        # and the mean runs over the sum of the n_b real predictions.
        total = E.new_zeros(())
        n_pred = 0
        for b in range(B):
            neg = (lab[b] < 0).nonzero()
            n = int(neg[0]) if len(neg) else L
            if n == 0:
                continue
            z = kt_logits(th, E[b, :n], lab[b, :n], shape)
            total = total + bce_with_logits_sum(z, lab[b, :n].to(E.dtype))
            n_pred += n
        return total / max(n_pred, 1)
    if shape.task == "nr":
        n_hist = L - shape.n_cand
        total = E.new_zeros(())
        for b in range(B):
            hist, cand = E[b, :n_hist], E[b, n_hist:]
            # a click history shorter than its slots: the slots with label -1 hold no click and are simply left out
            hist = hist[(lab[b, :n_hist] >= 0).nonzero()[:, 0]]
            total = total + softmax_ce_first(nr_scores(th, hist, cand, shape))
        return total / B
    raise KeyError(shape.task)


# ---------------------------------------------------------------------------
# helpers
# ---------------------------------------------------------------------------

def as_torch(params: Dict[str, np.ndarray], dtype=torch.float64, requires_grad=True) -> "OrderedDict[str, torch.Tensor]":
    out: "OrderedDict[str, torch.Tensor]" = OrderedDict()
    for k, v in params.items():
        t = torch.tensor(np.asarray(v), dtype=dtype)
        t.requires_grad_(requires_grad)
        out[k] = t
    return out


def _grads(th: Dict[str, torch.Tensor]) -> "OrderedDict[str, np.ndarray]":
    out: "OrderedDict[str, np.ndarray]" = OrderedDict()
    for k, t in th.items():
        out[k] = (t.grad if t.grad is not None else torch.zeros_like(t)).detach().numpy().copy()
    return out


# ---------------------------------------------------------------------------
# standard end-to-end training: the definition (Section 3.3)
# ---------------------------------------------------------------------------

def e2e_step(shape, ce_params, task_params, item_tokens, ids, labels, dtype=torch.float64):
    """One end-to-end gradient evaluation.  The encoder is called afresh for
    every occurrence; nothing is shared between two occurrences of an item.
    Returns dict(loss, grad_ce, grad_task, E)."""
    ids = np.asarray(ids)
    B, L = ids.shape
    th_ce = as_torch(ce_params, dtype)
    th_cf = as_torch(task_params, dtype)
    rows = []
    for b in range(B):
        rows.append(torch.stack([ce_forward(th_ce, item_tokens[int(ids[b, n])], shape) for n in range(L)]))
    E = torch.stack(rows)
    loss = task_loss(th_cf, E, labels, shape)
    loss.backward()
    return dict(loss=float(loss.detach()), grad_ce=_grads(th_ce), grad_task=_grads(th_cf),
                E=E.detach().numpy().copy())


# ---------------------------------------------------------------------------
# Single-step GRAM (Algorithm 1, N = 1), used to check the Proposition
# ---------------------------------------------------------------------------

def gram_single_step(shape, ce_params, task_params, item_tokens, ids, labels, dtype=torch.float64):
    """Returns dict(loss, grad_ce, grad_task, H, G, dE, unique, inverse)."""
    ids = np.asarray(ids)
    B, L = ids.shape
    unique, inverse, perm, seg_off = unique_inverse(ids)
    th_ce = as_torch(ce_params, dtype)
    th_cf = as_torch(task_params, dtype)
    # Eq. 4: one encoding per unique item
    H = torch.stack([ce_forward(th_ce, item_tokens[int(i)], shape) for i in unique])
    # the task module sees the encodings as leaves ("trainable embeddings")
    E = H.detach()[torch.as_tensor(inverse.astype(np.int64))].reshape(B, L, -1).clone().requires_grad_(True)
    loss = task_loss(th_cf, E, labels, shape)
    loss.backward()                                  # Eq. 5 gradients, and dL/dE
    dE = E.grad.reshape(B * L, -1).numpy()
    # Eq. 6: h~_i = h_i - sum over occurrences of dL/dE, so h_i - h~_i = G_i
    G = segment_sum(dE, perm, seg_off)
    # Eq. 7 / Eq. 9: gradient of 1/2 sum_i (h~_i - CE(c_i))^2 at the current
    # parameters is the VJP of CE with cotangent (h_i - h~_i) = G_i
    H.backward(torch.tensor(G, dtype=dtype))
    return dict(loss=float(loss.detach()), grad_ce=_grads(th_ce), grad_task=_grads(th_cf),
                H=H.detach().numpy().copy(), G=G, dE=dE.copy(), unique=unique, inverse=inverse)


def pseudo_loss_grad(shape, ce_params, item_tokens, items, h_tilde, dtype=torch.float64):
    """Gradient of the pseudo-loss 1/2 sum_i (h~_i - CE(c_i; theta'))^2 (Eq. 9)
    with respect to theta' at the given parameters; h_tilde is a constant."""
    th = as_torch(ce_params, dtype)
    H = torch.stack([ce_forward(th, item_tokens[int(i)], shape) for i in items])
    lt = 0.5 * ((torch.tensor(np.asarray(h_tilde), dtype=dtype) - H) ** 2).sum()
    lt.backward()
    return float(lt.detach()), _grads(th)


# ---------------------------------------------------------------------------
# Multi-step GRAM (Algorithm 1, N = K > 1)
# ---------------------------------------------------------------------------

def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16, returned in float64."""
    return torch.tensor(np.asarray(a), dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def encode_all(shape, ce_params, item_tokens, items, dtype=torch.float64) -> np.ndarray:
    th = as_torch(ce_params, dtype, requires_grad=False)
    with torch.no_grad():
        return torch.stack([ce_forward(th, item_tokens[int(i)], shape) for i in items]).numpy()


def multistep_window(shape, ce_params, task_params, item_tokens, batches, cache, lr_task: float,
                     cache_bf16: bool = False, dtype=torch.float64, lr_ce: Optional[float] = None,
                     refresh_after_update: bool = False):
    """One window of K = len(batches) steps of Algorithm 1, then the encoder
    pass.  Readings where the algorithm is silent or ambiguous:

    * Step 1 (Eq. 4) inside a window reads the per-item encoding from `cache`
      [n_items, d] (values computed before the window) instead of re-running
      CE, since CE's parameters do not change inside a window.
    * Step 2 (Eq. 5): `opt` is plain SGD with learning rate lr_task, applied
      after every step, so later steps of the window see updated task
      parameters.
    * Step 3 (Eq. 6): the per-item modification h_i - h~_i accumulates in a
      separate table (the cache itself stays unchanged during the window):
      table[i] += dL/dE[p] for every occurrence p of item i, in position order.
    * Step 4 fires after the K-th step of the window (the printed test
      `t mod N = 0` with t counted from 1), over ALL items touched in the
      window, with cotangent table[i]; its forward uses the current encoder
      parameters, and that forward value replaces cache[i].

    * lr_ce (optional): the encoder then takes a plain SGD step of that rate
      with the window's gradient (returned as ce_params).  With
      refresh_after_update the touched items are encoded once more with the
      updated parameters and those values go to the cache, which is Eq. 4 read
      literally (h is produced with the parameters of the current step).

    Returns dict(losses [K], grad_ce (sum over touched items in ascending item
    order), grad_task_last, task_params (after K SGD steps), table, touched,
    cache (updated), ce_params (after the step, when lr_ce is given))."""
    n_items, d = cache.shape
    cache = np.array(cache, dtype=np.float64)
    if cache_bf16:
        cache = round_to_bf16(cache)
    table = np.zeros((n_items, d), dtype=np.float64)
    touched = np.zeros(n_items, dtype=bool)
    cur_task = OrderedDict((k, np.array(v, dtype=np.float64)) for k, v in task_params.items())
    losses = []
    grad_task_last = None
    for ids, labels in batches:
        ids = np.asarray(ids)
        B, L = ids.shape
        th_cf = as_torch(cur_task, dtype)
        E = torch.tensor(cache[ids.ravel()], dtype=dtype).reshape(B, L, d).requires_grad_(True)
        loss = task_loss(th_cf, E, labels, shape)
        loss.backward()
        losses.append(float(loss.detach()))
        grad_task_last = _grads(th_cf)
        for k in cur_task:
            cur_task[k] = cur_task[k] - lr_task * grad_task_last[k]
        table_accumulate(table, touched, E.grad.reshape(B * L, d).numpy(), ids)
    items = np.nonzero(touched)[0]
    th_ce = as_torch(ce_params, dtype)
    H = torch.stack([ce_forward(th_ce, item_tokens[int(i)], shape) for i in items])
    H.backward(torch.tensor(table[items], dtype=dtype))
    newc = H.detach().numpy()
    grad_ce = _grads(th_ce)
    new_ce = None
    if lr_ce is not None:
        new_ce = OrderedDict((k, np.asarray(v, dtype=np.float64) - lr_ce * grad_ce[k]) for k, v in ce_params.items())
        if refresh_after_update:
            newc = encode_all(shape, new_ce, item_tokens, items, dtype)
    cache[items] = round_to_bf16(newc) if cache_bf16 else newc
    return dict(losses=losses, grad_ce=grad_ce, grad_task_last=grad_task_last, task_params=cur_task,
                table=table, touched=touched, cache=cache, items=items.astype(np.int32), ce_params=new_ce)


def multistep_window_pseudo_target(shape, ce_params, task_params, item_tokens, batches, cache, lr_task: float,
                                   dtype=torch.float64):
    """One window of K = len(batches) steps of Algorithm 1 under the *trainable-embedding* reading of
    Section 4.3: the content representation of an item is a trainable embedding h~_i that the task module
    keeps using after it has been modified (later steps of the window run on the updated representations),
    and the encoder regresses towards it (Eq. 9).

    * h~ starts as `cache` [n_items, d] (encoder outputs computed before the window).
    * Step 1 (Eq. 4) inside the window: the task module reads E[p] = h~[ids[p]], i.e. the cached encoding
      minus every gradient the item has received so far in this window.
    * Step 2 (Eq. 5): plain SGD with rate lr_task on the task parameters after every step.
    * Step 3 (Eq. 6): h~[i] <- h~[i] - dL/dE[p] for every occurrence p of item i, in position order
      (SGD with learning rate 1 on the embedding, as the paper prescribes).
    * Step 4 after the K-th step, over all items modified in the window: the gradient of the pseudo-loss
      1/2 sum_i (h~_i - CE(c_i; theta))^2 at the current encoder parameters, i.e. the encoder's VJP with
      cotangent CE(c_i; theta) - h~_i.  When `cache` is stale (computed with older encoder parameters) that
      cotangent carries the staleness CE(c_i; theta) - cache[i] besides the accumulated gradients.  The
      forward values CE(c_i; theta) replace cache[i].

    Returns dict(losses [K], grad_ce, grad_task_last, task_params, h_tilde (before the encoder pass), items,
    cache (updated))."""
    n_items, d = cache.shape
    cache = np.array(cache, dtype=np.float64)
    h_tilde = cache.copy()
    modified = np.zeros(n_items, dtype=bool)
    cur_task = OrderedDict((k, np.array(v, dtype=np.float64)) for k, v in task_params.items())
    losses = []
    grad_task_last = None
    for ids, labels in batches:
        ids = np.asarray(ids)
        B, L = ids.shape
        th_cf = as_torch(cur_task, dtype)
        E = torch.tensor(h_tilde[ids.ravel()], dtype=dtype).reshape(B, L, d).requires_grad_(True)
        loss = task_loss(th_cf, E, labels, shape)
        loss.backward()
        losses.append(float(loss.detach()))
        grad_task_last = _grads(th_cf)
        for k in cur_task:
            cur_task[k] = cur_task[k] - lr_task * grad_task_last[k]
        dE = E.grad.reshape(B * L, d).numpy()
        for p, i in enumerate(ids.ravel()):
            h_tilde[int(i), :] -= dE[p, :]
            modified[int(i)] = True
    items = np.nonzero(modified)[0]
    th_ce = as_torch(ce_params, dtype)
    H = torch.stack([ce_forward(th_ce, item_tokens[int(i)], shape) for i in items])
    pseudo = 0.5 * ((torch.tensor(h_tilde[items], dtype=dtype) - H) ** 2).sum()
    pseudo.backward()
    cache[items] = H.detach().numpy()
    return dict(losses=losses, grad_ce=_grads(th_ce), grad_task_last=grad_task_last, task_params=cur_task,
                h_tilde=h_tilde, items=items.astype(np.int32), cache=cache, pseudo_loss=float(pseudo.detach()))


# ---------------------------------------------------------------------------
# Optimiser (Appendix D, experiment details: Adam under the Noam learning-rate scheme, rate 1e-4)
# ---------------------------------------------------------------------------
def noam_rate(t: int, peak: float, warmup: int) -> float:
    """Learning rate at update t = 1, 2, ... under the Noam scheme (Vaswani et al. 2017, Eq. 3):
    rate proportional to min(t^-0.5, t * warmup^-1.5).  The paper gives one learning rate (1e-4) and no warm-up
    length; the reading taken here scales the curve so that its maximum, reached at t = warmup, is `peak`:
    rate = peak * min(t / warmup, sqrt(warmup / t)).  warmup <= 0 means a constant rate."""
    if warmup <= 0:
        return float(peak)
    t = float(t)
    return float(peak) * min(t / warmup, math.sqrt(warmup / t))


def adam_update(w: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, t: int, rate: float,
                beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8) -> None:
    """One Adam update in place (Kingma & Ba 2015, Algorithm 1), float64 arithmetic on whatever arrays are
    passed: first and second moment estimates, their bias corrections at update t (t >= 1), and the step."""
    g = g.astype(np.float64)
    m[...] = beta1 * m + (1.0 - beta1) * g
    v[...] = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** t)
    v_hat = v / (1.0 - beta2 ** t)
    w[...] = w - rate * m_hat / (np.sqrt(v_hat) + eps)


def train_steps_adam(shape, ce_params, task_params, item_tokens, batches, peak_ce: float, peak_task: float,
                     warmup: int, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8):
    """Successive end-to-end training steps (Section 3.3) with the Adam + Noam update applied to both modules
    after every batch (Single-step GRAM has the same gradients, hence the same trajectory).  batches: list of
    (ids, labels).  Returns (ce_params, task_params, losses) with float64 parameter copies."""
    ce = OrderedDict((k, np.array(a, dtype=np.float64)) for k, a in ce_params.items())
    tk = OrderedDict((k, np.array(a, dtype=np.float64)) for k, a in task_params.items())
    state = {id(d): (OrderedDict((k, np.zeros_like(a)) for k, a in d.items()),
                     OrderedDict((k, np.zeros_like(a)) for k, a in d.items())) for d in (ce, tk)}
    losses = []
    for t, (ids, labels) in enumerate(batches, start=1):
        r = e2e_step(shape, ce, tk, item_tokens, ids, labels)
        losses.append(r["loss"])
        for params, grads, peak in ((ce, r["grad_ce"], peak_ce), (tk, r["grad_task"], peak_task)):
            m, v = state[id(params)]
            rate = noam_rate(t, peak, warmup)
            for k in params:
                adam_update(params[k], grads[k], m[k], v[k], t, rate, beta1, beta2, eps)
    return ce, tk, losses
