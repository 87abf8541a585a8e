"""Pins for the oracle's encoder / task module and for the training schemes (CPU only)."""
import math
from collections import OrderedDict

import numpy as np
import pytest
import torch

from oracle import gram_oracle as orc
from paper_2204_04179_b200 import synth

T64 = torch.float64


def small_shape(**kw):
    base = dict(name="s", n_items=7, l_t=4, vocab=20, d=16, n_heads=2, d_ff=32, n_layers=1, pooling="mean",
                task="kt", task_layers=1, task_heads=2, task_d_ff=32, task_attn_only=True, B=2, L=5, zipf_s=1.1)
    base.update(kw)
    return synth.GramShape(**base)


def make(shape, seed=0, sigma=0.3):
    ce = synth.encoder_params(shape, seed, sigma=sigma, plain=False)
    tk = synth.task_params(shape, seed, sigma=sigma, plain=False)
    toks = synth.item_tokens(seed, shape.n_items, shape.l_t, shape.vocab)
    ids, lab = synth.batch(shape, seed)
    return ce, tk, toks, ids, lab


# ---- closed forms and library routines ------------------------------------

def test_gelu_and_layernorm_closed_forms():
    x = torch.tensor([0.0, 1.0, -1.0, 3.0], dtype=T64)
    phi = lambda v: 0.5 * (1 + math.erf(v / math.sqrt(2)))
    np.testing.assert_allclose(orc.gelu(x).numpy(), [0.0, phi(1.0), -phi(-1.0), 3 * phi(3.0)], rtol=1e-14)
    assert abs(float(orc.gelu(x)[1]) - 0.8413447460685429) < 1e-15
    r = torch.randn(5, 12, dtype=T64, generator=torch.Generator().manual_seed(0)) * 3 + 1
    y = orc.layer_norm(r, torch.ones(12, dtype=T64), torch.zeros(12, dtype=T64))
    np.testing.assert_allclose(y.mean(-1).numpy(), 0, atol=1e-14)
    var = r.var(-1, unbiased=False)
    np.testing.assert_allclose((y ** 2).mean(-1).numpy(), (var / (var + orc.LN_EPS)).numpy(), rtol=1e-12)
    g, b = torch.randn(12, dtype=T64), torch.randn(12, dtype=T64)
    np.testing.assert_allclose(orc.layer_norm(r, g, b).numpy(),
                               torch.nn.functional.layer_norm(r, (12,), g, b, eps=orc.LN_EPS).numpy(), rtol=1e-12, atol=1e-12)


def test_attention_uniform_scores_is_running_mean():
    # Q = 0 makes every score equal, so causal attention returns the running mean of V
    S, d = 6, 8
    th = {"a.wqkv": torch.zeros(3 * d, d, dtype=T64), "a.bqkv": torch.zeros(3 * d, dtype=T64),
          "a.wo": torch.eye(d, dtype=T64), "a.bo": torch.zeros(d, dtype=T64)}
    th["a.wqkv"][2 * d:] = torch.eye(d, dtype=T64)          # V = x
    x = torch.randn(S, d, dtype=T64, generator=torch.Generator().manual_seed(1))
    out = orc.attention(x, th, "a.", 2, causal=True)
    run = torch.cumsum(x, 0) / torch.arange(1, S + 1, dtype=T64)[:, None]
    np.testing.assert_allclose(out.numpy(), run.numpy(), rtol=1e-13, atol=1e-13)
    out = orc.attention(x, th, "a.", 2, causal=False)
    np.testing.assert_allclose(out.numpy(), x.mean(0, keepdim=True).expand(S, d).numpy(), rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_layer_matches_library_transformer_layer(causal):
    # the post-LayerNorm layer is the textbook one: torch's own encoder layer with the same weights
    shape = small_shape(d=16, n_heads=4, d_ff=24)
    p = synth._draw_params(synth._layer_spec("x.", 16, 24, False), np.random.default_rng(3), 0.4, False)
    th = orc.as_torch(p, T64, requires_grad=False)
    lib = torch.nn.TransformerEncoderLayer(16, 4, 24, dropout=0.0, activation="gelu", layer_norm_eps=orc.LN_EPS,
                                           batch_first=True, norm_first=False, dtype=T64)
    with torch.no_grad():
        lib.self_attn.in_proj_weight.copy_(th["x.wqkv"]); lib.self_attn.in_proj_bias.copy_(th["x.bqkv"])
        lib.self_attn.out_proj.weight.copy_(th["x.wo"]); lib.self_attn.out_proj.bias.copy_(th["x.bo"])
        lib.linear1.weight.copy_(th["x.w1"]); lib.linear1.bias.copy_(th["x.b1"])
        lib.linear2.weight.copy_(th["x.w2"]); lib.linear2.bias.copy_(th["x.b2"])
        lib.norm1.weight.copy_(th["x.ln1_g"]); lib.norm1.bias.copy_(th["x.ln1_b"])
        lib.norm2.weight.copy_(th["x.ln2_g"]); lib.norm2.bias.copy_(th["x.ln2_b"])
    lib.train()                                        # keep the plain (non-fused) code path
    x = torch.randn(9, 16, dtype=T64, generator=torch.Generator().manual_seed(2))
    mask = torch.triu(torch.full((9, 9), float("-inf"), dtype=T64), diagonal=1) if causal else None
    with torch.no_grad():
        want = lib(x[None], src_mask=mask)[0]
        got = orc.transformer_layer(x, th, "x.", 4, causal)
    np.testing.assert_allclose(got.numpy(), want.numpy(), rtol=1e-10, atol=1e-12)


def test_losses_at_zero_parameters():
    # all-zero task parameters: every logit is 0 -> BCE = ln 2; every score equal -> CE = ln(n_cand)
    kt = small_shape()
    z = OrderedDict((k, np.zeros(s, np.float32)) for k, s in synth.task_param_spec(kt))
    E = torch.randn(kt.B, kt.L, kt.d, dtype=T64)
    lab = synth.labels(0, kt.B, kt.L, 0.6)
    assert float(orc.task_loss(orc.as_torch(z, T64, False), E, lab, kt)) == pytest.approx(math.log(2), rel=1e-14)
    nr = small_shape(task="nr", n_cand=5, L=8, d_a=6, task_layers=0)
    z = OrderedDict((k, np.zeros(s, np.float32)) for k, s in synth.task_param_spec(nr))
    E = torch.zeros(nr.B, nr.L, nr.d, dtype=T64)
    assert float(orc.task_loss(orc.as_torch(z, T64, False), E, lab, nr)) == pytest.approx(math.log(5), rel=1e-14)


# ---- the task module's pieces: each pinned on the oracle's own function, each with a planted mistake -----------------

def _must_fail(check, *args):
    with pytest.raises(AssertionError):
        check(*args)


def _check_no_label_leak(logits_fn):
    # prediction n may depend on responses 0..n-1 only (Section 3.1): two label rows that differ at position 3
    # give identical logits 0..3 and a different logit 4
    shape = small_shape(task_attn_only=False)
    _, tk, _, _, _ = make(shape)
    th = orc.as_torch(tk, T64, False)
    E = torch.randn(shape.L, shape.d, dtype=T64, generator=torch.Generator().manual_seed(0))
    a = np.array([1, 0, 1, 1, 0]); b = a.copy(); b[3] = 0
    with torch.no_grad():
        la, lb = logits_fn(th, E, a, shape), logits_fn(th, E, b, shape)
    assert la.shape == (shape.L,)
    np.testing.assert_allclose(la[:4].numpy(), lb[:4].numpy(), rtol=0, atol=0)      # logits 0..3 unchanged
    assert abs(float(la[4] - lb[4])) > 1e-9                                         # logit 4 sees response 3
    # position 0 uses the "no previous response" row 2 of resp: it moves with that row and with nothing else of resp
    th2 = dict(th); th2["resp"] = th["resp"].clone(); th2["resp"][2] += 0.5
    th3 = dict(th); th3["resp"] = th["resp"].clone(); th3["resp"][:2] += 0.5
    with torch.no_grad():
        assert abs(float(logits_fn(th2, E, a, shape)[0] - la[0])) > 1e-9
        assert float(logits_fn(th3, E, a, shape)[0]) == float(la[0])


def test_kt_logits_do_not_see_the_label_they_predict():
    _check_no_label_leak(orc.kt_logits)

    def leaky(th, E, labels, shape):          # planted mistake: position n reads its own response r_n
        lab = torch.as_tensor(np.asarray(labels), dtype=torch.long)
        x = E + th["pos"][:E.shape[0]] + th["resp"][lab]
        for l in range(shape.task_layers):
            x = orc.transformer_layer(x, th, f"t{l}.", shape.task_heads, True, shape.task_attn_only)
        return x @ th["head_w"] + th["head_b"]

    def shifted_two(th, E, labels, shape):    # planted mistake: response n-2 instead of n-1
        lab = torch.as_tensor(np.asarray(labels), dtype=torch.long)
        prev = torch.cat([torch.full((2,), 2, dtype=torch.long), lab[:E.shape[0] - 2]])
        x = E + th["pos"][:E.shape[0]] + th["resp"][prev]
        for l in range(shape.task_layers):
            x = orc.transformer_layer(x, th, f"t{l}.", shape.task_heads, True, shape.task_attn_only)
        return x @ th["head_w"] + th["head_b"]
    _must_fail(_check_no_label_leak, leaky)
    _must_fail(_check_no_label_leak, shifted_two)


def test_kt_logits_with_one_position_is_the_plain_head():
    # a one-position history: causal attention over one key returns V itself, so with identity V / output
    # projections the logit is head_w . 2 x_0 + head_b with x_0 = e_0 + pos_0 + resp_2 (closed form)
    shape = small_shape(L=1)
    d = shape.d
    th = orc.as_torch(synth.task_params(shape, 1, sigma=0.3, plain=False), T64, False)
    th["t0.wqkv"][2 * d:] = torch.eye(d, dtype=T64); th["t0.bqkv"].zero_()
    th["t0.wo"] = torch.eye(d, dtype=T64); th["t0.bo"].zero_()
    e0 = torch.randn(1, d, dtype=T64, generator=torch.Generator().manual_seed(3))
    x0 = e0[0] + th["pos"][0] + th["resp"][2]
    z = orc.kt_logits(th, e0, np.array([1]), shape)
    assert float(z[0]) == pytest.approx(float(2 * x0 @ th["head_w"] + th["head_b"][0]), rel=1e-13)


def _check_bce(sum_fn):
    g = torch.Generator().manual_seed(5)
    z = torch.randn(40, dtype=T64, generator=g) * 4
    y = (torch.rand(40, generator=g) < 0.6).to(T64)
    want = torch.nn.functional.binary_cross_entropy_with_logits(z, y, reduction="sum")
    assert float(sum_fn(z, y)) == pytest.approx(float(want), rel=1e-13)
    # far tails stay finite and keep their asymptote |z| on the wrong side, 0 on the right side
    zt = torch.tensor([800.0, -800.0], dtype=T64)
    assert float(sum_fn(zt, torch.tensor([0.0, 1.0], dtype=T64))) == pytest.approx(1600.0, rel=1e-14)
    assert float(sum_fn(zt, torch.tensor([1.0, 0.0], dtype=T64))) == pytest.approx(0.0, abs=1e-300)


def test_binary_cross_entropy_matches_the_library_at_random_logits():
    _check_bce(orc.bce_with_logits_sum)
    _must_fail(_check_bce, lambda z, y: (torch.nn.functional.softplus(z) + y * z).sum())          # sign of y z
    _must_fail(_check_bce, lambda z, y: (torch.nn.functional.softplus(z) - (1 - y) * z).sum())    # inverted labels
    _must_fail(_check_bce, lambda z, y: (torch.nn.functional.softplus(-z) - y * z).sum())         # softplus of -z


def _check_first_candidate_ce(ce_fn):
    g = torch.Generator().manual_seed(6)
    for n in (2, 5):
        s = torch.randn(n, dtype=T64, generator=g) * 3
        want = torch.nn.functional.cross_entropy(s[None], torch.zeros(1, dtype=torch.long))
        assert float(ce_fn(s)) == pytest.approx(float(want), rel=1e-13)
    assert float(ce_fn(torch.tensor([900.0, 0.0, -900.0], dtype=T64))) == pytest.approx(0.0, abs=1e-300)
    assert float(ce_fn(torch.tensor([0.0, 900.0], dtype=T64))) == pytest.approx(900.0, rel=1e-14)


def test_candidate_cross_entropy_takes_the_first_candidate_as_the_click():
    _check_first_candidate_ce(orc.softmax_ce_first)
    _must_fail(_check_first_candidate_ce, lambda s: -torch.log_softmax(s, 0)[-1])     # positive = last candidate
    _must_fail(_check_first_candidate_ce, lambda s: torch.log_softmax(s, 0)[0])       # sign
    _must_fail(_check_first_candidate_ce, lambda s: -torch.log_softmax(-s, 0)[0])     # sign of the scores


def _check_user_vector(user_fn):
    shape = small_shape(task="nr", n_cand=3, L=8, d_a=6, task_layers=0)
    th = orc.as_torch(synth.task_params(shape, 2, sigma=0.5, plain=False), T64, False)
    h = torch.randn(5, shape.d, dtype=T64, generator=torch.Generator().manual_seed(7))
    # q = 0: every score equal, the user vector is the plain mean of the clicked rows
    th0 = dict(th); th0["qa"] = torch.zeros_like(th["qa"])
    np.testing.assert_allclose(user_fn(th0, h).numpy(), h.mean(0).numpy(), rtol=1e-13)
    # a one-click history: the user vector is that row, whatever the parameters
    np.testing.assert_allclose(user_fn(th, h[2:3]).numpy(), h[2].numpy(), rtol=1e-14)
    # general case: the weights are the library softmax of q . tanh(W h + b), a convex combination
    w = torch.softmax(torch.tanh(torch.nn.functional.linear(h, th["wa"], th["ba"])) @ th["qa"], 0)
    np.testing.assert_allclose(user_fn(th, h).numpy(), (w[:, None] * h).sum(0).numpy(), rtol=1e-13)
    # one saturated score picks its row: scale q so that row 4's score dominates
    t = torch.tanh(torch.nn.functional.linear(h, th["wa"], th["ba"]))
    thq = dict(th); thq["qa"] = 500.0 * (t[4] - t[:4].mean(0))
    sc = t @ thq["qa"]
    assert float(sc[4] - sc[:4].max()) > 50
    np.testing.assert_allclose(user_fn(thq, h).numpy(), h[4].numpy(), rtol=1e-12)


def test_user_vector_closed_forms():
    _check_user_vector(orc.nr_user_vector)

    def no_tanh(th, h):                       # planted mistake: scores without the tanh
        return torch.softmax(torch.nn.functional.linear(h, th["wa"], th["ba"]) @ th["qa"], 0) @ h

    def weights_on_projection(th, h):         # planted mistake: sums the projected rows instead of the encodings
        t = torch.tanh(torch.nn.functional.linear(h, th["wa"], th["ba"]))
        return torch.nn.functional.pad(torch.softmax(t @ th["qa"], 0) @ t, (0, h.shape[1] - t.shape[1]))

    def unnormalised(th, h):                  # planted mistake: exp weights without the softmax's division
        return torch.exp(torch.tanh(torch.nn.functional.linear(h, th["wa"], th["ba"])) @ th["qa"]) @ h
    _must_fail(_check_user_vector, no_tanh)
    _must_fail(_check_user_vector, weights_on_projection)
    _must_fail(_check_user_vector, unnormalised)


def test_scores_are_dot_products_with_the_user_vector_and_task_loss_is_the_mean_of_its_pieces():
    nr = small_shape(task="nr", n_cand=3, L=8, d_a=6, task_layers=0, B=3)
    th = orc.as_torch(synth.task_params(nr, 2, sigma=0.5, plain=False), T64, False)
    E = torch.randn(nr.B, nr.L, nr.d, dtype=T64, generator=torch.Generator().manual_seed(8))
    lab = np.zeros((nr.B, nr.L), np.int32)
    with torch.no_grad():
        s = orc.nr_scores(th, E[0, :5], E[0, 5:], nr)
        u = orc.nr_user_vector(th, E[0, :5])
        np.testing.assert_allclose(s.numpy(), [float(E[0, 5 + j] @ u) for j in range(3)], rtol=1e-13)
        # the batch loss is the library cross-entropy (target 0, mean over users) of the per-user scores
        S = torch.stack([orc.nr_scores(th, E[b, :5], E[b, 5:], nr) for b in range(nr.B)])
        want = torch.nn.functional.cross_entropy(S, torch.zeros(nr.B, dtype=torch.long))
        assert float(orc.task_loss(th, E, lab, nr)) == pytest.approx(float(want), rel=1e-13)
        # candidates are the LAST n_cand positions of a user's row: permuting the history rows leaves the loss alone,
        # swapping a history row with a candidate does not
        Ep = E.clone(); Ep[:, :5] = E[:, [4, 2, 0, 1, 3]]
        assert float(orc.task_loss(th, Ep, lab, nr)) == pytest.approx(float(want), rel=1e-13)
        Es = E.clone(); Es[:, 0], Es[:, 5] = E[:, 5], E[:, 0]
        assert abs(float(orc.task_loss(th, Es, lab, nr)) - float(want)) > 1e-6
    kt = small_shape(task_attn_only=False, B=3)
    thk = orc.as_torch(synth.task_params(kt, 2, sigma=0.3, plain=False), T64, False)
    Ek = torch.randn(kt.B, kt.L, kt.d, dtype=T64, generator=torch.Generator().manual_seed(9))
    labk = synth.labels(3, kt.B, kt.L, 0.6)
    with torch.no_grad():
        Z = torch.stack([orc.kt_logits(thk, Ek[b], labk[b], kt) for b in range(kt.B)])
        want = torch.nn.functional.binary_cross_entropy_with_logits(Z, torch.as_tensor(labk, dtype=T64), reduction="mean")
        assert float(orc.task_loss(thk, Ek, labk, kt)) == pytest.approx(float(want), rel=1e-13)


# ---- derivatives: central finite differences on a 1-layer encoder ----------

def _loss_only(shape, ce, tk, toks, ids, lab):
    th_ce, th_cf = orc.as_torch(ce, T64, False), orc.as_torch(tk, T64, False)
    with torch.no_grad():
        E = torch.stack([torch.stack([orc.ce_forward(th_ce, toks[int(i)], shape) for i in row]) for row in ids])
        return float(orc.task_loss(th_cf, E, lab, shape))


@pytest.mark.parametrize("variant", ["kt_attn_mean", "kt_full_cls", "nr_cls", "nr_mhsa"])
def test_e2e_gradients_match_finite_differences(variant):
    if variant == "kt_attn_mean":
        shape = small_shape()
    elif variant == "kt_full_cls":
        shape = small_shape(pooling="cls", task_attn_only=False)
    elif variant == "nr_mhsa":
        shape = small_shape(pooling="cls", task="nr", n_cand=3, L=7, d_a=5, task_layers=1, task_attn_only=True)
    else:
        shape = small_shape(pooling="cls", task="nr", n_cand=3, L=6, d_a=5, task_layers=0)
    ce, tk, toks, ids, lab = make(shape, seed=4)
    ce = OrderedDict((k, v.astype(np.float64)) for k, v in ce.items())
    tk = OrderedDict((k, v.astype(np.float64)) for k, v in tk.items())
    out = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    rng = np.random.default_rng(0)
    eps = 1e-5
    for params, grads, which in ((ce, out["grad_ce"], "ce"), (tk, out["grad_task"], "task")):
        for name, arr in params.items():
            if name == "tok_emb":        # only rows of tokens that occur carry gradient: sample among them
                used = np.unique(toks[np.unique(ids)])
                cand = [(int(r), int(c)) for r in used[:3] for c in (0, 5)]
            else:
                flat = rng.choice(arr.size, size=min(3, arr.size), replace=False)
                cand = [np.unravel_index(int(f), arr.shape) for f in flat]
            for idx in cand:
                old = arr[idx]
                arr[idx] = old + eps
                lp = _loss_only(shape, ce, tk, toks, ids, lab)
                arr[idx] = old - eps
                lm = _loss_only(shape, ce, tk, toks, ids, lab)
                arr[idx] = old
                fd = (lp - lm) / (2 * eps)
                an = grads[name][idx]
                assert abs(fd - an) <= 1e-6 * max(1.0, abs(fd)) + 1e-8, (which, name, idx, fd, an)


# ---- the Proposition: Single-step GRAM's gradients equal end-to-end's -------

@pytest.mark.parametrize("variant", ["tiny_cfg", "kt_full_cls", "nr_cls"])
def test_single_step_equals_e2e(variant):
    if variant == "tiny_cfg":
        shape = synth.config("tiny").replace(B=3, L=8, n_items=10)      # heavy reuse: 24 occurrences of <= 10 items
    elif variant == "kt_full_cls":
        shape = small_shape(pooling="cls", task_attn_only=False, B=3, L=6)
    else:
        shape = small_shape(pooling="cls", task="nr", n_cand=3, L=7, d_a=5, task_layers=0, B=3)
    ce, tk, toks, ids, lab = make(shape, seed=7)
    a = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    b = orc.gram_single_step(shape, ce, tk, toks, ids, lab)
    assert len(b["unique"]) < ids.size                                    # duplicates really occur
    assert a["loss"] == pytest.approx(b["loss"], rel=1e-13)
    for key in ("grad_ce", "grad_task"):
        for name in a[key]:
            scale = np.abs(a[key][name]).max() + 1e-30
            assert np.abs(a[key][name] - b[key][name]).max() <= 1e-11 * scale + 1e-15, (key, name)
    # and a planted mistake (one occurrence dropped from an item's sum) is seen
    unique, inverse, perm, seg_off = orc.unique_inverse(ids)
    u = int(np.argmax(np.diff(seg_off)))                                  # the most repeated item
    drop = int(np.argmax(np.abs(b["dE"][perm[seg_off[u]:seg_off[u + 1]]]).max(1))) + int(seg_off[u])
    so_bad = seg_off.copy(); so_bad[u + 1:] -= 1
    G_bad = orc.segment_sum(b["dE"], np.delete(perm, drop), so_bad)
    assert np.abs(G_bad - b["G"]).max() > 1e-6


def test_pseudo_loss_identity_and_lr1_sgd():
    # Eqs. 1-3: with h~ = h - dL/dh, the gradient of 1/2 (h~ - f(x; theta'))^2 at theta' = theta is dL/dtheta
    shape = small_shape(B=2, L=6)
    ce, tk, toks, ids, lab = make(shape, seed=9)
    s = orc.gram_single_step(shape, ce, tk, toks, ids, lab)
    h_tilde = s["H"] - s["G"]                          # Eq. 6: SGD with learning rate 1 on the embedding
    np.testing.assert_allclose(s["H"] - h_tilde, s["G"], rtol=1e-9, atol=1e-12)
    lt, g = orc.pseudo_loss_grad(shape, ce, toks, s["unique"], h_tilde)
    assert lt == pytest.approx(0.5 * (s["G"] ** 2).sum(), rel=1e-9)
    for name in g:
        scale = np.abs(s["grad_ce"][name]).max() + 1e-30
        assert np.abs(g[name] - s["grad_ce"][name]).max() <= 1e-9 * scale + 1e-14, name
    # a learning rate other than 1 in Eq. 6 breaks the identity
    _, g2 = orc.pseudo_loss_grad(shape, ce, toks, s["unique"], s["H"] - 0.5 * s["G"])
    assert np.abs(g2["l0.wqkv"] - s["grad_ce"]["l0.wqkv"]).max() > 1e-3 * np.abs(s["grad_ce"]["l0.wqkv"]).max()


# ---- Multi-step -------------------------------------------------------------

def test_multistep_k1_reduces_to_single_step():
    # Section 4.3: the algorithm is Single-step GRAM for N = 1 (given a cache that holds CE's current outputs)
    shape = small_shape(B=2, L=6)
    ce, tk, toks, ids, lab = make(shape, seed=11)
    cache = orc.encode_all(shape, ce, toks, range(shape.n_items))
    m = orc.multistep_window(shape, ce, tk, toks, [(ids, lab)], cache, lr_task=0.1)
    s = orc.gram_single_step(shape, ce, tk, toks, ids, lab)
    assert m["losses"][0] == pytest.approx(s["loss"], rel=1e-13)
    assert np.array_equal(m["items"], s["unique"])
    for name in s["grad_ce"]:
        scale = np.abs(s["grad_ce"][name]).max() + 1e-30
        assert np.abs(m["grad_ce"][name] - s["grad_ce"][name]).max() <= 1e-11 * scale, name
    for name in s["grad_task"]:
        np.testing.assert_allclose(m["task_params"][name], tk[name] - 0.1 * s["grad_task"][name], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(m["cache"], cache, rtol=1e-12, atol=1e-14)     # encoder unchanged -> same values


def test_multistep_table_and_touched_over_k_steps():
    shape = small_shape(B=2, L=6, K=3)
    ce, tk, toks, _, _ = make(shape, seed=13)
    cache = orc.encode_all(shape, ce, toks, range(shape.n_items))
    batches = [synth.batch(shape, 13, step=k) for k in range(3)]
    m = orc.multistep_window(shape, ce, tk, toks, batches, cache, lr_task=0.0)
    # with lr_task = 0 the task module is frozen, so each step's dE is the single-step dE on the cached encodings
    expect = np.zeros_like(m["table"]); union = set()
    for ids, lab in batches:
        s = orc.gram_single_step(shape, ce, tk, toks, ids, lab)
        expect[s["unique"]] += s["G"]
        union |= set(int(i) for i in s["unique"])
    np.testing.assert_allclose(m["table"], expect, rtol=1e-10, atol=1e-13)
    assert set(int(i) for i in m["items"]) == union
    # the encoder gradient is the VJP with the table rows: linear in the table
    th = orc.as_torch(ce, T64)
    H = torch.stack([orc.ce_forward(th, toks[int(i)], shape) for i in m["items"]])
    H.backward(torch.tensor(expect[m["items"]]))
    np.testing.assert_allclose(m["grad_ce"]["l0.w1"], th["l0.w1"].grad.numpy(), rtol=1e-9, atol=1e-13)


def test_multistep_later_steps_see_updated_task_parameters():
    shape = small_shape(B=2, L=6, K=2)
    ce, tk, toks, _, _ = make(shape, seed=15)
    cache = orc.encode_all(shape, ce, toks, range(shape.n_items))
    batches = [synth.batch(shape, 15, step=k) for k in range(2)]
    a = orc.multistep_window(shape, ce, tk, toks, batches, cache, lr_task=0.5)
    b = orc.multistep_window(shape, ce, tk, toks, batches, cache, lr_task=0.0)
    assert a["losses"][0] == pytest.approx(b["losses"][0], rel=1e-13)
    assert abs(a["losses"][1] - b["losses"][1]) > 1e-6


# ---- Multi-step under the trainable-embedding reading (Section 4.3, Eqs. 6 and 9) ------------------------------------

def test_pseudo_target_window_k1_fresh_cache_is_e2e():
    # one step, cache computed with the current encoder: h~ - CE = -sum dL/dE, so Eq. 9's gradient is end-to-end's
    shape = small_shape(pooling="cls")
    ce, tk, toks, ids, lab = make(shape, seed=4)
    cache = orc.encode_all(shape, ce, toks, range(shape.n_items))
    got = orc.multistep_window_pseudo_target(shape, ce, tk, toks, [(ids, lab)], cache, lr_task=0.1)
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    assert abs(got["losses"][0] - want["loss"]) < 1e-12
    for k in want["grad_ce"]:
        np.testing.assert_allclose(got["grad_ce"][k], want["grad_ce"][k], rtol=1e-9, atol=1e-12)
    assert np.array_equal(got["items"], np.unique(ids))


def test_pseudo_target_embedding_follows_library_sgd_with_rate_one():
    # the encoding treated as a trainable embedding (Section 4.3): a torch Parameter updated by torch.optim.SGD(lr=1) over the same batches
    # must end at the oracle's h~ (duplicates of an item inside a batch add up through autograd's index backward)
    shape = small_shape(n_items=6, B=2, L=6)
    ce, tk, toks, _, _ = make(shape, seed=6)
    batches = [synth.batch(shape, 6, step=k) for k in range(3)]
    assert any(len(np.unique(i)) < i.size for i, _ in batches)                    # duplicates inside a batch
    assert len(np.intersect1d(batches[0][0], batches[1][0])) > 0                  # and an item seen in two steps
    cache = orc.encode_all(shape, ce, toks, range(shape.n_items))
    lr = 0.2
    got = orc.multistep_window_pseudo_target(shape, ce, tk, toks, batches, cache, lr_task=lr)
    emb = torch.nn.Parameter(torch.tensor(cache, dtype=T64))
    th = orc.as_torch(tk)
    opt_e = torch.optim.SGD([emb], lr=1.0)
    opt_t = torch.optim.SGD(list(th.values()), lr=lr)
    losses = []
    for ids, lab in batches:
        opt_e.zero_grad(); opt_t.zero_grad()
        E = emb[torch.as_tensor(ids.astype(np.int64))]
        loss = orc.task_loss(th, E, lab, shape)
        loss.backward()
        opt_e.step(); opt_t.step()
        losses.append(float(loss.detach()))
    np.testing.assert_allclose(got["losses"], losses, rtol=1e-12)
    np.testing.assert_allclose(got["h_tilde"], emb.detach().numpy(), rtol=1e-12, atol=1e-14)
    for k in th:
        np.testing.assert_allclose(got["task_params"][k], th[k].detach().numpy(), rtol=1e-12, atol=1e-14)
    # the later step really saw the modified embedding: with the unmodified cache its loss differs
    plain = orc.multistep_window(shape, ce, tk, toks, batches, cache, lr_task=lr)
    assert abs(plain["losses"][0] - got["losses"][0]) < 1e-14 and abs(plain["losses"][1] - got["losses"][1]) > 1e-9


def test_pseudo_target_gradient_with_a_stale_cache_matches_finite_differences():
    # a cache computed with other encoder parameters: the cotangent CE(c; theta) - h~ then carries the staleness term.
    # Central differences of the pseudo-loss of Eq. 9 (h~ held constant) pin its sign and scale.
    shape = small_shape(n_items=5, B=1, L=4, d=8, d_ff=16, vocab=12)
    ce, tk, toks, ids, lab = make(shape, seed=8)
    ce = OrderedDict((k, np.asarray(v, np.float64)) for k, v in ce.items())        # so that +-eps is exact enough
    ce_old = OrderedDict((k, v + 0.05 * np.random.default_rng(1).standard_normal(v.shape)) for k, v in ce.items())
    cache = orc.encode_all(shape, ce_old, toks, range(shape.n_items))
    got = orc.multistep_window_pseudo_target(shape, ce, tk, toks, [(ids, lab)], cache, lr_task=0.0)
    items, h_t = got["items"], got["h_tilde"][got["items"]]

    def pseudo(params):
        H = orc.encode_all(shape, params, toks, items)
        return 0.5 * float(((h_t - H) ** 2).sum())
    assert abs(pseudo(ce) - got["pseudo_loss"]) < 1e-12
    rng = np.random.default_rng(2)
    for name in ("l0.wqkv", "l0.w2", "tok_emb", "l0.ln2_b"):
        flat_idx = rng.integers(0, ce[name].size, 3)
        for fi in flat_idx:
            idx = np.unravel_index(fi, ce[name].shape)
            eps = 1e-6
            up = OrderedDict((k, v.copy()) for k, v in ce.items()); up[name][idx] += eps
            dn = OrderedDict((k, v.copy()) for k, v in ce.items()); dn[name][idx] -= eps
            fd = (pseudo(up) - pseudo(dn)) / (2 * eps)
            assert abs(fd - got["grad_ce"][name][idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, got["grad_ce"][name][idx])
    # dropping the staleness term (the table-only cotangent of the other reading) gives a different gradient here
    plain = orc.multistep_window(shape, ce, tk, toks, [(ids, lab)], cache, lr_task=0.0)
    assert max(np.abs(plain["grad_ce"][k] - got["grad_ce"][k]).max() for k in ce) > 1e-4
    np.testing.assert_allclose(got["cache"][items], orc.encode_all(shape, ce, toks, items), rtol=1e-13)


# ---- texts of different lengths (Table 3: 5 to 271 tokens per item) ---------------------------------------------------

def test_short_text_equals_library_layer_with_padding_mask():
    # the oracle encodes a short text as a short sequence; a padded sequence run through torch's own encoder layer
    # with a key-padding mask must give the same rows for the text tokens
    d, heads, dff, n, l_t = 16, 4, 24, 5, 9
    p = synth._draw_params(synth._layer_spec("x.", d, dff, False), np.random.default_rng(5), 0.4, False)
    th = orc.as_torch(p, T64, requires_grad=False)
    lib = torch.nn.TransformerEncoderLayer(d, heads, dff, dropout=0.0, activation="gelu", layer_norm_eps=orc.LN_EPS,
                                           batch_first=True, norm_first=False, dtype=T64)
    with torch.no_grad():
        lib.self_attn.in_proj_weight.copy_(th["x.wqkv"]); lib.self_attn.in_proj_bias.copy_(th["x.bqkv"])
        lib.self_attn.out_proj.weight.copy_(th["x.wo"]); lib.self_attn.out_proj.bias.copy_(th["x.bo"])
        lib.linear1.weight.copy_(th["x.w1"]); lib.linear1.bias.copy_(th["x.b1"])
        lib.linear2.weight.copy_(th["x.w2"]); lib.linear2.bias.copy_(th["x.b2"])
        lib.norm1.weight.copy_(th["x.ln1_g"]); lib.norm1.bias.copy_(th["x.ln1_b"])
        lib.norm2.weight.copy_(th["x.ln2_g"]); lib.norm2.bias.copy_(th["x.ln2_b"])
    lib.train()
    x = torch.randn(l_t, d, dtype=T64, generator=torch.Generator().manual_seed(4))      # rows n.. play the padding
    pad = torch.zeros(1, l_t, dtype=torch.bool); pad[0, n:] = True
    with torch.no_grad():
        want = lib(x[None], src_key_padding_mask=pad)[0, :n]
        got = orc.transformer_layer(x[:n], th, "x.", heads, causal=False)
    np.testing.assert_allclose(got.numpy(), want.numpy(), rtol=1e-10, atol=1e-12)


def test_short_text_encoding_ignores_what_follows_it():
    shape = small_shape(l_t=6, pooling="mean")
    ce, tk, toks, ids, lab = make(shape, seed=9)
    th = orc.as_torch(ce, T64, requires_grad=False)
    with torch.no_grad():
        a = orc.ce_forward(th, toks[0][:4], shape)
        other = toks[0].copy(); other[4:] = (other[4:] + 1) % shape.vocab
        b = orc.ce_forward(th, other[:4], shape)
        full = orc.ce_forward(th, toks[0], shape)
    assert torch.equal(a, b) and not torch.allclose(a, full)
    # mean pooling is over the text tokens: a one-token text pools to that token's own output row
    one = orc.ce_forward(th, toks[0][:1], shape)
    x = orc.layer_norm(th["tok_emb"][int(toks[0][0])] + th["pos_emb"][0], th["emb_ln_g"], th["emb_ln_b"])[None]
    for l in range(shape.n_layers):
        x = orc.transformer_layer(x, th, f"l{l}.", shape.n_heads, causal=False)
    np.testing.assert_allclose(one.numpy(), x[0].numpy(), rtol=1e-13)


# ---- histories of different lengths (padding at the end, label -1) -----------------------------------------------------

def test_padded_history_is_the_shorter_history():
    # two histories, the second with n < L real positions: the loss is the prediction-weighted mean of the two
    # histories evaluated on their own (the second one as a batch whose L is n), and nothing at a padded position
    # (its encoding, its gradient) takes part
    shape = small_shape(B=2, L=6, task_attn_only=False, task_layers=2)
    ce, tk, toks, ids, lab = make(shape, seed=12)
    n = 4
    lab = lab.copy(); lab[1, n:] = -1
    E = torch.randn(2, 6, shape.d, dtype=T64, generator=torch.Generator().manual_seed(1))
    th = orc.as_torch(tk, T64)
    Eg = E.clone().requires_grad_(True)
    loss = orc.task_loss(th, Eg, lab, shape)
    loss.backward()
    with torch.no_grad():
        one = orc.task_loss(th, E[:1], lab[:1], shape.replace(B=1))
        th_short = dict(th); th_short["pos"] = th["pos"][:n]
        two = orc.task_loss(th_short, E[1:, :n], lab[1:, :n], shape.replace(B=1, L=n))
    assert abs(float(loss.detach()) - (6 * float(one) + n * float(two)) / (6 + n)) < 1e-13
    assert torch.count_nonzero(Eg.grad[1, n:]) == 0 and torch.count_nonzero(Eg.grad[1, :n]) > 0
    E2 = E.clone(); E2[1, n:] += 3.0
    with torch.no_grad():
        assert float(orc.task_loss(th, E2, lab, shape)) == float(loss.detach())
    # the mean is over real predictions, not over B*L
    lab_all = lab.copy(); lab_all[1, n:] = 0
    with torch.no_grad():
        assert abs(float(orc.task_loss(th, E, lab_all, shape)) - float(loss.detach())) > 1e-6


def test_refreshed_cache_makes_one_step_windows_end_to_end_training():
    # windows of one step, SGD on the encoder, cache refreshed after the update: when the next batch only uses items the
    # previous one touched, its loss and gradient are those of end-to-end training at the updated parameters (Eq. 4
    # with the parameters of the current step); without the refresh the cache is one update stale and they differ
    shape = small_shape(pooling="cls")
    ce, tk, toks, ids, lab = make(shape, seed=14)
    cache = orc.encode_all(shape, ce, toks, range(shape.n_items))
    lr_c = 0.05
    w1 = orc.multistep_window(shape, ce, tk, toks, [(ids, lab)], cache, lr_task=0.0, lr_ce=lr_c, refresh_after_update=True)
    lab2 = 1 - lab
    w2 = orc.multistep_window(shape, w1["ce_params"], tk, toks, [(ids, lab2)], w1["cache"], lr_task=0.0)
    e2e = orc.e2e_step(shape, w1["ce_params"], tk, toks, ids, lab2)
    assert abs(w2["losses"][0] - e2e["loss"]) < 1e-12
    for k in e2e["grad_ce"]:
        np.testing.assert_allclose(w2["grad_ce"][k], e2e["grad_ce"][k], rtol=1e-9, atol=1e-12)
    for k in ce:      # and the step itself was plain SGD with the window's gradient
        np.testing.assert_allclose(w1["ce_params"][k], np.asarray(ce[k], np.float64) - lr_c * w1["grad_ce"][k], rtol=0, atol=0)
    stale = orc.multistep_window(shape, ce, tk, toks, [(ids, lab)], cache, lr_task=0.0, lr_ce=lr_c)
    s2 = orc.multistep_window(shape, stale["ce_params"], tk, toks, [(ids, lab2)], stale["cache"], lr_task=0.0)
    assert abs(s2["losses"][0] - e2e["loss"]) > 1e-7


# ---- additive-attention pooling of an item's tokens ---------------------------------------------------------------------

def test_additive_pooling_special_cases_and_finite_differences():
    shape = small_shape(pooling="additive", d_a=6, l_t=5)
    ce, tk, toks, ids, lab = make(shape, seed=16)
    ce = OrderedDict((k, np.asarray(v, np.float64)) for k, v in ce.items())
    th = orc.as_torch(ce, T64, requires_grad=False)
    # q = 0: every score is equal, the pooled vector is the plain mean of the token outputs
    z = OrderedDict(ce); z["pool_qa"] = np.zeros_like(ce["pool_qa"])
    mean_shape = shape.replace(pooling="mean")
    a = orc.encode_all(shape, z, toks, [0, 3])
    b = orc.encode_all(mean_shape, {k: v for k, v in ce.items() if not k.startswith("pool_")}, toks, [0, 3])
    np.testing.assert_allclose(a, b, rtol=1e-13)
    # one dominant score: a huge q along tanh's saturated sign pattern of one token picks that token's output (convex
    # combination in general: inside the hull of the token outputs)
    with torch.no_grad():
        h = orc.ce_forward(th, toks[1], shape)
        x = th["tok_emb"][torch.as_tensor(toks[1], dtype=torch.long)] + th["pos_emb"]
        x = orc.layer_norm(x, th["emb_ln_g"], th["emb_ln_b"])
        for l in range(shape.n_layers):
            x = orc.transformer_layer(x, th, f"l{l}.", shape.n_heads, causal=False)
        al = torch.linalg.lstsq(x.T, h[:, None]).solution[:, 0]            # h = sum alpha_s x_s has a solution ...
        assert torch.allclose(x.T @ al, h, atol=1e-10)
        sc = torch.tanh(x @ th["pool_wa"].T + th["pool_ba"]) @ th["pool_qa"]
        want = torch.softmax(sc, 0)                                           # ... and it is the library softmax of the scores
        assert torch.allclose(want @ x, h, atol=1e-13) and abs(float(want.sum()) - 1) < 1e-14
    # gradients of the end-to-end step through the pooling parameters against central differences
    res = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    def loss_at(params):
        thp = orc.as_torch(params, T64, requires_grad=False)
        with torch.no_grad():
            E = torch.stack([torch.stack([orc.ce_forward(thp, toks[int(i)], shape) for i in row]) for row in ids])
            return float(orc.task_loss(orc.as_torch(tk, T64, requires_grad=False), E, lab, shape))
    rng = np.random.default_rng(0)
    for name in ("pool_wa", "pool_ba", "pool_qa", "l0.w1"):
        for fi in rng.integers(0, ce[name].size, 2):
            idx = np.unravel_index(fi, ce[name].shape)
            up = OrderedDict((k, v.copy()) for k, v in ce.items()); up[name][idx] += 1e-6
            dn = OrderedDict((k, v.copy()) for k, v in ce.items()); dn[name][idx] -= 1e-6
            fd = (loss_at(up) - loss_at(dn)) / 2e-6
            assert abs(fd - res["grad_ce"][name][idx]) <= 1e-7 + 1e-5 * abs(fd), (name, idx, fd, res["grad_ce"][name][idx])


def test_user_self_attention_layer_is_the_library_attention_with_empty_slots_masked():
    # NR with one self-attention layer over the clicked items (Appendix D): the scores equal those computed from
    # torch.nn.MultiheadAttention run over ALL history slots with the empty ones masked as keys, its rows for
    # the clicked slots (plus the residual) fed to the user vector
    shape = small_shape(task="nr", task_layers=1, task_heads=4, task_attn_only=True, n_cand=3, L=9, d_a=6, B=1)
    d = shape.d
    tk = synth.task_params(shape, 5, sigma=0.4, plain=False)
    assert list(tk)[:4] == ["t0.wqkv", "t0.bqkv", "t0.wo", "t0.bo"] and list(tk)[-3:] == ["wa", "ba", "qa"]
    th = orc.as_torch(tk, T64, False)
    E = torch.randn(9, d, dtype=T64, generator=torch.Generator().manual_seed(11))
    clicked = [0, 2, 3, 5]                                   # slots 1 and 4 are empty
    mha = torch.nn.MultiheadAttention(d, 4, dropout=0.0, batch_first=True, dtype=T64)
    with torch.no_grad():
        mha.in_proj_weight.copy_(th["t0.wqkv"]); mha.in_proj_bias.copy_(th["t0.bqkv"])
        mha.out_proj.weight.copy_(th["t0.wo"]); mha.out_proj.bias.copy_(th["t0.bo"])
        pad = torch.ones(1, 6, dtype=torch.bool); pad[0, clicked] = False
        y = E[None, :6] + mha(E[None, :6], E[None, :6], E[None, :6], key_padding_mask=pad, need_weights=False)[0]
        want = E[6:] @ orc.nr_user_vector(th, y[0, clicked])
        got = orc.nr_scores(th, E[clicked], E[6:], shape)
    np.testing.assert_allclose(got.numpy(), want.numpy(), rtol=1e-11)
    # and task_loss routes the same way: label -1 marks the empty slots
    lab = np.zeros((1, 9), np.int32); lab[0, [1, 4]] = -1
    with torch.no_grad():
        loss = orc.task_loss(th, E[None], lab, shape)
    assert float(loss) == pytest.approx(float(torch.nn.functional.cross_entropy(want[None], torch.zeros(1, dtype=torch.long))), rel=1e-11)
    # the layer matters: without it the scores differ
    with torch.no_grad():
        assert float((orc.nr_scores(th, E[clicked], E[6:], shape.replace(task_layers=0)) - got).abs().max()) > 1e-3


def test_empty_click_slots_are_left_out():
    # NR: history slots with label -1 take no part: the loss equals that of the same users with those rows removed
    shape = small_shape(task="nr", task_layers=0, n_cand=2, L=7, d_a=6, B=2, pooling="cls")
    tk = synth.task_params(shape, 3, sigma=0.3, plain=False)
    th = orc.as_torch(tk, T64)
    E = torch.randn(2, 7, shape.d, dtype=T64, generator=torch.Generator().manual_seed(5))
    lab = np.zeros((2, 7), np.int32)
    lab[0, [1, 3]] = -1
    lab[1, 4] = -1
    Eg = E.clone().requires_grad_(True)
    loss = orc.task_loss(th, Eg, lab, shape)
    loss.backward()
    with torch.no_grad():
        keep0 = [0, 2, 4, 5, 6]; keep1 = [0, 1, 2, 3, 5, 6]
        l0 = orc.task_loss(th, E[0:1, keep0], np.zeros((1, 5), np.int32), shape.replace(B=1, L=5))
        l1 = orc.task_loss(th, E[1:2, keep1], np.zeros((1, 6), np.int32), shape.replace(B=1, L=6))
    assert abs(float(loss.detach()) - (float(l0) + float(l1)) / 2) < 1e-13
    assert torch.count_nonzero(Eg.grad[0, [1, 3]]) == 0 and torch.count_nonzero(Eg.grad[1, 4]) == 0
    assert torch.count_nonzero(Eg.grad[0, 0]) > 0
