"""Pins for the oracle's optimiser (Adam with the Noam learning-rate scheme, Appendix D of the paper).

None of them re-types the oracle's formula: the Noam curve is checked at values that follow from its definition by
hand, the Adam update against torch.optim.Adam (a library routine, constant rate) and against the closed form of the
first update from a zero state, and planted mistakes in a copy of the routine must fail these checks.
"""
import math

import numpy as np
import pytest
import torch

from oracle import gram_oracle as O


def test_noam_values():
    # rate proportional to min(t^-0.5, t * w^-1.5), scaled to peak at t = w (Vaswani et al. 2017, Eq. 3)
    peak, w = 1e-4, 100
    assert O.noam_rate(w, peak, w) == pytest.approx(peak, rel=1e-15)
    assert O.noam_rate(1, peak, w) == pytest.approx(peak / 100, rel=1e-15)          # linear warm-up
    assert O.noam_rate(50, peak, w) == pytest.approx(peak / 2, rel=1e-15)
    assert O.noam_rate(400, peak, w) == pytest.approx(peak / 2, rel=1e-15)          # inverse square root decay
    assert O.noam_rate(10000, peak, w) == pytest.approx(peak / 10, rel=1e-15)
    rates = [O.noam_rate(t, peak, w) for t in range(1, 1000)]
    assert int(np.argmax(rates)) + 1 == w                                            # the maximum sits at t = warmup
    # ratio of consecutive rates in the decay is sqrt(t / (t + 1)): the t^-0.5 law
    assert rates[500] / rates[499] == pytest.approx(math.sqrt(500 / 501), rel=1e-12)
    assert O.noam_rate(7, 3e-3, 0) == 3e-3                                           # no warm-up: constant


def test_adam_first_step_closed_form():
    # from m = v = 0 the bias-corrected moments of the first update are g and g^2: step = rate * g / (|g| + eps)
    rng = np.random.default_rng(0)
    w = rng.standard_normal(50); g = rng.standard_normal(50) * 10.0 ** rng.integers(-6, 3, 50)
    g[:3] = 0.0
    w0 = w.copy(); m = np.zeros(50); v = np.zeros(50)
    O.adam_update(w, g, m, v, 1, 0.01, 0.9, 0.999, 1e-8)
    np.testing.assert_allclose(w0 - w, 0.01 * g / (np.abs(g) + 1e-8), rtol=1e-9, atol=1e-18)
    assert np.all(w[:3] == w0[:3])                                                   # zero gradient: no movement


@pytest.mark.parametrize("betas,eps", [((0.9, 0.999), 1e-8), ((0.8, 0.95), 1e-6)])
def test_adam_matches_library_routine(betas, eps):
    rng = np.random.default_rng(1)
    w = rng.standard_normal((7, 5)); m = np.zeros_like(w); v = np.zeros_like(w)
    p = torch.tensor(w.copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=3e-3, betas=betas, eps=eps)
    for t in range(1, 12):
        g = rng.standard_normal((7, 5)) * (1.0 + 0.1 * t)
        O.adam_update(w, g, m, v, t, 3e-3, betas[0], betas[1], eps)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(w, p.detach().numpy(), rtol=1e-10, atol=1e-13)


def _broken_adam(kind):
    def f(w, g, m, v, t, rate, b1=0.9, b2=0.999, eps=1e-8):
        m[...] = b1 * m + (1 - b1) * g
        v[...] = b2 * v + (1 - b2) * (g if kind == "no_square" else g * g)
        mh = m if kind == "no_bias_correction_m" else m / (1 - b1 ** t)
        vh = v if kind == "no_bias_correction_v" else v / (1 - b2 ** t)
        den = np.sqrt(vh + eps) if kind == "eps_inside" else np.sqrt(np.abs(vh)) + eps
        w[...] = w + rate * mh / den if kind == "wrong_sign" else w - rate * mh / den
    return f


@pytest.mark.parametrize("kind", ["no_square", "no_bias_correction_m", "no_bias_correction_v", "eps_inside", "wrong_sign"])
def test_planted_mistakes_fail_the_pins(kind):
    f = _broken_adam(kind)
    rng = np.random.default_rng(2)
    g = rng.standard_normal(40) * 10.0 ** rng.integers(-6, 1, 40)
    w = np.zeros(40); m = np.zeros(40); v = np.zeros(40)
    f(w, g, m, v, 1, 0.01)
    ok_first = np.allclose(-w, 0.01 * g / (np.abs(g) + 1e-8), rtol=1e-9, atol=1e-18)
    w2 = np.zeros(40); m2 = np.zeros(40); v2 = np.zeros(40)
    p = torch.zeros(40, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=0.01)
    ok_lib = True
    for t in range(1, 5):
        gt = g * t
        f(w2, gt, m2, v2, t, 0.01)
        p.grad = torch.tensor(gt); opt.step()
        ok_lib = ok_lib and np.allclose(w2, p.detach().numpy(), rtol=1e-10, atol=1e-13)
    assert not (ok_first and ok_lib)


def test_train_steps_adam_moves_against_the_gradient():
    # one step from zero state: every parameter with a non-negligible gradient moves by rate(1) against its sign
    from paper_2204_04179_b200 import synth
    sub = synth.config("tiny").replace(B=2, L=6)
    ce = synth.encoder_params(sub, seed=3); tk = synth.task_params(sub, seed=4)
    toks = synth.item_tokens(5, sub.n_items, sub.l_t, sub.vocab)
    ids, labels = synth.batch(sub, seed=6)
    r = O.e2e_step(sub, ce, tk, toks, ids, labels)
    ce1, tk1, losses = O.train_steps_adam(sub, ce, tk, toks, [(ids, labels)], 1e-3, 2e-3, 10)
    assert losses[0] == pytest.approx(r["loss"])
    for new, old, grads, peak in ((ce1, ce, r["grad_ce"], 1e-3), (tk1, tk, r["grad_task"], 2e-3)):
        for k in old:
            g = grads[k]; big = np.abs(g) > 1e-5
            step = new[k] - np.asarray(old[k], dtype=np.float64)
            np.testing.assert_allclose(step[big], -np.sign(g[big]) * peak / 10, rtol=1e-3)
            assert np.all(step[g == 0] == 0)
