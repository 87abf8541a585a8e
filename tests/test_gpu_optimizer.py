"""Adam with the Noam scheme (Appendix D) on the GPU against the oracle: the update kernel element by element, and
whole training steps through gram_step."""
import numpy as np
import pytest
import torch

from oracle import gram_oracle as O
from paper_2204_04179_b200 import binding, synth
from tests import gram_helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [0, 1, 3, 4, 1000, 4 * 70001 + 3])       # empty, below one vector, ragged tail, several blocks
@pytest.mark.parametrize("with_bf16", [False, True])
def test_adam_update_matches_oracle(n, with_bf16):
    cfg = binding.GramConfig(); cfg.n_items = 8; cfg.P_max = 8; cfg.d = 8
    g = binding.Gram(cfg)
    rng = np.random.default_rng(n + 7)
    w = rng.standard_normal(n).astype(np.float32)
    m = (rng.standard_normal(n) * 0.1).astype(np.float32)
    v = (rng.random(n) * 0.01).astype(np.float32)
    gr = (rng.standard_normal(n) * 10.0 ** rng.integers(-5, 2, n)).astype(np.float32)
    gr[: n // 10] = 0.0
    dw, dm, dv, dg = (torch.from_numpy(a.copy()).to(H.DEV) for a in (w, m, v, gr))
    wb = torch.zeros(n, dtype=torch.bfloat16, device=H.DEV) if with_bf16 else None
    w64, m64, v64 = w.astype(np.float64), m.astype(np.float64), v.astype(np.float64)
    for t in (1, 2, 50):
        m_prev, v_prev, w_prev = m64.copy(), v64.copy(), w64.copy()
        g.adam_update(dw, dg, dm, dv, t, 3e-3, 0.9, 0.98, 1e-6, w_bf16=wb)
        O.adam_update(w64, gr, m64, v64, t, 3e-3, 0.9, 0.98, 1e-6)
        g.sync()
        # fp32 against fp64.  Each moment is a sum of two rounded products: a few units of 2^-24 of the larger term
        # (the sum itself may cancel).  The step is rate * m^ / (sqrt(v^) + eps): the moments' errors carried through,
        # plus a few ulp of the quotient; and w - step rounds once more.
        g64 = gr.astype(np.float64)
        tol_m = 3e-7 * (np.abs(m_prev) + np.abs(g64)) + 1e-30
        tol_v = 3e-7 * (np.abs(v_prev) + g64 * g64) + 1e-30
        assert np.all(np.abs(dm.cpu().numpy() - m64) <= tol_m)
        assert np.all(np.abs(dv.cpu().numpy() - v64) <= tol_v)
        c1, c2 = 1 / (1 - 0.9 ** t), 1 / (1 - 0.98 ** t)
        den = np.sqrt(v64 * c2) + 1e-6
        step = 3e-3 * np.abs(m64) * c1 / den
        tol_w = 3e-3 * (tol_m * c1 / den) + step * (0.5 * tol_v / np.maximum(v64, 1e-30) + 1e-6) + 1.2e-7 * np.abs(w_prev) + 1e-12
        assert np.all(np.abs(dw.cpu().numpy() - w64) <= tol_w)
        if with_bf16:
            assert torch.equal(wb, dw.to(torch.bfloat16))           # round-to-nearest-even copy of the new parameters
        # continue from the GPU's state so that rounding does not accumulate into the comparison
        w64, m64, v64 = (a.cpu().numpy().astype(np.float64) for a in (dw, dm, dv))
    g.close()


def test_adam_update_rejects_bad_arguments():
    cfg = binding.GramConfig(); cfg.n_items = 8; cfg.P_max = 8; cfg.d = 8
    g = binding.Gram(cfg)
    a = torch.zeros(8, device=H.DEV)
    with pytest.raises(binding.GramError):
        g.adam_update(a, a, a, a, 0, 1e-3)                          # the update count starts at 1
    with pytest.raises(binding.GramError):
        g.adam_update(a, a, a, a, 1, 1e-3, beta1=1.0)
    with pytest.raises(binding.GramError):
        g.adam_update(a[1:], a[1:], a[1:], a[1:], 1, 1e-3)          # not 16-byte aligned
    g.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_training_steps_with_adam_follow_the_oracle(dtype):
    """Three gram_step calls with Adam + Noam against end-to-end training with the oracle's optimiser.  Adam divides by
    sqrt(v): where a gradient element is at rounding-noise level the direction of its step is not determined, so the
    comparison is over elements whose gradient is clear of the noise in every step; the rest may differ by at most
    the sum of the rates."""
    shape = synth.config("tiny").replace(dtype=dtype)
    ce, tk, toks, _, _ = H.make_inputs(shape, seed=11)
    batches = [synth.batch(shape, 11, step=s) for s in range(3)]
    peak_ce, peak_tk, warm = 2e-3, 1e-3, 2
    g = H.make_ctx(shape, ce, tk, toks, optimizer=binding.GRAM_OPT_ADAM, lr_ce=peak_ce, lr_task=peak_tk, noam_warmup=warm)
    losses = []
    for ids, lab in batches:
        rep = g.step(torch.from_numpy(np.ascontiguousarray(ids, np.int32)).to(H.DEV),
                     torch.from_numpy(np.ascontiguousarray(lab, np.int32)).to(H.DEV), ids.shape[0])
        losses.append(rep.loss)
    got_ce = synth.unflatten(g.get_params(binding.GRAM_MODULE_CE), synth.encoder_param_spec(shape))
    got_tk = synth.unflatten(g.get_params(binding.GRAM_MODULE_TASK), synth.task_param_spec(shape))
    g.close()
    # the oracle's trajectory, and per step which gradient elements are clear of the noise
    ce64 = {k: np.array(a, np.float64) for k, a in ce.items()}; tk64 = {k: np.array(a, np.float64) for k, a in tk.items()}
    st = {}
    clear_ce = {k: np.ones(a.shape, bool) for k, a in ce.items()}; clear_tk = {k: np.ones(a.shape, bool) for k, a in tk.items()}
    tol_g = 1e-4 if dtype == "f32" else 5e-2
    want_losses = []
    for t, (ids, lab) in enumerate(batches, start=1):
        r = O.e2e_step(shape, ce64, tk64, toks, ids, lab)
        want_losses.append(r["loss"])
        for params, grads, peak, clear in ((ce64, r["grad_ce"], peak_ce, clear_ce), (tk64, r["grad_task"], peak_tk, clear_tk)):
            for k in params:
                mm, vv = st.setdefault((id(params), k), (np.zeros_like(params[k]), np.zeros_like(params[k])))
                clear[k] &= (np.abs(grads[k]) > tol_g * np.abs(grads[k]).max()) | (grads[k] == 0)
                O.adam_update(params[k], grads[k], mm, vv, t, O.noam_rate(t, peak, warm))
    total_rate = lambda peak: sum(O.noam_rate(t, peak, warm) for t in (1, 2, 3))
    rel = 2e-3 if dtype == "f32" else 0.25        # of the distance moved; bf16 gradients carry up to 2e-2 error each step
    np.testing.assert_allclose(losses, want_losses, rtol=1e-4 if dtype == "f32" else 2e-2)
    for got, want, start, clear, peak in ((got_ce, ce64, ce, clear_ce, peak_ce), (got_tk, tk64, tk, clear_tk, peak_tk)):
        for k in want:
            moved_w = want[k] - np.asarray(start[k], np.float64)
            moved_g = np.asarray(got[k], np.float64) - np.asarray(start[k], np.float64)
            # Adam's bound on one step: rate * max(1, (1 - beta1) / sqrt(1 - beta2)) (Kingma & Ba, Section 2.1)
            assert np.all(np.abs(moved_g) <= total_rate(peak) * 0.1 / np.sqrt(0.001) * 1.001 + 1e-7), k
            c = clear[k]
            if c.any():
                assert np.abs(moved_g[c] - moved_w[c]).max() <= rel * total_rate(peak) + 1e-7, k
