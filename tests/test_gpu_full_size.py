"""Parity at the full size of the knowledge-tracing workload (B = 256 histories x L = 100 positions, 10,000 items,
BERT-base-shaped encoder, bf16), in the launch configuration the benchmark times (all unique items in one encoder
pass), stage by stage through the C ABI.

The per-occurrence oracle cannot run 25,600 encoder calls, so each stage is compared on outputs the oracle can compute
one by one, from inputs the oracle builds itself, and on properties that hold at any size:

* dedup: every index output against the oracle, bit-exact;
* encode: sampled rows of H against the oracle's encoder forward;
* gather: E[p] == H[inverse[p]] bit-exact for every position;
* task module: the gradient rows dL/dE of one whole history against the oracle (histories are independent in the
  knowledge-tracing module, and the loss is a mean over all B*L predictions);
* accumulate: sampled rows of G against a float64 sum over that item's occurrences, and conservation of column sums;
* encoder backward: the VJP is linear in its cotangent, so a cotangent that is zero except for a few sampled items
  yields exactly those items' gradient, which the oracle computes as the gradient of the pseudo-loss (Eq. 9) with
  pseudo-targets h - g; the kernels still run over all unique items' activations.  With token-0 pooling the last
  LayerNorm's bias gradient is the plain column sum of G.
"""
import numpy as np
import pytest
import torch

from oracle import gram_oracle as orc
from paper_2204_04179_b200 import binding, synth
from tests import gram_helpers as gh

pytestmark = pytest.mark.gpu
DEV = gh.DEV
TOL = 2e-2


def _row_err(got, want):
    got = np.asarray(got, np.float64); want = np.asarray(want, np.float64)
    return float(np.abs(got - want).max() / np.abs(want).max())


def test_kt_workload_stage_by_stage():
    shape = synth.config("kt")
    seed = 0
    ce = synth.encoder_params(shape, seed)
    tk = synth.task_params(shape, seed)
    toks = synth.item_tokens(seed, shape.n_items, shape.l_t, shape.vocab)
    ids, lab = synth.batch(shape, seed, step=0)
    P, d, B, L = ids.size, shape.d, shape.B, shape.L
    assert (B, L, shape.n_items, d, shape.n_layers) == (256, 100, 10_000, 768, 12)
    g = gh.make_ctx(shape, ce, tk, toks, ce_micro_batch=5120)
    rng = np.random.default_rng(5)

    # ---- stage 1 ----
    ids_d = torch.from_numpy(ids.ravel().copy()).to(DEV)
    lab_d = torch.from_numpy(lab.ravel().copy()).to(DEV)
    cap = min(P, shape.n_items)
    unique = torch.zeros(cap, dtype=torch.int32, device=DEV); inverse = torch.zeros(P, dtype=torch.int32, device=DEV)
    perm = torch.zeros(P, dtype=torch.int32, device=DEV); seg = torch.zeros(cap + 1, dtype=torch.int32, device=DEV)
    nu = torch.zeros(1, dtype=torch.int32, device=DEV)
    g.dedup(ids_d, shape.n_items, unique, inverse, perm, seg, nu)
    g.sync()
    U = int(nu.item())
    w_unique, w_inverse, w_perm, w_seg = orc.unique_inverse(ids)
    assert U == len(w_unique) and 4000 < U <= 5120
    assert np.array_equal(unique[:U].cpu().numpy(), w_unique) and np.array_equal(inverse.cpu().numpy(), w_inverse)
    assert np.array_equal(perm.cpu().numpy(), w_perm) and np.array_equal(seg[:U + 1].cpu().numpy(), w_seg)

    # ---- stage 2: sampled encodings ----
    H = torch.zeros(U, d, device=DEV)
    g.encode_unique(None, unique, U, H, save_activations=True)
    g.sync()
    counts = np.diff(w_seg)
    sample_u = sorted({0, U - 1, int(np.argmax(counts))} | {int(x) for x in rng.integers(0, U, 3)})
    want_H = orc.encode_all(shape, ce, toks, [w_unique[u] for u in sample_u])
    H_np = H.cpu().numpy()
    for k, u in enumerate(sample_u):
        assert _row_err(H_np[u], want_H[k]) <= TOL, (u, _row_err(H_np[u], want_H[k]))

    # ---- stage 3: every position, exact ----
    E = torch.zeros(P, d, device=DEV)
    g.gather(H, inverse, E)
    g.sync()
    assert torch.equal(E, H[inverse.long()])

    # ---- task module: one whole history against the oracle ----
    dE = torch.zeros(P, d, device=DEV); loss = torch.zeros(1, device=DEV)
    g.task(E, lab_d, B, dE, loss)
    g.sync()
    b = int(rng.integers(0, B))
    hist_items, hist_inv = np.unique(ids[b], return_inverse=True)
    E_b = orc.encode_all(shape, ce, toks, hist_items)[hist_inv]                      # the oracle's own encodings
    th_cf = orc.as_torch(tk)
    E_t = torch.tensor(E_b[None], dtype=torch.float64, requires_grad=True)
    loss_b = orc.task_loss(th_cf, E_t, lab[b:b + 1], shape.replace(B=1))             # mean over this history's L
    loss_b.backward()
    want_dE_b = E_t.grad[0].numpy() / B                                              # mean over all B*L predictions
    got_dE_b = dE.view(B, L, d)[b].cpu().numpy()
    assert _row_err(got_dE_b, want_dE_b) <= TOL, _row_err(got_dE_b, want_dE_b)
    assert np.isfinite(float(loss.item())) and 0.3 < float(loss.item()) < 1.5       # near log 2 at this initialisation

    # ---- stage 4 ----
    G = torch.zeros(U, d, device=DEV)
    g.accumulate(dE, perm, seg, U, G)
    g.sync()
    dE64 = dE.double()
    col = dE64.sum(0)
    assert float((G.double().sum(0) - col).abs().max()) <= 1e-5 * float(dE64.abs().sum(0).max())
    for u in sample_u:
        rows = torch.from_numpy(w_perm[w_seg[u]:w_seg[u + 1]].astype(np.int64)).to(DEV)
        want = dE64[rows].sum(0)
        bound = float(dE64[rows].abs().sum(0).max()) * len(rows) * 2.0 ** -24 + 1e-12
        assert float((G[u].double() - want).abs().max()) <= bound, u

    # ---- stage 5: the VJP of a few sampled items, computed over the full set of saved activations ----
    picks = sorted({int(x) for x in rng.integers(0, U, 3)})
    items = [int(w_unique[u]) for u in picks]
    g_rows = rng.standard_normal((len(picks), d))
    G_sparse = torch.zeros(U, d, device=DEV)
    G_sparse[torch.tensor(picks, device=DEV)] = torch.from_numpy(g_rows).float().to(DEV)
    g.zero_grads(binding.GRAM_MODULE_CE)
    g.encoder_backward(G_sparse, unique, U)
    gce, _ = gh.gpu_grads(g, shape)
    h = orc.encode_all(shape, ce, toks, items)
    _, want_g = orc.pseudo_loss_grad(shape, ce, toks, items, h - g_rows)             # Eq. 9 with h~ = h - g
    worst, name = gh.worst_rel_err(gce, want_g)
    print("full-size encoder backward, 3 sampled items: worst tensor", name, worst)
    assert worst <= TOL, (name, worst)

    # the full cotangent: the last LayerNorm's bias gradient is the column sum of G (token-0 pooling)
    g.zero_grads(binding.GRAM_MODULE_CE)
    g.encoder_backward(G, unique, U)
    gce, _ = gh.gpu_grads(g, shape)
    last = f"l{shape.n_layers - 1}.ln2_b"
    want_b = G.double().sum(0).cpu().numpy()
    assert _row_err(gce[last], want_b) <= 1e-4
    for k, v in gce.items():
        assert np.all(np.isfinite(v)), k
    g.close()


def test_kt_workload_step_equals_stages_and_micro_batches():
    """gram_step at full size: the same report counts as the oracle's index work, and gradients that do not depend
    on how the unique items are cut into encoder passes (a property that holds at any size)."""
    shape = synth.config("kt")
    seed = 0
    ce = synth.encoder_params(shape, seed)
    tk = synth.task_params(shape, seed)
    toks = synth.item_tokens(seed, shape.n_items, shape.l_t, shape.vocab)
    ids, lab = synth.batch(shape, seed, step=1)
    U = len(np.unique(ids))
    grads = []
    for mb in (5120, 1536):
        rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab, ce_micro_batch=mb)
        assert rep.n_unique == U and rep.n_encoded == U and rep.n_positions == ids.size
        grads.append((rep.loss, gce, gtk))
    assert abs(grads[0][0] - grads[1][0]) <= 1e-5 * abs(grads[0][0])
    for k in grads[0][1]:
        assert gh.rel_err(grads[1][1][k], grads[0][1][k]) <= 2e-3, k
    for k in grads[0][2]:
        assert np.array_equal(grads[1][2][k], grads[0][2][k]), k        # the task module does not see the cut


def test_bf16_step_is_bit_reproducible():
    """Two contexts, the same state and batch: every gradient and the loss agree bit for bit on the tensor-core path (split
    weight-gradient products, bias sums left by fused producers, attention column sums: all added in fixed orders)."""
    shape = synth.config("kt").replace(B=16, n_items=2000, n_layers=2)
    ce = synth.encoder_params(shape, 3); tk = synth.task_params(shape, 3)
    toks = synth.item_tokens(3, shape.n_items, shape.l_t, shape.vocab)
    ids, lab = synth.batch(shape, 3)
    runs = [gh.gpu_single_step(shape, ce, tk, toks, ids, lab) for _ in range(2)]
    assert runs[0][0].loss == runs[1][0].loss
    for which in (1, 2):
        for k in runs[0][which]:
            assert np.array_equal(runs[0][which][k], runs[1][which][k]), k
            assert np.all(np.isfinite(runs[0][which][k])), k


def test_kt_multistep_window_full_size():
    """Multi-step GRAM at the full size of the knowledge-tracing workload: K = 8, a 10,000 x 768 fp32 table, a bf16 cache,
    one encoder pass over the ~9,700 touched items in two micro-batches (Section 4.2; Algorithm 1 with N = 8).

    * before the window: sampled cache rows against the oracle's encoder, rounded to bf16;
    * steps 1..7 through gram_step: the number of touched items and the touched bitmap against the union of the batches'
      IDs (brute force, bit-exact); sampled table rows (the hottest item, an item touched once, random ones) against a
      float64 sum of that item's rows of dL/dE, step by step, where each step's dL/dE comes from the task module run on
      the same cached encodings with the task parameters of that step (gram_task, which changes no parameter);
    * step 8: the encoder pass is linear in the table, so with a table that is zero except for three sampled items
      (imported through gram_state_import, touched bits kept) and an all-padding last batch (which adds nothing), the
      parameter gradient is those three items' VJP, which the oracle computes as the gradient of Eq. 9's pseudo-loss;
      the kernels still run over every touched item.  The encoder parameters are replaced before that step, so the cache
      rows of touched items must afterwards hold the NEW encodings and the rows of untouched items the old ones."""
    shape = synth.config("kt_multistep")
    seed, K = 0, 8
    ce = synth.encoder_params(shape, seed); tk = synth.task_params(shape, seed)
    toks = synth.item_tokens(seed, shape.n_items, shape.l_t, shape.vocab)
    N, d, B, L = shape.n_items, shape.d, shape.B, shape.L
    assert (K, N, d) == (shape.K, 10_000, 768)
    g = gh.make_ctx(shape, ce, tk, toks, ce_micro_batch=5120, lr_task=1e-3)
    g.cache_fill()
    _, _, cache0 = g.get_window(want_table=False, want_touched=False)
    rng = np.random.default_rng(11)
    some = sorted({int(x) for x in rng.integers(0, N, 4)})
    want = orc.round_to_bf16(orc.encode_all(shape, ce, toks, some))
    for k, i in enumerate(some):
        assert _row_err(cache0[i], want[k]) <= TOL, i
    cache_d = torch.from_numpy(cache0).to(DEV)

    batches = [synth.batch(shape, seed, step=k) for k in range(K)]
    union = set()
    table64 = {}                                                # item -> float64 sum, for the sampled items only
    all_ids = np.concatenate([b[0].ravel() for b in batches[:K - 1]])
    vals, cnts = np.unique(all_ids, return_counts=True)
    watch = sorted({int(vals[np.argmax(cnts)]), int(vals[np.argmin(cnts)])} | {int(x) for x in rng.choice(vals, 4, replace=False)})
    for i in watch:
        table64[i] = np.zeros(d)
    for k in range(K - 1):
        ids, lab = batches[k]
        ids_d = torch.from_numpy(ids).to(DEV); lab_d = torch.from_numpy(lab).to(DEV)
        # this step's dL/dE, from the stage call, before the step itself updates the task parameters
        E = cache_d[ids_d.view(-1).long()].contiguous()
        dE = torch.zeros(B * L, d, device=DEV); loss = torch.zeros(1, device=DEV)
        g.task(E, lab_d.view(-1), B, dE, loss)
        g.sync()
        flat = ids.ravel()
        for i in watch:
            rows = np.nonzero(flat == i)[0]
            if len(rows):
                table64[i] += dE[torch.from_numpy(rows).to(DEV)].double().sum(0).cpu().numpy()
        rep = g.step(ids_d, lab_d, B)
        union |= set(int(x) for x in flat)
        assert rep.encoder_pass == 0 and rep.n_touched == len(union) and rep.n_unique == len(np.unique(flat))
        assert abs(rep.loss - float(loss.item())) <= 1e-6 * abs(rep.loss)
    table, touched, cache, steps = g.state_export()
    assert steps == K - 1
    bits = np.unpackbits(touched.view(np.uint8), bitorder="little")[:N].astype(bool)
    assert np.array_equal(np.nonzero(bits)[0], np.array(sorted(union)))          # bit-exact touched set
    assert np.array_equal(cache, cache0)                                           # the cache does not move inside a window
    assert not table[~bits].any()
    for i in watch:
        n_occ = int((all_ids == i).sum())
        bound = np.abs(table64[i]).max() * n_occ * 2.0 ** -22 + 1e-9
        assert np.abs(table[i] - table64[i]).max() <= bound, (i, n_occ)

    # ---- step 8: sparse table, new encoder parameters, a batch that adds nothing ----
    picks = sorted(int(x) for x in rng.choice(np.array(sorted(union)), 3, replace=False))
    sparse = np.zeros_like(table)
    sparse[picks] = table[picks]
    g.state_import(sparse, touched, None, K - 1)
    ce2 = synth.encoder_params(shape, seed + 1)                                    # other parameters than the cache was built with
    g.set_params(binding.GRAM_MODULE_CE, synth.flatten(ce2))
    ids8 = batches[K - 1][0]
    lab8 = np.full_like(batches[K - 1][1], -1)                                     # every position is padding: no prediction, dL/dE = 0
    rep = g.step(torch.from_numpy(ids8).to(DEV), torch.from_numpy(lab8).to(DEV), B)
    union8 = union | set(int(x) for x in ids8.ravel())
    assert rep.encoder_pass == 1 and rep.n_touched == len(union8) == rep.n_encoded and rep.n_touched > 9000
    gce, _ = gh.gpu_grads(g, shape)
    h = orc.encode_all(shape, ce2, toks, picks)
    _, want_g = orc.pseudo_loss_grad(shape, ce2, toks, picks, h - table[picks].astype(np.float64))
    worst, name = gh.worst_rel_err(gce, want_g)
    print("Multi-step encoder pass at full size, 3 sampled table rows: worst tensor", name, worst)
    assert worst <= TOL, (name, worst)
    table_after, touched_after, cache_after, steps = g.state_export()
    assert steps == 0 and not table_after.any() and not touched_after.any()       # the window is closed
    bits8 = np.zeros(N, bool); bits8[sorted(union8)] = True
    assert np.array_equal(cache_after[~bits8], cache0[~bits8])                     # untouched rows keep their old encodings
    fresh = sorted(int(x) for x in rng.choice(np.array(sorted(union8)), 4, replace=False))
    want = orc.round_to_bf16(orc.encode_all(shape, ce2, toks, fresh))
    for k, i in enumerate(fresh):
        assert _row_err(cache_after[i], want[k]) <= TOL, i
        assert _row_err(cache_after[i], cache0[i]) > 0.1                           # and they really are the new parameters' values
    g.close()


def test_nr_workload_stage_by_stage():
    """The news-recommendation workload at full size (64 users x 55 positions over 100,000 items, 32-token titles), stage by
    stage like the knowledge-tracing one: dedup bit-exact at N = 10^5, sampled encodings, the gather on every position, one
    user's rows of dL/dE against the oracle (users are independent; the loss is a mean over the 64 users), sampled
    segment sums, and the encoder VJP of three sampled items with every other cotangent row zero."""
    shape = synth.config("nr")
    seed = 0
    ce = synth.encoder_params(shape, seed); tk = synth.task_params(shape, seed)
    toks = synth.item_tokens(seed, shape.n_items, shape.l_t, shape.vocab)
    ids, lab = synth.batch(shape, seed, step=0)
    P, d, B, L = ids.size, shape.d, shape.B, shape.L
    assert (B, L, shape.n_items, shape.l_t) == (64, 55, 100_000, 32)
    g = gh.make_ctx(shape, ce, tk, toks)
    rng = np.random.default_rng(7)
    ids_d = torch.from_numpy(ids.ravel().copy()).to(DEV); lab_d = torch.from_numpy(lab.ravel().copy()).to(DEV)
    cap = min(P, shape.n_items)
    unique = torch.zeros(cap, dtype=torch.int32, device=DEV); inverse = torch.zeros(P, dtype=torch.int32, device=DEV)
    perm = torch.zeros(P, dtype=torch.int32, device=DEV); seg = torch.zeros(cap + 1, dtype=torch.int32, device=DEV)
    nu = torch.zeros(1, dtype=torch.int32, device=DEV)
    g.dedup(ids_d, shape.n_items, unique, inverse, perm, seg, nu)
    g.sync()
    U = int(nu.item())
    w_unique, w_inverse, w_perm, w_seg = orc.unique_inverse(ids)
    assert U == len(w_unique) and 1000 < U < 2000
    assert np.array_equal(unique[:U].cpu().numpy(), w_unique) and np.array_equal(inverse.cpu().numpy(), w_inverse)
    assert np.array_equal(perm.cpu().numpy(), w_perm) and np.array_equal(seg[:U + 1].cpu().numpy(), w_seg)
    H = torch.zeros(U, d, device=DEV)
    g.encode_unique(None, unique, U, H, save_activations=True)
    g.sync()
    counts = np.diff(w_seg)
    sample_u = sorted({0, U - 1, int(np.argmax(counts))} | {int(x) for x in rng.integers(0, U, 3)})
    want_H = orc.encode_all(shape, ce, toks, [w_unique[u] for u in sample_u])
    H_np = H.cpu().numpy()
    for k, u in enumerate(sample_u):
        assert _row_err(H_np[u], want_H[k]) <= TOL, (u, _row_err(H_np[u], want_H[k]))
    E = torch.zeros(P, d, device=DEV)
    g.gather(H, inverse, E)
    g.sync()
    assert torch.equal(E, H[inverse.long()])
    dE = torch.zeros(P, d, device=DEV); loss = torch.zeros(1, device=DEV)
    g.task(E, lab_d, B, dE, loss)
    g.sync()
    b = int(rng.integers(0, B))
    user_items, user_inv = np.unique(ids[b], return_inverse=True)
    E_b = orc.encode_all(shape, ce, toks, user_items)[user_inv]
    E_t = torch.tensor(E_b[None], dtype=torch.float64, requires_grad=True)
    loss_b = orc.task_loss(orc.as_torch(tk), E_t, lab[b:b + 1], shape.replace(B=1))
    loss_b.backward()
    got = dE.view(B, L, d)[b].cpu().numpy()
    assert _row_err(got, E_t.grad[0].numpy() / B) <= TOL, _row_err(got, E_t.grad[0].numpy() / B)
    # the batch loss: the oracle's task module in float64 on the encodings the device holds (already checked above)
    with torch.no_grad():
        want_loss = float(orc.task_loss(orc.as_torch(tk, requires_grad=False), E.view(B, L, d).double().cpu(), lab, shape))
    assert abs(float(loss.item()) - want_loss) <= TOL * abs(want_loss), (float(loss.item()), want_loss)
    G = torch.zeros(U, d, device=DEV)
    g.accumulate(dE, perm, seg, U, G)
    g.sync()
    dE64 = dE.double()
    assert float((G.double().sum(0) - dE64.sum(0)).abs().max()) <= 1e-5 * float(dE64.abs().sum(0).max())
    for u in sample_u:
        rows = torch.from_numpy(w_perm[w_seg[u]:w_seg[u + 1]].astype(np.int64)).to(DEV)
        bound = float(dE64[rows].abs().sum(0).max()) * len(rows) * 2.0 ** -24 + 1e-12
        assert float((G[u].double() - dE64[rows].sum(0)).abs().max()) <= bound, u
    picks = sorted({int(x) for x in rng.integers(0, U, 3)})
    items = [int(w_unique[u]) for u in picks]
    g_rows = rng.standard_normal((len(picks), d))
    G_sparse = torch.zeros(U, d, device=DEV)
    G_sparse[torch.tensor(picks, device=DEV)] = torch.from_numpy(g_rows).float().to(DEV)
    g.zero_grads(binding.GRAM_MODULE_CE)
    g.encoder_backward(G_sparse, unique, U)
    gce, _ = gh.gpu_grads(g, shape)
    h = orc.encode_all(shape, ce, toks, items)
    _, want_g = orc.pseudo_loss_grad(shape, ce, toks, items, h - g_rows)
    worst, name = gh.worst_rel_err(gce, want_g)
    print("news workload, encoder backward of 3 sampled items at full size: worst tensor", name, worst)
    assert worst <= TOL, (name, worst)
    # and the whole step reports the same counts
    rep = g.step(torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV), B)
    assert rep.n_unique == U and rep.n_positions == P and abs(rep.loss - float(loss.item())) <= 1e-5 * abs(rep.loss)
    g.close()
