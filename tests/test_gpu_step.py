"""Gradient parity of the whole step and of its stages with the oracle (end-to-end training), through the C ABI.

Tolerances: max |g_gpu - g_oracle| / max |g_oracle| per parameter tensor, 1e-3 for fp32 contexts and 2e-2 for bf16.
"""
import numpy as np
import pytest
import torch

from oracle import gram_oracle as orc
from paper_2204_04179_b200 import binding, synth
from tests import gram_helpers as gh

pytestmark = pytest.mark.gpu
DEV = gh.DEV
TOL = {"f32": 1e-3, "bf16": 2e-2}


def small(**kw):
    base = dict(name="s", n_items=40, l_t=8, vocab=50, d=32, n_heads=2, d_ff=64, n_layers=2, pooling="mean",
                task="kt", task_layers=1, task_heads=2, task_d_ff=64, task_attn_only=True, B=4, L=12, zipf_s=1.1)
    base.update(kw)
    return synth.GramShape(**base)


CASES = {
    "tiny_cfg": synth.config("tiny"),
    "cls_full_task": small(pooling="cls", task_attn_only=False, task_layers=2),
    "odd_sizes": small(n_items=23, l_t=5, d=24, n_heads=3, d_ff=40, B=3, L=7, task_heads=2),
    "nr": small(task="nr", task_layers=0, n_cand=3, L=9, d_a=16, pooling="cls"),
    # the news task with one self-attention layer over the clicked items (Appendix D), attention only and with the whole layer
    "nr_mhsa": small(task="nr", task_layers=1, task_heads=2, task_attn_only=True, n_cand=3, L=9, d_a=16, pooling="cls"),
    "nr_mhsa_full": small(task="nr", task_layers=1, task_heads=2, task_attn_only=False, n_cand=3, L=9, d_a=16, pooling="cls"),
    "bf16_nr_mhsa": small(dtype="bf16", task="nr", task_layers=1, task_heads=2, task_attn_only=True, n_cand=3, L=9, d_a=16,
                          pooling="cls", d=64, d_ff=128),
    "bf16_nr_mhsa_dh64": small(dtype="bf16", task="nr", task_layers=1, task_heads=2, task_attn_only=False, task_d_ff=128, n_cand=4,
                               L=24, B=5, d_a=16, pooling="cls", d=128, d_ff=128, l_t=16),
    "tiny_bf16": synth.config("tiny").replace(dtype="bf16"),
    "bf16_cls_full": small(dtype="bf16", pooling="cls", task_attn_only=False, d=64, d_ff=128, task_d_ff=128),
    "bf16_nr": small(dtype="bf16", task="nr", task_layers=0, n_cand=3, L=9, d_a=16, pooling="cls", d=64, d_ff=128),
    # sequences that span several 16-row attention tiles with a ragged tail (70 tokens, 100 positions)
    "long_seq": small(l_t=70, L=100, B=2, d=64, n_heads=1, d_ff=64, task_d_ff=64, n_items=30, task_attn_only=False),
    "bf16_long_seq": small(dtype="bf16", l_t=70, L=100, B=2, d=64, n_heads=1, d_ff=64, task_d_ff=64, n_items=30,
                           task_attn_only=False),
    "bf16_seq128": small(dtype="bf16", l_t=128, L=128, B=1, d=64, n_heads=2, d_ff=64, task_d_ff=64, n_items=12, pooling="cls"),
    # heads of width 64: the tcgen05 attention kernels.  Sequences packed into 128-row tiles in slots of 16 (whole tiles in
    # one copy) and 32 rows with an empty slot at the end (3 histories), slots wider than the sequences (24 in 32, 20 in 32),
    # two sequences per tile, and one sequence per tile with a ragged tail (100 of 128 rows, causal)
    "bf16_dh64_s16": small(dtype="bf16", d=128, n_heads=2, task_heads=2, d_ff=128, task_d_ff=128, l_t=16, L=32, B=3, n_items=40,
                           pooling="cls", task_attn_only=False),
    "bf16_dh64_s24": small(dtype="bf16", d=128, n_heads=2, task_heads=2, d_ff=128, task_d_ff=128, l_t=24, L=20, B=5, n_items=40,
                           pooling="mean"),
    "bf16_dh64_s64": small(dtype="bf16", d=128, n_heads=2, task_heads=2, d_ff=128, task_d_ff=128, l_t=64, L=64, B=3, n_items=30,
                           pooling="cls", task_attn_only=False),
    "bf16_dh64_s128": small(dtype="bf16", d=64, n_heads=1, task_heads=1, d_ff=64, task_d_ff=64, l_t=128, L=100, B=2, n_items=14,
                            pooling="mean"),
    # texts longer than one 128-row tile (Table 3 lists mean lengths of 147 and 271 tokens, Appendix D truncates at 512):
    # several query tiles per sequence, a running maximum and sum over the key tiles, a ragged last tile; and histories
    # of 200 positions through the causal task module
    "bf16_dh64_t147": small(dtype="bf16", d=64, n_heads=1, task_heads=1, d_ff=64, task_d_ff=64, l_t=147, L=6, B=2, n_items=8,
                            n_layers=1, pooling="mean"),
    "bf16_dh64_t271": small(dtype="bf16", d=128, n_heads=2, task_heads=2, d_ff=128, task_d_ff=128, l_t=271, L=6, B=2, n_items=8,
                            n_layers=1, pooling="cls"),
    "bf16_dh64_t512": small(dtype="bf16", d=64, n_heads=1, task_heads=1, d_ff=64, task_d_ff=64, l_t=512, L=12, B=3, n_items=8,
                            n_layers=1, pooling="mean"),
    "bf16_dh64_L200": small(dtype="bf16", d=64, n_heads=1, task_heads=1, d_ff=64, task_d_ff=64, l_t=8, L=200, B=2, n_items=30,
                            n_layers=1, pooling="mean", task_attn_only=False),
}


@pytest.mark.parametrize("name", list(CASES))
def test_single_step_matches_e2e(name):
    shape = CASES[name]
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=3)
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab)
    tol = TOL[shape.dtype]
    assert rep.n_unique == len(np.unique(ids)) and rep.encoder_pass == 1
    assert rep.boost_ratio == pytest.approx(ids.size / rep.n_unique, rel=1e-6)
    assert abs(rep.loss - want["loss"]) <= tol * abs(want["loss"])
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    print(name, "worst CE", e1, n1, "worst task", e2, n2)
    assert e1 <= tol, (n1, e1)
    assert e2 <= tol, (n2, e2)


def test_host_entry_point_and_determinism():
    shape = CASES["tiny_cfg"]
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=5)
    r1, a1, b1 = gh.gpu_single_step(shape, ce, tk, toks, ids, lab)
    r2, a2, b2 = gh.gpu_single_step(shape, ce, tk, toks, ids, lab, host=True)
    assert r1.loss == r2.loss
    for k in a1:
        assert np.array_equal(a1[k], a2[k]), k        # bit-identical across runs and entry points
    for k in b1:
        assert np.array_equal(b1[k], b2[k]), k


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_micro_batched_encoder_pass_gives_the_same_gradients(dtype):
    shape = small(dtype=dtype, d=64, d_ff=128, task_d_ff=128, n_items=60, B=6, L=16)
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=7)
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    U = len(np.unique(ids))
    assert U > 16
    rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab, ce_micro_batch=7)     # several ragged passes
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    assert e1 <= TOL[dtype] and e2 <= TOL[dtype], (e1, n1, e2, n2)


def test_stages_one_by_one():
    """gram_dedup -> gram_encode_unique -> gram_gather -> gram_task -> gram_accumulate -> gram_encoder_backward."""
    shape = small(pooling="cls", task_attn_only=False)
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=9)
    ref = orc.gram_single_step(shape, ce, tk, toks, ids, lab)
    g = gh.make_ctx(shape, ce, tk, toks)
    P, d = ids.size, shape.d
    ids_d = torch.from_numpy(ids.ravel().copy()).to(DEV)
    lab_d = torch.from_numpy(lab.ravel().copy()).to(DEV)
    cap = min(P, shape.n_items)
    unique = torch.zeros(cap, dtype=torch.int32, device=DEV); inverse = torch.zeros(P, dtype=torch.int32, device=DEV)
    perm = torch.zeros(P, dtype=torch.int32, device=DEV); seg = torch.zeros(cap + 1, dtype=torch.int32, device=DEV)
    nu = torch.zeros(1, dtype=torch.int32, device=DEV)
    g.dedup(ids_d, shape.n_items, unique, inverse, perm, seg, nu)
    U = int(nu.item())
    assert np.array_equal(unique[:U].cpu().numpy(), ref["unique"]) and np.array_equal(inverse.cpu().numpy(), ref["inverse"])
    H = torch.zeros(U, d, device=DEV)
    g.encode_unique(None, unique, U, H, save_activations=True)
    g.sync()
    assert gh.rel_err(H.cpu().numpy(), ref["H"]) <= 1e-4
    E = torch.zeros(P, d, device=DEV)
    g.gather(H, inverse, E)
    dE = torch.zeros(P, d, device=DEV); loss = torch.zeros(1, device=DEV)
    g.task(E, lab_d, shape.B, dE, loss)
    g.sync()
    assert abs(float(loss.item()) - ref["loss"]) <= 1e-4 * abs(ref["loss"])
    assert gh.rel_err(dE.cpu().numpy(), ref["dE"]) <= 1e-3
    G = torch.zeros(U, d, device=DEV)
    g.accumulate(dE, perm, seg, U, G)
    g.sync()
    assert gh.rel_err(G.cpu().numpy(), ref["G"]) <= 1e-3
    g.zero_grads(binding.GRAM_MODULE_CE)
    g.encoder_backward(G, unique, U)
    gce, gtk = gh.gpu_grads(g, shape)
    e1, n1 = gh.worst_rel_err(gce, ref["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, ref["grad_task"])
    assert e1 <= 1e-3 and e2 <= 1e-3, (e1, n1, e2, n2)
    # Fig. 1's count: the encoder backward ran over U rows, not P
    assert U < P
    g.close()


def test_fig1_counts_through_the_step():
    shape = small(n_items=10, B=3, L=4)
    ce, tk, toks, _, lab = gh.make_inputs(shape, seed=1)
    ids = np.array([[3, 7, 3, 9], [7, 7, 1, 3], [9, 4, 1, 3]], np.int32)      # 12 interactions, 5 items
    rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab)
    assert rep.n_positions == 12 and rep.n_unique == 5 and rep.n_encoded == 5
    assert rep.boost_ratio == pytest.approx(2.4)
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    assert gh.worst_rel_err(gce, want["grad_ce"])[0] <= 1e-3


def test_step_rejects_bad_input_without_faulting():
    shape = small()
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=2)
    g = gh.make_ctx(shape, ce, tk, toks)
    bad = ids.copy(); bad[1, 2] = shape.n_items
    with pytest.raises(binding.GramError) as e:
        g.step(torch.from_numpy(bad).to(DEV), torch.from_numpy(lab).to(DEV), shape.B)
    assert e.value.status == 2
    with pytest.raises(binding.GramError) as e:
        g.step(torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV), shape.B + 1)
    assert e.value.status == 3
    rep = g.step(torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV), shape.B)      # still usable
    assert rep.n_unique == len(np.unique(ids))
    g.close()


@pytest.mark.parametrize("K,opt", [(1, binding.GRAM_OPT_SGD), (3, binding.GRAM_OPT_SGD), (3, binding.GRAM_OPT_ADAM)])
def test_a_rejected_step_changes_no_state(K, opt):
    # a batch with an item ID out of range is refused with GRAM_ERR_ID_RANGE, and nothing that outlives the step has
    # moved: parameters of both modules, the optimiser's state and counts, the Multi-step table, touched bits, cache and
    # the position inside the window are bit-identical to what they were, also with learning rates above zero, in the
    # middle of a window and on its last step
    shape = small(d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=K, pooling="cls")
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=5)
    g = gh.make_ctx(shape, ce, tk, toks, K=K, lr_task=0.05, lr_ce=0.02, optimizer=opt, ce_micro_batch=16)
    if K > 1:
        g.cache_fill()

    def snapshot(c=None):
        c = g if c is None else c
        st = [c.get_params(binding.GRAM_MODULE_CE), c.get_params(binding.GRAM_MODULE_TASK)]
        for mod in (binding.GRAM_MODULE_CE, binding.GRAM_MODULE_TASK):
            m, v, upd = c.optimizer_export(mod)
            st += [np.array([upd])] + ([m, v] if m is not None else [])
        if K > 1:
            table, touched, cache, steps = c.state_export()
            st += [table, touched, cache, np.array([steps])]
        return st

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a, np.int32)).to(DEV)
    n_good = 0
    for step in range(2 * K + 1):
        ids, lab = synth.batch(shape, 5, step=step)
        if K > 1 and step in (1, K - 1 + K):          # mid-window, and on what would be the window's last step
            before = snapshot()
            bad = ids.copy(); bad[2, 3] = shape.n_items + 7
            for host in (False, True):
                with pytest.raises(binding.GramError) as e:
                    if host:
                        g.step_host(np.ascontiguousarray(bad, np.int32), np.ascontiguousarray(lab, np.int32), shape.B)
                    else:
                        g.step(dev(bad), dev(lab), shape.B)
                assert e.value.status == 2
                for a, b in zip(before, snapshot()):
                    assert np.array_equal(a, b)
        if K == 1 and step == 1:
            before = snapshot()
            bad = ids.copy(); bad[0, 0] = -1
            with pytest.raises(binding.GramError) as e:
                g.step(dev(bad), dev(lab), shape.B)
            assert e.value.status == 2
            for a, b in zip(before, snapshot()):
                assert np.array_equal(a, b)
        rep = g.step(dev(ids), dev(lab), shape.B)                # the context stays usable and keeps its place
        n_good += 1
        assert rep.n_unique == len(np.unique(ids))
        if K > 1:
            assert rep.encoder_pass == int(n_good % K == 0)
    # the rejected steps left no trace: a second context that never saw them ends in the same state
    g2 = gh.make_ctx(shape, ce, tk, toks, K=K, lr_task=0.05, lr_ce=0.02, optimizer=opt, ce_micro_batch=16)
    if K > 1:
        g2.cache_fill()
    for step in range(2 * K + 1):
        ids, lab = synth.batch(shape, 5, step=step)
        g2.step(dev(ids), dev(lab), shape.B)
    for x, y in zip(snapshot(g), snapshot(g2)):
        assert np.array_equal(x, y)
    g.close(); g2.close()


@pytest.mark.parametrize("dtype,K", [("f32", 1), ("f32", 3), ("bf16", 2)])
def test_multistep_window_matches_algorithm(dtype, K):
    shape = small(dtype=dtype, d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=max(K, 2), pooling="cls")
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=21)
    lr = 0.05
    batches = [synth.batch(shape, 21, step=k) for k in range(K)]
    cfg_K = K if K > 1 else 2
    g = gh.make_ctx(shape, ce, tk, toks, K=cfg_K, lr_task=lr, ce_micro_batch=16)
    g.cache_fill()
    _, _, cache0 = g.get_window(want_table=False, want_touched=False)
    enc = orc.encode_all(shape, ce, toks, range(shape.n_items))
    assert gh.rel_err(cache0, enc) <= (1e-4 if dtype == "f32" else 2e-2)
    # the oracle starts from the cache values the device really holds, so that bf16 rounding of the cache
    # is an input, not an error
    want = orc.multistep_window(shape, ce, tk, toks, batches, cache0.astype(np.float64), lr_task=lr,
                                cache_bf16=(dtype == "bf16"))
    reps = [g.step(torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV), shape.B) for ids, lab in batches]
    tol = TOL[dtype]
    for k in range(len(reps)):
        assert abs(reps[k].loss - want["losses"][k]) <= tol * abs(want["losses"][k])
    if K >= 2:
        assert [r.encoder_pass for r in reps] == [0] * (K - 1) + [1]
        assert reps[-1].n_touched == len(want["items"]) == reps[-1].n_encoded
        gce, gtk = gh.gpu_grads(g, shape)
        e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
        e2, n2 = gh.worst_rel_err(gtk, want["grad_task_last"])
        assert e1 <= tol and e2 <= tol, (e1, n1, e2, n2)
        tp = synth.unflatten(g.get_params(binding.GRAM_MODULE_TASK), synth.task_param_spec(shape))
        for name in tp:
            assert gh.rel_err(tp[name], want["task_params"][name]) <= tol, name
        table, touched, cache = g.get_window()
        assert np.all(table == 0) and np.all(touched == 0)                 # the window was cleared
        assert gh.rel_err(cache, want["cache"]) <= tol
    else:
        # K = 1 of a K = 2 context: first step only; table and touched set equal the single-step sums
        table, touched, _ = g.get_window(want_cache=False)
        bits = np.unpackbits(touched.view(np.uint8), bitorder="little")[:shape.n_items].astype(bool)
        ids, lab = batches[0]
        assert np.array_equal(np.nonzero(bits)[0], np.unique(ids))
        one = orc.multistep_window(shape, ce, tk, toks, batches[:1], cache0.astype(np.float64), lr_task=lr)
        assert gh.rel_err(table, one["table"]) <= tol
    g.close()


def test_multistep_pseudo_target_two_windows_f32():
    """GRAM_MULTI_PSEUDO_TARGET against Algorithm 1 under the trainable-embedding reading (Section 4.3): two windows of
    K = 3 steps with an encoder update in between, so that the second window's cache is stale and the cotangent of
    Eq. 9 carries CE(c; theta) - cache besides the accumulated gradients."""
    K = 3
    shape = small(dtype="f32", d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=K, pooling="cls")
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=23)
    lr_t, lr_c = 0.05, 0.02
    batches = [synth.batch(shape, 23, step=k) for k in range(2 * K)]
    g = gh.make_ctx(shape, ce, tk, toks, K=K, lr_task=lr_t, lr_ce=lr_c, ce_micro_batch=16,
                    multistep_variant=binding.GRAM_MULTI_PSEUDO_TARGET)
    g.cache_fill()
    _, _, cache0 = g.get_window(want_table=False, want_touched=False)
    assert gh.rel_err(cache0, orc.encode_all(shape, ce, toks, range(shape.n_items))) <= 1e-4
    cur_ce = {k: np.asarray(v, np.float64) for k, v in ce.items()}
    cur_tk = {k: np.asarray(v, np.float64) for k, v in tk.items()}
    cache = cache0.astype(np.float64)
    plain_losses = orc.multistep_window(shape, ce, tk, toks, batches[:K], cache, lr_task=lr_t)["losses"]
    for w in range(2):
        want = orc.multistep_window_pseudo_target(shape, cur_ce, cur_tk, toks, batches[w * K:(w + 1) * K], cache, lr_task=lr_t)
        reps = [g.step(torch.from_numpy(i).to(DEV), torch.from_numpy(l).to(DEV), shape.B) for i, l in batches[w * K:(w + 1) * K]]
        assert [r.encoder_pass for r in reps] == [0] * (K - 1) + [1]
        assert reps[-1].n_touched == len(want["items"]) == reps[-1].n_encoded
        for k in range(K):
            assert abs(reps[k].loss - want["losses"][k]) <= 1e-4 * abs(want["losses"][k]), (w, k)
        if w == 0:      # the later steps really read the modified embeddings, not the cached ones
            assert abs(reps[1].loss - plain_losses[1]) > 10 * abs(reps[1].loss - want["losses"][1])
        gce, gtk = gh.gpu_grads(g, shape)
        e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
        e2, n2 = gh.worst_rel_err(gtk, want["grad_task_last"])
        print("window", w, "worst CE", e1, n1, "worst task", e2, n2)
        assert e1 <= 1e-3 and e2 <= 1e-3, (w, e1, n1, e2, n2)
        _, _, cache_gpu = g.get_window(want_table=False, want_touched=False)
        assert gh.rel_err(cache_gpu, want["cache"]) <= 1e-4
        cur_ce = {k: cur_ce[k] - lr_c * want["grad_ce"][k] for k in cur_ce}
        cur_tk = want["task_params"]
        cache = want["cache"]
    g.close()


def test_multistep_pseudo_target_first_window_bf16():
    # a bf16 context keeps the cache in fp32 for this variant; in the first window after a cache fill the staleness
    # term is zero on both sides, so the comparison is the usual one for bf16 encoders
    K = 2
    shape = small(dtype="bf16", d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=K, pooling="cls")
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=25)
    batches = [synth.batch(shape, 25, step=k) for k in range(K)]
    g = gh.make_ctx(shape, ce, tk, toks, K=K, lr_task=0.05, ce_micro_batch=16,
                    multistep_variant=binding.GRAM_MULTI_PSEUDO_TARGET)
    g.cache_fill()
    cache = orc.encode_all(shape, ce, toks, range(shape.n_items))
    want = orc.multistep_window_pseudo_target(shape, ce, tk, toks, batches, cache, lr_task=0.05)
    reps = [g.step(torch.from_numpy(i).to(DEV), torch.from_numpy(l).to(DEV), shape.B) for i, l in batches]
    for k in range(K):
        assert abs(reps[k].loss - want["losses"][k]) <= 2e-2 * abs(want["losses"][k])
    gce, gtk = gh.gpu_grads(g, shape)
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task_last"])
    print("bf16 pseudo-target worst CE", e1, n1, "worst task", e2, n2)
    assert e1 <= 2e-2 and e2 <= 2e-2, (e1, n1, e2, n2)
    g.close()


VARLEN = {
    "f32_mean": small(l_t=9, pooling="mean"),
    "f32_cls_full_task": small(l_t=9, pooling="cls", task_attn_only=False, task_layers=2),
    "f32_nr": small(task="nr", task_layers=0, n_cand=3, L=9, d_a=16, pooling="cls", l_t=7),
    # tensor-core attention: texts of 1..40 tokens in a 64-row tile, and 1..70 in a 96-row tile
    "bf16_mean_40": small(dtype="bf16", l_t=40, d=64, n_heads=2, d_ff=128, task_d_ff=128, n_items=30, pooling="mean"),
    "bf16_cls_70": small(dtype="bf16", l_t=70, d=64, n_heads=1, d_ff=64, task_d_ff=64, n_items=30, pooling="cls", B=2),
    # heads of width 64 (tcgen05 attention): packed rows, one launch per length group, slots of 32, 64 and 128 rows
    "bf16_dh64_var40": small(dtype="bf16", l_t=40, d=128, n_heads=2, task_heads=2, d_ff=128, task_d_ff=128, n_items=30, pooling="mean"),
    "bf16_dh64_var128": small(dtype="bf16", l_t=128, d=64, n_heads=1, task_heads=1, d_ff=64, task_d_ff=64, n_items=24, pooling="cls", B=3),
    # texts of 1..300 tokens: the three short groups, and a last group that mixes 97..128-row texts with multi-tile ones
    "bf16_dh64_var300": small(dtype="bf16", l_t=300, d=64, n_heads=1, task_heads=1, d_ff=64, task_d_ff=64, n_items=16, n_layers=1,
                              pooling="mean", B=2, L=8),
    # several ragged encoder passes of 7 items, each with its own packed layout
    "f32_cls_micro_batches": small(l_t=9, pooling="cls", n_items=60, B=6, L=16),
}
VARLEN_OVER = {"f32_cls_micro_batches": dict(ce_micro_batch=7)}


@pytest.mark.parametrize("name", list(VARLEN))
def test_texts_of_different_lengths(name):
    """gram_set_item_lengths: padded storage on the device, plain shorter sequences in the oracle."""
    shape = VARLEN[name]
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=31)
    lengths = synth.item_lengths(31, shape.n_items, shape.l_t)
    assert lengths.min() == 1 and lengths.max() == shape.l_t
    want = orc.e2e_step(shape, ce, tk, synth.ragged(toks, lengths), ids, lab)
    junk = toks.copy()
    for i, n in enumerate(lengths):                       # whatever sits in the padding slots must not matter
        junk[i, n:] = (junk[i, n:] * 7 + 3) % shape.vocab
    tol = TOL[shape.dtype]
    results = []
    over = VARLEN_OVER.get(name, {})
    for tokens in (toks, junk):
        g = gh.make_ctx(shape, ce, tk, tokens, **over)
        g.set_item_lengths(lengths)
        rep = g.step(torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV), shape.B)
        gce, gtk = gh.gpu_grads(g, shape)
        g.close()
        assert abs(rep.loss - want["loss"]) <= tol * abs(want["loss"])
        e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
        e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
        print(name, "worst CE", e1, n1, "worst task", e2, n2)
        assert e1 <= tol and e2 <= tol, (e1, n1, e2, n2)
        results.append((rep.loss, gce))
    assert results[0][0] == results[1][0]
    for k in results[0][1]:
        if k != "tok_emb":                                # the padding tokens' embedding rows receive exact zeros either way
            assert np.array_equal(results[0][1][k], results[1][1][k]), k
    # back to fixed-length texts
    g = gh.make_ctx(shape, ce, tk, toks)
    g.set_item_lengths(lengths)
    g.set_item_lengths(None)
    rep = g.step(torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV), shape.B)
    full = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    assert abs(rep.loss - full["loss"]) <= tol * abs(full["loss"])
    with pytest.raises(binding.GramError):
        bad = lengths.copy(); bad[3] = shape.l_t + 1
        g.set_item_lengths(bad)
    g.close()


@pytest.mark.parametrize("dtype,variant", [("f32", binding.GRAM_MULTI_TABLE), ("bf16", binding.GRAM_MULTI_TABLE),
                                           ("f32", binding.GRAM_MULTI_PSEUDO_TARGET)])
def test_checkpoint_and_resume_continue_bit_for_bit(dtype, variant):
    """Parameters, optimiser state and the open Multi-step window exported after two steps of a window of three and
    imported into a fresh context: the third step (with its encoder pass and both Adam updates) gives identical
    results in both contexts."""
    K = 3
    shape = small(dtype=dtype, d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=K, pooling="cls")
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=41)
    batches = [synth.batch(shape, 41, step=k) for k in range(K + 1)]
    over = dict(K=K, lr_task=1e-2, lr_ce=1e-2, ce_micro_batch=16, multistep_variant=variant, optimizer=binding.GRAM_OPT_ADAM,
                noam_warmup=4)
    a = gh.make_ctx(shape, ce, tk, toks, **over)
    a.cache_fill()
    to_dev = lambda x: torch.from_numpy(x).to(DEV)
    for k in range(4):                     # one whole window (so that the optimiser state is not trivial), then one step
        a.step(to_dev(batches[k % (K + 1)][0]), to_dev(batches[k % (K + 1)][1]), shape.B)
    table, touched, cache, steps = a.state_export()
    assert steps == 1 and touched.any() and np.abs(table).max() > 0
    b = gh.make_ctx(shape, ce, tk, toks, **over)
    for mod in (binding.GRAM_MODULE_CE, binding.GRAM_MODULE_TASK):
        b.set_params(mod, a.get_params(mod))
        m_, v_, upd = a.optimizer_export(mod)
        assert upd == (1 if mod == binding.GRAM_MODULE_CE else 4) and np.abs(m_).max() > 0
        b.optimizer_import(mod, m_, v_, upd)
    b.state_import(table, touched, cache, steps)
    for k in (1, 2):
        ra = a.step(to_dev(batches[k][0]), to_dev(batches[k][1]), shape.B)
        rb = b.step(to_dev(batches[k][0]), to_dev(batches[k][1]), shape.B)
        assert ra.loss == rb.loss and ra.n_touched == rb.n_touched and ra.encoder_pass == rb.encoder_pass
    assert rb.encoder_pass == 1
    for mod in (binding.GRAM_MODULE_CE, binding.GRAM_MODULE_TASK):
        assert np.array_equal(a.get_params(mod), b.get_params(mod))
        assert np.array_equal(a.get_grads(mod), b.get_grads(mod))
    ta, ua, ca, sa = a.state_export(); tb, ub, cb, sb = b.state_export()
    assert sa == sb == 0 and np.array_equal(ca, cb) and np.array_equal(ta, tb) and np.array_equal(ua, ub)
    with pytest.raises(binding.GramError):
        b.state_import(None, None, None, K)
    a.close(); b.close()


@pytest.mark.parametrize("name", ["tiny_cfg", "cls_full_task", "bf16_cls_full"])
def test_histories_that_end_in_padding(name):
    """Label -1 marks padding at the end of a history: no prediction there, zero gradient rows, loss averaged over the
    real predictions; the oracle evaluates the shorter histories themselves."""
    shape = CASES[name]
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=33)
    lab = lab.copy()
    rng = np.random.default_rng(0)
    lens = rng.integers(1, shape.L + 1, shape.B)
    lens[0] = shape.L
    for b, n in enumerate(lens):
        lab[b, n:] = -1
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab)
    tol = TOL[shape.dtype]
    assert abs(rep.loss - want["loss"]) <= tol * abs(want["loss"])
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    print(name, "worst CE", e1, n1, "worst task", e2, n2)
    assert e1 <= tol and e2 <= tol, (e1, n1, e2, n2)
    # the gradient rows of padded positions are exactly zero
    g = gh.make_ctx(shape, ce, tk, toks)
    P, d = ids.size, shape.d
    E = torch.randn(P, d, device=DEV); dE = torch.full((P, d), float("nan"), device=DEV); loss = torch.zeros(1, device=DEV)
    g.task(E, torch.from_numpy(lab.ravel().copy()).to(DEV), shape.B, dE, loss)
    g.sync()
    pad = torch.from_numpy((lab.ravel() < 0)).to(DEV)
    assert pad.any() and torch.count_nonzero(dE[pad]) == 0 and torch.isfinite(dE).all()
    g.close()


def test_multistep_window_with_texts_of_different_lengths():
    # the cache fill (items by range) and the encoder pass over the touched items (items by list) both run on packed rows
    K = 2
    shape = small(dtype="f32", d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=K, pooling="cls", l_t=9)
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=27)
    lengths = synth.item_lengths(27, shape.n_items, shape.l_t)
    ragged = synth.ragged(toks, lengths)
    batches = [synth.batch(shape, 27, step=k) for k in range(K)]
    g = gh.make_ctx(shape, ce, tk, toks, K=K, lr_task=0.05, ce_micro_batch=16)
    g.set_item_lengths(lengths)
    g.cache_fill()
    _, _, cache0 = g.get_window(want_table=False, want_touched=False)
    assert gh.rel_err(cache0, orc.encode_all(shape, ce, ragged, range(shape.n_items))) <= 1e-4
    want = orc.multistep_window(shape, ce, tk, ragged, batches, cache0.astype(np.float64), lr_task=0.05)
    reps = [g.step(torch.from_numpy(i).to(DEV), torch.from_numpy(l).to(DEV), shape.B) for i, l in batches]
    assert reps[-1].encoder_pass == 1 and reps[-1].n_encoded == len(want["items"])
    gce, gtk = gh.gpu_grads(g, shape)
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    assert e1 <= 1e-3, (e1, n1)
    _, _, cache = g.get_window(want_table=False, want_touched=False)
    assert gh.rel_err(cache, want["cache"]) <= 1e-4
    g.close()


def test_multistep_cache_refresh_after_the_encoder_update():
    """refresh_after_update: after a window's encoder step the touched items are encoded again with the new parameters,
    so the next window reads fresh encodings (two windows against the oracle; without the flag the cache differs)."""
    K = 2
    shape = small(dtype="f32", d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=K, pooling="cls")
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=43)
    lr_t, lr_c = 0.05, 0.05
    batches = [synth.batch(shape, 43, step=k) for k in range(2 * K)]
    g = gh.make_ctx(shape, ce, tk, toks, K=K, lr_task=lr_t, lr_ce=lr_c, ce_micro_batch=16, refresh_after_update=1)
    g.cache_fill()
    _, _, cache0 = g.get_window(want_table=False, want_touched=False)
    cur_ce, cur_tk, cache = ce, tk, cache0.astype(np.float64)
    for w in range(2):
        want = orc.multistep_window(shape, cur_ce, cur_tk, toks, batches[w * K:(w + 1) * K], cache, lr_task=lr_t, lr_ce=lr_c,
                                    refresh_after_update=True)
        reps = [g.step(torch.from_numpy(i).to(DEV), torch.from_numpy(l).to(DEV), shape.B) for i, l in batches[w * K:(w + 1) * K]]
        for k in range(K):
            assert abs(reps[k].loss - want["losses"][k]) <= 1e-4 * abs(want["losses"][k]), (w, k)
        gce, _ = gh.gpu_grads(g, shape)
        e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
        assert e1 <= 1e-3, (w, e1, n1)
        _, _, cache_gpu = g.get_window(want_table=False, want_touched=False)
        assert gh.rel_err(cache_gpu, want["cache"]) <= 1e-4
        if w == 0:
            stale = orc.multistep_window(shape, cur_ce, cur_tk, toks, batches[:K], cache, lr_task=lr_t, lr_ce=lr_c)
            assert gh.rel_err(cache_gpu, stale["cache"]) > 1e-3
        cur_ce, cur_tk, cache = want["ce_params"], want["task_params"], want["cache"]
    g.close()


ADDITIVE = {
    "f32_kt": small(pooling="additive", d_a=16),
    "f32_nr_odd": small(task="nr", task_layers=0, n_cand=3, L=9, d_a=12, pooling="additive", l_t=7, d=24, n_heads=3, d_ff=40),
    "bf16_kt": small(dtype="bf16", pooling="additive", d_a=16, d=64, d_ff=128, task_d_ff=128, l_t=24, n_items=30),
}


@pytest.mark.parametrize("name", list(ADDITIVE))
@pytest.mark.parametrize("var_len", [False, True])
def test_additive_attention_pooling(name, var_len):
    """GRAM_POOL_ADDITIVE against the oracle, with texts of one length and of different lengths (packed rows)."""
    shape = ADDITIVE[name]
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=37)
    assert "pool_wa" in ce and ce["pool_wa"].shape == (shape.d_a, shape.d)
    lengths = synth.item_lengths(37, shape.n_items, shape.l_t) if var_len else None
    want = orc.e2e_step(shape, ce, tk, synth.ragged(toks, lengths) if var_len else toks, ids, lab)
    g = gh.make_ctx(shape, ce, tk, toks, ce_micro_batch=11)
    if var_len:
        g.set_item_lengths(lengths)
    rep = g.step(torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV), shape.B)
    gce, gtk = gh.gpu_grads(g, shape)
    g.close()
    tol = TOL[shape.dtype]
    assert abs(rep.loss - want["loss"]) <= tol * abs(want["loss"])
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    print(name, var_len, "worst CE", e1, n1, "worst task", e2, n2)
    assert e1 <= tol and e2 <= tol, (e1, n1, e2, n2)
    assert np.abs(gce["pool_qa"]).max() > 0 and np.abs(gce["pool_wa"]).max() > 0


@pytest.mark.parametrize("name", ["nr", "bf16_nr", "nr_mhsa", "nr_mhsa_full", "bf16_nr_mhsa"])
def test_click_histories_with_empty_slots(name):
    """NR: history slots with label -1 hold no click: they take no part in the user vector and get zero gradient rows."""
    shape = CASES[name]
    ce, tk, toks, ids, lab = gh.make_inputs(shape, seed=39)
    lab = np.zeros_like(lab)
    n_hist = shape.L - shape.n_cand
    rng = np.random.default_rng(1)
    for b in range(shape.B):
        empty = rng.choice(n_hist, size=rng.integers(0, n_hist), replace=False)     # at least one click stays
        lab[b, empty] = -1
    assert (lab < 0).any()
    want = orc.e2e_step(shape, ce, tk, toks, ids, lab)
    rep, gce, gtk = gh.gpu_single_step(shape, ce, tk, toks, ids, lab)
    tol = TOL[shape.dtype]
    assert abs(rep.loss - want["loss"]) <= tol * abs(want["loss"])
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task"])
    print(name, "worst CE", e1, n1, "worst task", e2, n2)
    assert e1 <= tol and e2 <= tol, (e1, n1, e2, n2)
    full = orc.e2e_step(shape, ce, tk, toks, ids, np.zeros_like(lab))
    assert abs(full["loss"] - want["loss"]) > 1e-6                                  # the mask matters


def test_tcgen05_attention_on_short_sequences_too():
    """Sequences of up to 128 rows take the warp-level attention kernels by default (they are the faster ones there); the
    tcgen05 kernels serve them as well when GRAM_ATTN_TC=1.  The choice is read once per process, so the cases with heads of
    width 64 are run again in a child process with the switch set: slots of 8 to 128 rows, packed rows, causal tiles."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, GRAM_ATTN_TC="1")
    sel = "bf16_dh64_s16 or bf16_dh64_s24 or bf16_dh64_s64 or bf16_dh64_s128 or bf16_dh64_var40 or bf16_dh64_var128 or bf16_long_seq"
    out = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_step.py"), "-m", "gpu", "-q", "-x",
                          "-k", f"({sel}) and not tcgen05_attention_on_short"], cwd=root, env=env, capture_output=True, text=True,
                         timeout=1200)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-1000:]
    assert " passed" in out.stdout and "failed" not in out.stdout


@pytest.mark.parametrize("K", [1, 2])
def test_deferred_update_and_device_gradient_buffers(K):
    """defer_update: gram_step leaves the gradients in place and applies nothing; the device gradient buffers seen through
    gram_grads_device are the ones gram_get_grads copies; gram_optimizer_step then applies the configured update, and
    the result equals a context that updates inside the step (what a data-parallel trainer relies on between the two)."""
    from paper_2204_04179_b200 import dist as gdist
    shape = small(d=64, d_ff=128, task_d_ff=128, n_items=50, B=4, L=10, K=K, pooling="cls")
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=8)
    kw = dict(K=K, lr_task=0.05, lr_ce=0.02, optimizer=binding.GRAM_OPT_ADAM, ce_micro_batch=16)
    a = gh.make_ctx(shape, ce, tk, toks, **kw)
    b = gh.make_ctx(shape, ce, tk, toks, defer_update=1, **kw)
    if K > 1:
        a.cache_fill(); b.cache_fill()
    for step in range(2 * K):
        ids, lab = synth.batch(shape, 8, step=step)
        i_d, l_d = torch.from_numpy(ids).to(DEV), torch.from_numpy(lab).to(DEV)
        ra = a.step(i_d, l_d, shape.B)
        before = [b.get_params(m) for m in (binding.GRAM_MODULE_CE, binding.GRAM_MODULE_TASK)]
        rb = b.step(i_d, l_d, shape.B)
        assert ra.loss == rb.loss and ra.encoder_pass == rb.encoder_pass
        for m, p0 in zip((binding.GRAM_MODULE_CE, binding.GRAM_MODULE_TASK), before):
            assert np.array_equal(b.get_params(m), p0)                      # nothing applied yet
        tens = gdist.gradient_tensors(b)
        assert np.array_equal(tens[0].cpu().numpy(), b.get_grads(binding.GRAM_MODULE_CE))
        assert np.array_equal(tens[1].cpu().numpy(), b.get_grads(binding.GRAM_MODULE_TASK))
        assert gdist.allreduce_grads(b, gdist.n_predictions(shape, lab), None) == shape.B * shape.L     # one rank: unchanged
        if rb.encoder_pass:
            b.optimizer_step(binding.GRAM_MODULE_CE)
        b.optimizer_step(binding.GRAM_MODULE_TASK)
        for m in (binding.GRAM_MODULE_CE, binding.GRAM_MODULE_TASK):
            assert np.array_equal(a.get_params(m), b.get_params(m))
    a.close(); b.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_multistep_window_of_the_news_task(dtype):
    """Multi-step GRAM with the news task module: the materialised gather from the cache (widened from bf16 in one pass in
    bf16 contexts), K = 2 steps into the table, one encoder pass; losses, gradients, updated task parameters and the refreshed
    cache against Algorithm 1 stepped by the oracle from the cache values the device holds."""
    shape = small(dtype=dtype, task="nr", task_layers=0, n_cand=3, L=9, d_a=16, pooling="cls", d=64, d_ff=128, n_items=50, B=4, K=2)
    ce, tk, toks, _, _ = gh.make_inputs(shape, seed=23)
    lr = 0.05
    batches = []
    for k in range(2):
        ids, lab = synth.batch(shape, 23, step=k)
        batches.append((ids, np.zeros_like(lab)))
    g = gh.make_ctx(shape, ce, tk, toks, K=2, lr_task=lr, ce_micro_batch=16)
    g.cache_fill()
    _, _, cache0 = g.get_window(want_table=False, want_touched=False)
    want = orc.multistep_window(shape, ce, tk, toks, batches, cache0.astype(np.float64), lr_task=lr, cache_bf16=(dtype == "bf16"))
    reps = [g.step(torch.from_numpy(i).to(DEV), torch.from_numpy(l).to(DEV), shape.B) for i, l in batches]
    tol = TOL[dtype]
    for k in range(2):
        assert abs(reps[k].loss - want["losses"][k]) <= tol * abs(want["losses"][k])
    assert [r.encoder_pass for r in reps] == [0, 1] and reps[-1].n_touched == len(want["items"])
    gce, gtk = gh.gpu_grads(g, shape)
    e1, n1 = gh.worst_rel_err(gce, want["grad_ce"])
    e2, n2 = gh.worst_rel_err(gtk, want["grad_task_last"])
    print(dtype, "worst CE", e1, n1, "worst task", e2, n2)
    assert e1 <= tol and e2 <= tol, (e1, n1, e2, n2)
    _, _, cache = g.get_window(want_table=False, want_touched=False)
    assert gh.rel_err(cache, want["cache"]) <= tol
    g.close()
