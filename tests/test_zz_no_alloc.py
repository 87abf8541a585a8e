"""gram_accumulate_static: the segmented sum for callers that cannot allocate device memory.

Some users of this library run where allocation is off limits: inside another application's plug-in
interface, between the steps of a job whose memory was planned up front, or in a loop with a latency
budget.  For them the library keeps the sum's scratch in a fixed array of its own image.  The call must
give the same sums as gram_accumulate (to rounding: it cuts the work into fewer pieces, so the order of
additions differs), must not depend on what an earlier call left in the shared array, and must refuse
rows wider than the array was sized for.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2204_04179_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dedup(g, ids_np, n_items):
    P = ids_np.size
    cap = min(P, n_items)
    ids = torch.from_numpy(ids_np).to(DEV)
    unique = torch.empty(cap, dtype=torch.int32, device=DEV); inverse = torch.empty(P, dtype=torch.int32, device=DEV)
    perm = torch.empty(P, dtype=torch.int32, device=DEV); seg = torch.empty(cap + 1, dtype=torch.int32, device=DEV)
    nu = torch.zeros(1, dtype=torch.int32, device=DEV)
    g.dedup(ids, n_items, unique, inverse, perm, seg, nu)
    g.sync()
    return int(nu.item()), perm, seg


def test_static_scratch_matches_context_scratch_on_two_calls_in_a_row():
    cfg = binding.GramConfig(); cfg.n_items = 20_000; cfg.P_max = 120_000; cfg.d_max = 1024; cfg.d = 1024
    g = binding.Gram(cfg)
    # the second call is smaller and differently shaped, so anything it wrongly reused from the first would show
    for call, (P, N, s, d) in enumerate([(120_000, 20_000, 1.1, 768), (30_001, 50, 1.5, 1024)]):
        ids = synth.zipf_ids(31 + call, N, s, P)
        dE_np = synth.position_gradients(31 + call, P, d)
        U, perm, seg = _dedup(g, ids, N)
        dE = torch.from_numpy(dE_np).to(DEV)
        want = torch.full((U, d), float("nan"), device=DEV)
        g.accumulate(dE, perm, seg, U, want)
        g.sync()
        got = torch.full((U, d), float("nan"), device=DEV)
        binding.accumulate_static(dE, perm, seg, U, got)
        torch.cuda.synchronize()
        counts = np.diff(seg[:U + 1].cpu().numpy()).astype(np.float64)[:, None]
        bound = 2.0 * (counts * 2.0 ** -24) * counts + 1e-6       # both sums carry the fp32 bound of test_gpu_index
        err = np.abs(got.cpu().numpy().astype(np.float64) - want.cpu().numpy().astype(np.float64))
        assert np.isfinite(got.cpu().numpy()).all()
        assert np.all(err <= bound), float(err.max())
        # against float64 as well, and bit-identical when repeated
        exact = np.zeros((U, d)); inv = np.empty(P, np.int64)
        seg_np, perm_np = seg[:U + 1].cpu().numpy(), perm.cpu().numpy()
        inv[perm_np] = np.repeat(np.arange(U), np.diff(seg_np))
        np.add.at(exact, inv, dE_np.astype(np.float64))
        assert np.all(np.abs(got.cpu().numpy() - exact) <= bound)
        again = torch.empty(U, d, device=DEV)
        binding.accumulate_static(dE, perm, seg, U, again)
        torch.cuda.synchronize()
        assert torch.equal(got, again)
    g.close()


def test_static_scratch_rejects_rows_beyond_its_maximum():
    dE = torch.zeros(8, 2048, device=DEV)
    perm = torch.arange(8, dtype=torch.int32, device=DEV)
    seg = torch.arange(9, dtype=torch.int32, device=DEV)
    G = torch.zeros(8, 2048, device=DEV)
    with pytest.raises(binding.GramError) as e:
        binding.accumulate_static(dE, perm, seg, 8, G)
    assert e.value.status == 3 and "1024" in str(e.value)
    # and the call still works afterwards
    dE = torch.ones(8, 16, device=DEV); G = torch.zeros(8, 16, device=DEV)
    binding.accumulate_static(dE, perm, seg, 8, G)
    torch.cuda.synchronize()
    assert torch.equal(G, dE)


def test_static_scratch_narrow_rows_spanning_many_work_units():
    # rows of 64 columns (one 128-column slab per warp) with a heavy-tailed draw: the hottest items span many of the
    # 592 work units, so the second launch really adds partial sums on this path as well
    P, N, s, d = 200_000, 3_000, 1.5, 64
    cfg = binding.GramConfig(); cfg.n_items = N; cfg.P_max = P; cfg.d_max = d; cfg.d = d
    g = binding.Gram(cfg)
    ids = synth.zipf_ids(77, N, s, P)
    dE_np = synth.position_gradients(77, P, d)
    U, perm, seg = _dedup(g, ids, N)
    seg_np, perm_np = seg[:U + 1].cpu().numpy(), perm.cpu().numpy()
    counts = np.diff(seg_np)
    assert counts.max() > 16 * (P // 592)                     # one item alone covers more than sixteen work units
    dE = torch.from_numpy(dE_np).to(DEV)
    got = torch.full((U, d), float("nan"), device=DEV)
    binding.accumulate_static(dE, perm, seg, U, got)
    torch.cuda.synchronize()
    exact = np.zeros((U, d)); inv = np.empty(P, np.int64)
    inv[perm_np] = np.repeat(np.arange(U), counts)
    np.add.at(exact, inv, dE_np.astype(np.float64))
    c = counts.astype(np.float64)[:, None]
    assert np.all(np.abs(got.cpu().numpy() - exact) <= c * 2.0 ** -24 * c + 1e-6)
    # a position outside the batch in d_perm is documented to be read as row 0, without an error
    bad = perm.clone(); j = int(seg_np[3])                    # first occurrence of item 3
    bad[j] = P
    again = torch.full((U, d), float("nan"), device=DEV)
    binding.accumulate_static(dE, bad, seg, U, again)
    torch.cuda.synchronize()
    moved = exact.copy()
    moved[3] += dE_np[0].astype(np.float64) - dE_np[perm_np[j]].astype(np.float64)
    assert np.all(np.abs(again.cpu().numpy() - moved) <= c * 2.0 ** -24 * c + 1e-6)
    g.close()


def test_static_scratch_refuses_what_it_cannot_serve():
    perm = torch.arange(8, dtype=torch.int32, device=DEV); seg = torch.arange(9, dtype=torch.int32, device=DEV)
    with pytest.raises(binding.GramError) as e:               # rows must be whole 16-byte pieces
        binding.accumulate_static(torch.zeros(8, 6, device=DEV), perm, seg, 8, torch.zeros(8, 6, device=DEV))
    assert e.value.status == 4
    base = torch.zeros(8 * 16 + 1, device=DEV)
    with pytest.raises(binding.GramError) as e:               # an output that does not start on a 16-byte boundary
        binding.accumulate_static(torch.zeros(8, 16, device=DEV), perm, seg, 8, base[1:].view(8, 16))
    assert e.value.status == 4
    with pytest.raises(binding.GramError) as e:               # more positions than 32-bit offsets reach (sizes only, no memory touched)
        binding.accumulate_static(torch.zeros(8, 16, device=DEV), perm, seg, 8, torch.zeros(8, 16, device=DEV), P=2 ** 31, d=16)
    assert e.value.status == 3
    with pytest.raises(binding.GramError) as e:
        binding.accumulate_static(torch.zeros(8, 16, device=DEV), perm, seg, 9, torch.zeros(8, 16, device=DEV), P=8, d=16)
    assert e.value.status == 1                                # more items than positions
