"""Pins for the oracle's index work and per-item sums (CPU only)."""
import os

import numpy as np
import pytest

from oracle import gram_oracle as orc
from paper_2204_04179_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_kv(path):
    out = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        out[k] = int(v)
    return out


def test_fig1_worked_count():
    # Fig. 1: 3 users, 12 interactions, 5 unique items -> 5 encoder gradients instead of 12
    g = _read_kv(os.path.join(GOLD, "fig1_counts.txt"))
    ids = np.array([[3, 7, 3, 9], [7, 7, 1, 3], [9, 4, 1, 3]])          # 3 users x 4, 5 distinct items
    assert ids.shape[0] == g["users"] and ids.size == g["interactions"]
    for fn in (orc.unique_inverse_bruteforce, orc.unique_inverse):
        unique, inverse, perm, seg_off = fn(ids)
        assert len(unique) == g["unique_items"] == g["gram_encoder_gradients"]
        assert orc.boost_ratio(ids.size, len(unique)) == pytest.approx(12 / 5)


def test_table3_epoch_level_ratio():
    # Section 4.4: with one-epoch latency R = interactions / items of the dataset (Table 3 values)
    rows = [l.split() for l in open(os.path.join(GOLD, "table3_datasets.txt")) if l[0] != "#"]
    got = {r[0]: orc.boost_ratio(int(r[3]), int(r[2])) for r in rows}
    # TOEIC has by far the largest ratio, which is where the paper reports its largest speed-up
    assert max(got, key=got.get) == "TOEIC"
    assert round(got["TOEIC"], 1) == 10096.9 and round(got["MIND"], 1) == 36.1
    assert round(got["Spanish"], 1) == 60.4 and round(got["French"], 1) == 42.9 and round(got["POJ"], 1) == 345.9


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("P,N", [(1, 5), (17, 3), (64, 200), (200, 40)])
def test_sorted_matches_bruteforce(seed, P, N):
    ids = synth.zipf_ids(seed, N, 1.1, P)
    a = orc.unique_inverse_bruteforce(ids)
    b = orc.unique_inverse(ids)
    for x, y in zip(a, b):
        assert x.dtype == np.int32 and np.array_equal(x, y)


@pytest.mark.parametrize("P,N,s", [(1000, 50, 1.5), (5000, 10_000, 0.8)])
def test_index_invariants(P, N, s):
    ids = synth.zipf_ids(3, N, s, P)
    unique, inverse, perm, seg_off = orc.unique_inverse(ids)
    U = len(unique)
    assert np.all(np.diff(unique) > 0)                            # strictly ascending
    assert np.array_equal(unique[inverse], ids)                   # inverse really inverts
    assert np.array_equal(np.sort(perm), np.arange(P))            # perm is a permutation
    assert seg_off[0] == 0 and seg_off[U] == P and np.all(np.diff(seg_off) > 0)
    for u in range(U):
        seg = perm[seg_off[u]:seg_off[u + 1]]
        assert np.all(ids[seg] == unique[u]) and np.all(np.diff(seg) > 0)   # one item, ascending positions


def test_empty_and_single():
    u, inv, perm, so = orc.unique_inverse(np.zeros(0, np.int32))
    assert len(u) == 0 and len(inv) == 0 and list(so) == [0]
    u, inv, perm, so = orc.unique_inverse(np.array([7], np.int32))
    assert list(u) == [7] and list(inv) == [0] and list(perm) == [0] and list(so) == [0, 1]


def test_segment_sum_special_cases():
    rng = np.random.default_rng(0)
    P, d = 37, 5
    dE = rng.standard_normal((P, d))
    # all-distinct IDs: G is dE reordered by the sort
    ids = rng.permutation(P)
    unique, inverse, perm, seg_off = orc.unique_inverse(ids)
    assert np.array_equal(orc.segment_sum(dE, perm, seg_off), dE[perm])
    # all-equal IDs: G is the column sum
    unique, inverse, perm, seg_off = orc.unique_inverse(np.full(P, 4))
    np.testing.assert_allclose(orc.segment_sum(dE, perm, seg_off)[0], dE.sum(0), rtol=1e-13)
    # general: column sums conserved, and equals a one-hot matrix product
    ids = synth.zipf_ids(1, 9, 1.1, P)
    unique, inverse, perm, seg_off = orc.unique_inverse(ids)
    G = orc.segment_sum(dE, perm, seg_off)
    np.testing.assert_allclose(G.sum(0), dE.sum(0), rtol=1e-12, atol=1e-12)
    onehot = (inverse[None, :] == np.arange(len(unique))[:, None]).astype(np.float64)
    np.testing.assert_allclose(G, onehot @ dE, rtol=1e-12, atol=1e-12)


def test_table_accumulate_is_scattered_segment_sum():
    rng = np.random.default_rng(1)
    N, d = 30, 4
    table = np.zeros((N, d))
    touched = np.zeros(N, bool)
    expect = np.zeros((N, d))
    union = set()
    for step in range(3):
        ids = synth.zipf_ids(5, N, 1.0, 25, step=step)
        dE = rng.standard_normal((25, d))
        orc.table_accumulate(table, touched, dE, ids)
        unique, inverse, perm, seg_off = orc.unique_inverse(ids)
        expect[unique] += orc.segment_sum(dE, perm, seg_off)
        union |= set(int(i) for i in ids)
    np.testing.assert_allclose(table, expect, rtol=1e-12, atol=1e-12)
    assert set(np.nonzero(touched)[0]) == union
    assert np.all(table[~touched] == 0)


def test_zipf_generator_shape():
    ids = synth.zipf_ids(0, 1000, 1.5, 20000)
    assert ids.min() >= 0 and ids.max() < 1000 and ids.dtype == np.int32
    top = np.bincount(ids, minlength=1000).max() / ids.size
    # rank-0 probability for s=1.5, N=1000 is 1/H(1000,1.5) ~ 0.392
    assert 0.37 < top < 0.42
    assert np.array_equal(ids, synth.zipf_ids(0, 1000, 1.5, 20000))        # seeded
    assert not np.array_equal(ids, synth.zipf_ids(0, 1000, 1.5, 20000, step=1))
