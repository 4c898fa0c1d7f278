"""Pins for the CPU oracle: things fixed by the operator definition and by
arithmetic, none of which call the oracle's own formula back.

* rank-counting brute force (pure Python, O(L^2)) on exhaustive tiny rows
* closed forms for structured rows
* the exactness criterion of Section 6.1 plus the tie rule
* torch.sort (an unrelated library routine) where its order coincides
* fixed key values for signed zeros, infinities, subnormals
"""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import native, topk_definition as D
from tests.helpers import py_key, rank_count_topk

NINF, PINF = float("-inf"), float("inf")
SELECTORS = {
    "numpy_stable_sort": lambda s, st, ln, K: D.topk_rows(s, st, ln, K),
    "cpp_stable_sort": lambda s, st, ln, K: native.topk_stable_sort(s, st, ln, K)[:2],
    "cpp_nth_element": lambda s, st, ln, K: native.topk_nth_element(s, st, ln, K)[:2],
}


def pack(rows):
    lengths = np.array([len(r) for r in rows], dtype=np.int32)
    starts = np.zeros(len(rows), dtype=np.int32)
    starts[1:] = np.cumsum(lengths[:-1])
    flat = np.concatenate([np.asarray(r, dtype=np.float32) for r in rows]) if len(rows) else np.zeros(0, np.float32)
    return flat, starts, lengths


def run_one(sel, row, K):
    flat, st, ln = pack([row])
    idx, val = SELECTORS[sel](flat, st, ln, K)
    return idx[0], val[0]


def test_key_fixed_points():
    assert py_key(-0.0) == 0x7FFFFFFF and py_key(0.0) == 0x80000000
    assert py_key(PINF) == 0xFF800000 and py_key(NINF) == 0x007FFFFF
    vals = np.array([NINF, -3.5, -1e-40, -0.0, 0.0, 1e-45, 1e-40, 2.0, 3.4e38, PINF], dtype=np.float32)
    keys = D.key_ascending(D.float_bits(vals))
    assert (np.diff(keys.astype(np.int64)) > 0).all()          # strictly increasing with value
    assert [int(k) for k in keys] == [py_key(float(v)) for v in vals]
    rng = np.random.default_rng(0)
    x = np.sort(rng.normal(size=4096).astype(np.float32) * np.float32(1e3))
    assert (np.diff(D.key_ascending(D.float_bits(x)).astype(np.int64)) >= 0).all()


@pytest.mark.parametrize("sel", list(SELECTORS))
def test_exhaustive_tiny_rows_against_rank_counting(sel):
    alphabet = [NINF, -0.0, 0.0, 1.0, PINF]
    rows, want = [], {}
    for L in range(0, 6):
        for row in itertools.product(alphabet, repeat=L):
            rows.append(list(row))
    flat, st, ln = pack(rows)
    for K in (1, 2, 3, 5, 8):
        idx, val = SELECTORS[sel](flat, st, ln, K)
        for r, row in enumerate(rows):
            m = min(K, len(row))
            assert sorted(idx[r, :m].tolist()) == rank_count_topk(row, K)
            assert (idx[r, m:] == -1).all()
            assert (val[r, m:].view(np.uint32) == 0xFF800000).all()
            got_bits = val[r, :m].view(np.uint32)
            src_bits = np.asarray(row, dtype=np.float32).view(np.uint32)[idx[r, :m]] if m else got_bits
            assert np.array_equal(got_bits, src_bits)


@pytest.mark.parametrize("sel", list(SELECTORS))
def test_random_small_rows_against_rank_counting(sel):
    rng = np.random.default_rng(7)
    for trial in range(120):
        L = int(rng.integers(0, 65))
        K = int(rng.integers(1, 9))
        row = rng.integers(-3, 4, size=L).astype(np.float32) * np.float32(0.5)   # many ties
        if L and rng.random() < 0.5:
            row[rng.integers(0, L)] = -0.0
        idx, _ = run_one(sel, row, K)
        m = min(K, L)
        assert sorted(idx[:m].tolist()) == rank_count_topk(row, K)
        # best-first slot order: keys non-increasing, equal keys by ascending index
        keys = [py_key(float(row[i])) for i in idx[:m]]
        assert all(keys[j] > keys[j + 1] or (keys[j] == keys[j + 1] and idx[j] < idx[j + 1])
                   for j in range(m - 1))


@pytest.mark.parametrize("sel", list(SELECTORS))
def test_closed_forms(sel):
    K, L = 64, 1000
    first = list(range(K))
    # constant row: all keys tie, lowest indices win
    assert sorted(run_one(sel, np.full(L, 2.5), K)[0].tolist()) == first
    # strictly ascending / descending
    asc = np.arange(L, dtype=np.float32)
    assert sorted(run_one(sel, asc, K)[0].tolist()) == list(range(L - K, L))
    assert sorted(run_one(sel, asc[::-1].copy(), K)[0].tolist()) == first
    # one contiguous block of K large values
    x = np.zeros(L, dtype=np.float32)
    x[300:300 + K] = 7.0
    assert sorted(run_one(sel, x, K)[0].tolist()) == list(range(300, 300 + K))
    # 4 levels, x_i = i mod 4: level 3 entirely (250 > K) -> lowest-index positions of level 3
    lev = (np.arange(L) % 4).astype(np.float32)
    assert sorted(run_one(sel, lev, K)[0].tolist()) == [4 * j + 3 for j in range(K)]
    # level 3 (250) + lowest indices of level 2 when K = 300
    want = sorted([i for i in range(L) if i % 4 == 3] + [4 * j + 2 for j in range(50)])
    assert sorted(run_one(sel, lev, 300)[0].tolist()) == want
    # signed zeros: +0.0 beats -0.0; among each, lower index first
    z = np.array([-0.0, 0.0, -0.0, 0.0, -0.0, 0.0, -0.0], dtype=np.float32)
    assert sorted(run_one(sel, z, 3)[0].tolist()) == [1, 3, 5]
    assert sorted(run_one(sel, z, 5)[0].tolist()) == [0, 1, 2, 3, 5]
    # fewer than K finite values: all finite positions, then lowest-index -inf
    p = np.full(20, NINF, dtype=np.float32)
    p[[4, 9, 15]] = [1.0, -2.0, 0.5]
    assert sorted(run_one(sel, p, 6)[0].tolist()) == [0, 1, 2, 4, 9, 15]
    # short rows: every index, then sentinels
    idx, val = run_one(sel, np.array([3.0, 1.0, 2.0], dtype=np.float32), 5)
    assert sorted(idx[:3].tolist()) == [0, 1, 2] and (idx[3:] == -1).all()
    assert np.isneginf(val[3:]).all()
    idx, _ = run_one(sel, np.zeros(0, dtype=np.float32), 4)
    assert (idx == -1).all()
    # L == K: every index, no padding
    assert sorted(run_one(sel, np.arange(8, dtype=np.float32), 8)[0].tolist()) == list(range(8))


@pytest.mark.parametrize("sel", list(SELECTORS))
def test_periodic_rows_closed_form(sel):
    s, L, K = 32, 32 * 40, 100          # x_i = v[i mod s]; each residue occurs 40 times
    v = np.random.default_rng(3).permutation(s).astype(np.float32)
    x = v[np.arange(L) % s]
    top = np.argsort(-v)                 # residues from best to worst
    want = [i for i in range(L) if i % s in top[:2]]             # 80 positions taken whole
    want += [top[2] + s * j for j in range(20)]                  # lowest 20 of the boundary residue
    assert sorted(run_one(sel, x, K)[0].tolist()) == sorted(int(i) for i in want)


@pytest.mark.parametrize("sel", list(SELECTORS))
def test_exactness_criterion_and_tie_rule(sel):
    """Section 6.1: no unselected valid score exceeds a selected one; plus the tie rule."""
    rng = np.random.default_rng(11)
    for trial in range(20):
        L = int(rng.integers(50, 5000))
        K = int(rng.integers(1, 600))
        x = np.round(rng.standard_t(3, size=L), 1).astype(np.float32)     # ties + heavy tail
        idx, val = run_one(sel, x, K)
        m = min(K, L)
        chosen = idx[:m]
        assert len(set(chosen.tolist())) == m and chosen.min() >= 0 and chosen.max() < L
        mask = np.zeros(L, bool)
        mask[chosen] = True
        if m < L:
            assert x[mask].min() >= x[~mask].max()
            T = x[mask].min()
            ties = np.nonzero(x == T)[0]                                   # no signed zeros here
            x_nozero = not np.any(x == 0)
            if x_nozero:
                n_sel = int(mask[ties].sum())
                assert np.array_equal(np.nonzero(mask[ties])[0], np.arange(n_sel))
        assert np.array_equal(val[:m].view(np.uint32), x[chosen].view(np.uint32))


def test_torch_stable_sort_agrees_where_orders_coincide():
    g = torch.Generator().manual_seed(5)
    for L, K in ((1000, 17), (40000, 2048), (5000, 5000)):
        x = torch.randn(L, generator=g)
        x = torch.round(x * 50) / 50 + 0.001          # ties, but never a zero of either sign
        order = torch.sort(x, descending=True, stable=True).indices[:K].numpy()
        for sel in SELECTORS:
            idx, val = run_one(sel, x.numpy(), K)
            assert np.array_equal(idx[:min(K, L)], order[:min(K, L)])
        tv = torch.topk(x, min(K, L)).values.numpy()
        assert np.array_equal(np.sort(val[:min(K, L)]), np.sort(tv))


def test_three_selectors_agree_on_config_batches():
    from paper_2609_08450_b200 import workloads as W
    for batch, K in ((W.config1(), 2048), (W.config5(512, 32, num_rows=96, long_len=9000), 512)):
        s, st, ln = batch.host()
        a = SELECTORS["numpy_stable_sort"](s, st, ln, K)
        b = SELECTORS["cpp_stable_sort"](s, st, ln, K)
        c = SELECTORS["cpp_nth_element"](s, st, ln, K)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[0], c[0])
        assert np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
        assert np.array_equal(a[1].view(np.uint32), c[1].view(np.uint32))


def test_nan_has_a_defined_place():
    x = np.array([1.0, np.nan, PINF, -1.0], dtype=np.float32)
    neg_nan = np.array([0xFFC00000], dtype=np.uint32).view(np.float32)[0]
    x[3] = neg_nan
    for sel in SELECTORS:
        idx, _ = run_one(sel, x, 2)
        assert sorted(idx.tolist()) == [1, 2]          # +NaN above +inf
        idx, _ = run_one(sel, x, 3)
        assert sorted(idx.tolist()) == [0, 1, 2]       # -NaN below everything
