"""Pins for the step-by-step restatement of the sampled selector (oracle/sampled_steps.py).

Its selected set must equal the plain definition on every row (Theorem
"End-to-End Exactness"); its intermediate quantities are pinned by the paper's
constants (tests/golden/paper_constants.txt), by Lemma "Validated Top-K
Containment", by the monotonicity of the coarse map and by the finite-population
order statistic of Section 3.2.
"""
import os

import numpy as np
import pytest

from oracle import sampled_steps as S, topk_definition as D
from paper_2609_08450_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = [int(t) for t in v.split()]
    return out


def test_constants_match_the_paper():
    g = golden()
    assert S.B_C == g["coarse_bins"][0]
    assert list(S.DIGIT_WIDTHS) == g["digit_widths"] and sum(S.DIGIT_WIDTHS) == 32
    K = g["K_eval"][0]
    assert S.stride_for(K) == g["stride_wide"][0]
    q, q1 = S.sample_ranks(K, S.stride_for(K))
    assert (q, q1) == (g["q_eval"][0], g["q1_eval"][0])
    # q = ceil(rho K / s) for a few other (K, s), by the paper's formula in rationals
    for K, s in ((512, 32), (1024, 64), (4096, 128), (2048, 64), (1000, 32)):
        q, q1 = S.sample_ranks(K, s)
        assert q == int(np.ceil(g["rho_num"][0] * K / (g["rho_den"][0] * s) - 1e-12))
        assert q1 == int(np.ceil(g["rho1_num"][0] * K / (g["rho1_den"][0] * s) - 1e-12))
    # the coarse map uses the 11 leading bits of a 16-bit key
    assert 16 - g["coarse_shift"][0] == 11


def test_phase_schedule_is_a_permutation():
    for s in (1, 2, 32, 64, 128):
        offs = [S.phase_offset(r, s) for r in range(s)]
        assert sorted(offs) == list(range(s))                      # every block of s rows uses each phase once
        assert [S.phase_offset(r + s, s) for r in range(s)] == offs


def test_coarse_map_is_monotone_and_many_to_one():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.normal(size=20000) * 10 ** rng.uniform(-42, 38, size=20000),
                        [0.0, -0.0, np.inf, -np.inf, 65504.0, 65520.0, 1e5, -1e5, 6e-8, -6e-8]]).astype(np.float32)
    key = D.key_ascending(D.float_bits(x))
    order = np.argsort(key, kind="stable")
    c = S.coarse_bin(x)[order]
    assert (np.diff(c) <= 0).all()            # x_i > x_j  =>  c(x_i) <= c(x_j), Eq. "coarse-order"
    assert c.min() >= 0 and c.max() < S.B_C
    # fixed points of the fp16 projection: 1.0 -> h = 0x3C00 -> asc 0xBC00 -> desc 0x43FF -> bin 0x21F
    assert S.coarse_bin(np.float32([1.0]))[0] == 0x43FF >> 5
    assert S.coarse_bin(np.float32([np.inf]))[0] == (0xFFFF - 0xFC00) >> 5
    assert S.coarse_bin(np.float32([65520.0]))[0] == S.coarse_bin(np.float32([np.inf]))[0]   # RN overflow
    assert S.coarse_bin(np.float32([65519.0]))[0] == S.coarse_bin(np.float32([65504.0]))[0]
    assert S.coarse_bin(np.float32([0.0]))[0] == 0x7FFF >> 5
    assert S.coarse_bin(np.float32([-0.0]))[0] == 0x8000 >> 5
    # kappa_32 digits tile the key exactly
    k = S.kappa32_desc(x)
    rebuilt = (S.digit(k, 0).astype(np.uint64) << 21) | (S.digit(k, 1).astype(np.uint64) << 10) | S.digit(k, 2)
    assert np.array_equal(rebuilt.astype(np.uint32), k)
    assert np.array_equal(~k, key)


def _check_batch(batch, K, stride=None, capacity=None):
    s, st, ln = batch.host()
    want, _ = D.topk_rows(s, st, ln, K)
    sets, traces = S.select_rows(s, st, ln, K, stride, capacity)
    for r in range(len(ln)):
        m = min(K, max(int(ln[r]), 0))
        assert np.array_equal(np.sort(want[r, :m]), sets[r]), (batch.name, r, S.ROUTE_NAMES[traces[r].route])
    return traces


def test_equals_definition_on_random_rows():
    traces = _check_batch(W.config1(), 2048)
    assert {t.route for t in traces} >= {S.ROUTE_SHORT, S.ROUTE_PRIMARY}
    traces = _check_batch(W.config1(seed=4, num_rows=40, max_len=9000, K=128), 128)
    assert {t.route for t in traces} >= {S.ROUTE_PRIMARY, S.ROUTE_DIRECT}


def test_equals_definition_on_indexer_and_heavy_tail_rows():
    _check_batch(W.config2(num_rows=6, len_lo=9000, len_hi=20000, heads=8, dim=32), 2048)
    _check_batch(W.config3(num_rows=8, seq_len=12000, offset=11000, heads=8, dim=32, slab=4), 2048)
    _check_batch(W.config4(num_rows=3, len_lo=30000, len_hi=60000), 2048)
    _check_batch(W.config4(num_rows=3, len_lo=30000, len_hi=60000), 4096)


@pytest.mark.parametrize("K", [512, 1024, 2048])
def test_equals_definition_on_adversarial_rows_and_reaches_every_route(K):
    s = S.stride_for(K)
    traces = _check_batch(W.config5(K, s, num_rows=96, long_len=20000), K)
    routes = {t.route for t in traces}
    assert routes >= {S.ROUTE_SHORT, S.ROUTE_DIRECT, S.ROUTE_OVERFLOW}


def test_forced_band_and_recovery_routes():
    """A tight capacity / a stride that aliases the data drive the rare branches."""
    rng = np.random.default_rng(2)
    K, s = 256, 16
    hit = set()
    for trial in range(300):
        L = int(rng.integers(5000, 9000))
        x = rng.normal(size=L).astype(np.float32)
        idx, t = S.select_row(x, trial, K, stride=s, capacity=4096)
        want = D.topk_row(x, K)
        assert np.array_equal(np.sort(want), idx)
        hit.add(t.route)
        if t.route == S.ROUTE_BAND:
            assert t.C0 < K <= t.C1 and t.tau1 >= t.tau0
        if t.route == S.ROUTE_PRIMARY:
            assert t.C0 >= K
    assert S.ROUTE_PRIMARY in hit and (S.ROUTE_BAND in hit or S.ROUTE_RECOVERY in hit)


def test_containment_lemma_and_refinement_recurrence():
    rng = np.random.default_rng(9)
    K = 300
    for trial in range(10):
        L = 20000
        x = rng.standard_t(3, size=L).astype(np.float32)
        idx, t = S.select_row(x, trial, K, stride=16, capacity=1 << 20)
        c = S.coarse_bin(x)
        if t.route in (S.ROUTE_PRIMARY, S.ROUTE_BAND):
            tau = t.tau0 if t.route == S.ROUTE_PRIMARY else t.tau1
            admitted = c <= tau
            assert admitted.sum() >= K
            assert x[admitted].min() >= x[~admitted].max()          # Lemma: admitted >= excluded
            assert admitted[idx].all()                               # the answer lies inside A(tau)
        # k_{j+1} = k_j - |R_j| with |R_j| = H_j(b_j - 1), and frontiers shrink
        assert t.quotas[0] == K - (0 if t.tau_star < 0 else int((c < t.tau_star).sum()))
        assert all(a >= b for a, b in zip(t.frontier, t.frontier[1:]))
        assert all(q <= f for q, f in zip(t.quotas, t.frontier))


def test_sample_rank_matches_finite_population_order_statistic():
    """Eq. "exchangeable": E[J_a(q)] = q (L + 1) / (n_a + 1); C(tau_0) >= J_a(q)."""
    g = golden()
    L, s, K = 131071, 128, 2048
    q, _ = S.sample_ranks(K, s)
    rng = np.random.default_rng(12)
    Js = []
    for r in range(48):
        x = rng.normal(size=L).astype(np.float32)
        a = S.phase_offset(r, s)
        view = x[a::s]
        n_a = len(view)
        assert n_a in (L // s, L // s + 1)
        qth = np.sort(view)[::-1][q - 1]
        J = int((x >= qth).sum())                       # complete-row rank of the q-th largest sample
        Js.append(J)
        _, t = S.select_row(x, r, K, stride=s)
        assert t.n_view == n_a and t.a_r == a
        assert t.C0 >= J                                # the whole boundary bin is admitted
    n_a = 1023
    mean = q * (L + 1) / (n_a + 1)
    assert mean == g["EJ_L131071_n1023_q24"][0]
    var = q * (n_a - q + 1) * (L + 1) * (L - n_a) / ((n_a + 1) ** 2 * (n_a + 2))
    assert abs(np.mean(Js) - mean) < 4 * np.sqrt(var / len(Js))
