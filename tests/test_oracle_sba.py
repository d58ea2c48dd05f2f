"""Pins of the oracle's SBA search (Algorithm 2, func SBA; Sec. 3.2.2, Eq. 4) against things other than
itself: a library KL, closed forms, invariances, a scalar brute force and constructed optima."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl


def _layer(N, K, M, name="sba", block=0, outliers=True):
    seed = wl.layer_seed("test", f"{name}-{N}x{K}", block)
    W = wl.make_weight(seed, N, K, outlier_frac=0.01 if outliers else 0.0)
    return W, wl.make_x(seed, M, K), wl.make_act_norms(seed, K)


# ------------------------------------------------------------------------------------------ the error measure
def test_kl_matches_the_library_definition():
    rng = np.random.default_rng(7)
    a = rng.normal(0, 2.0, (5, 37))
    b = a + rng.normal(0, 0.3, (5, 37))
    got = orc.softmax_kl(a, b)
    for t in range(5):
        want = scipy.stats.entropy(scipy.special.softmax(a[t]), scipy.special.softmax(b[t]))
        assert abs(got[t] - want) <= 1e-12 * max(1.0, abs(want))


def test_kl_two_outputs_is_the_bernoulli_closed_form():
    # softmax([u, 0]) = (sigmoid(u), 1 - sigmoid(u))
    for u, v in [(0.3, -1.2), (2.0, 2.5), (-4.0, 1.0)]:
        p, q = 1 / (1 + math.exp(-u)), 1 / (1 + math.exp(-v))
        want = p * math.log(p / q) + (1 - p) * math.log((1 - p) / (1 - q))
        got = orc.softmax_kl(np.array([[u, 0.0]]), np.array([[v, 0.0]]))[0]
        assert abs(got - want) <= 1e-14


def test_kl_is_zero_only_for_equal_distributions_and_ignores_row_shifts():
    rng = np.random.default_rng(3)
    a = rng.normal(0, 1.0, (4, 64))
    b = a + rng.normal(0, 0.1, (4, 64))
    assert np.abs(orc.softmax_kl(a, a)).max() <= 1e-15
    d = orc.softmax_kl(a, b)
    assert (d > 0).all()
    shift_a, shift_b = rng.normal(0, 50, (4, 1)), rng.normal(0, 50, (4, 1))
    assert np.abs(orc.softmax_kl(a + shift_a, b + shift_b) - d).max() <= 1e-12
    # not symmetric, and large logits do not overflow
    assert np.abs(orc.softmax_kl(b, a) - d).max() > 0
    assert np.isfinite(orc.softmax_kl(a * 1e3, b * 1e3)).all()


# ------------------------------------------------------------------------------------------ the search
def test_budget_and_double_pointer_shape():
    for avg in (2, 3):
        W, x, a = _layer(64, 1024, 8, block=avg)
        p_star, bits, errs = orc.sba_search(W, x, a, avg)
        G = 8
        assert len(errs) == G // 2 + 1 and 0 <= p_star <= G // 2
        assert int(bits.sum()) == avg * G                               # the average bit-width is kept exactly
        assert (bits == avg + 1).sum() == (bits == avg - 1).sum() == p_star
        S = orc.group_salience(W, a)
        order = sorted(range(G), key=lambda j: (-S[j], j))
        assert set(np.nonzero(bits == avg + 1)[0]) == set(order[:p_star])
        assert set(np.nonzero(bits == avg - 1)[0]) == set(order[G - p_star:] if p_star else [])
        assert errs[p_star] == min(errs) and all(e > errs[p_star] for e in errs[:p_star])   # first minimum


def _scalar_candidate_error(W, x, bits, g=128):
    """Error of one bit map, element by element with Python floats: Eq. 1 per (row, group), output, softmax, KL."""
    N, K = W.shape
    M = x.shape[0]
    What = [[0.0] * K for _ in range(N)]
    for n in range(N):
        for j, b in enumerate(bits):
            w = [float(W[n, k]) for k in range(g * j, g * j + g)]
            lo, hi, levels = min(min(w), 0.0), max(max(w), 0.0), 2 ** int(b) - 1
            s = float(np.float16((hi - lo) / levels))
            if s == 0.0:
                s = 1.0
            z = min(max(-float(np.rint(lo / s)), 0.0), levels)
            for i, v in enumerate(w):
                q = min(max(float(np.rint(v / s)) + z, 0.0), levels)
                What[n][g * j + i] = s * (q - z)
    total = 0.0
    for t in range(M):
        yf = [sum(float(x[t, k]) * float(W[n, k]) for k in range(K)) for n in range(N)]
        yq = [sum(float(x[t, k]) * What[n][k] for k in range(K)) for n in range(N)]
        lf = math.log(sum(math.exp(v - max(yf)) for v in yf)) + max(yf)
        lq = math.log(sum(math.exp(v - max(yq)) for v in yq)) + max(yq)
        total += sum(math.exp(a - lf) * ((a - lf) - (b - lq)) for a, b in zip(yf, yq))
    return total / M


def test_search_against_scalar_brute_force():
    W, x, a = _layer(3, 512, 2, name="sba-brute")
    p_star, bits, errs = orc.sba_search(W, x, a, 2)
    S = orc.group_salience(W, a)
    want = [_scalar_candidate_error(W, x, orc.allocate_bits(S, 2, p)) for p in range(3)]
    for e, w in zip(errs, want):
        assert abs(e - w) <= 1e-9 * max(w, 1e-12)
    assert p_star == min(range(3), key=lambda p: (want[p], p))


@pytest.mark.parametrize("g", [32, 64, 256])
def test_search_against_scalar_brute_force_at_other_group_sizes(g):
    """The search ranks, quantises and scores groups of g columns (the group-size ablation of the appendix)."""
    W, x, a = _layer(3, 4 * g, 2, name=f"sba-brute-g{g}")
    p_star, bits, errs = orc.sba_search(W, x, a, 2, g=g)
    S = orc.group_salience(W, a, g)
    assert len(bits) == 4 and len(errs) == 3
    want = [_scalar_candidate_error(W, x, orc.allocate_bits(S, 2, p), g) for p in range(3)]
    for e, w in zip(errs, want):
        assert abs(e - w) <= 1e-9 * max(w, 1e-12)
    assert p_star == min(range(3), key=lambda p: (want[p], p))


def test_constructed_optimum_all_pairs_when_low_groups_cost_nothing():
    # half of the groups are zero (no salience, exact at any width); the others gain from every extra bit
    W, x, a = _layer(32, 1024, 6, name="sba-zero-groups", outliers=False)
    W = W.copy()
    for j in (1, 3, 4, 6):
        W[:, 128 * j:128 * (j + 1)] = 0
    p_star, bits, errs = orc.sba_search(W, x, a, 2)
    assert p_star == 4 and all(errs[i + 1] < errs[i] for i in range(4))
    assert all(bits[j] == 1 for j in (1, 3, 4, 6)) and all(bits[j] == 3 for j in (0, 2, 5, 7))


def test_constructed_optimum_uniform_when_the_weight_is_on_the_grid():
    # every group takes values on a 4-level grid containing 0: exact at 2 bits, so p = 0 has error 0
    rng = np.random.default_rng(11)
    W = (rng.integers(0, 4, (16, 512)) * 0.125 - 0.125).astype(np.float16)
    W[:, ::128] = -0.125
    W[:, 1::128] = 0.25          # every (row, group) spans the whole grid
    x = rng.normal(0, 1, (4, 512)).astype(np.float16)
    a = np.exp(rng.normal(0, 1, 512))
    p_star, bits, errs = orc.sba_search(W, x, a, 2)
    assert p_star == 0 and errs[0] <= 1e-20 and (bits == 2).all()
    p1, bits1, errs1 = orc.sba_search(W, x, a, 2, include_uniform=False)      # Algorithm 2's loop as printed
    assert p1 >= 1 and len(errs1) == 2 and (bits1 == 3).sum() == p1


def test_ties_keep_the_first_candidate_and_groups_permute_with_the_map():
    Wz = np.zeros((8, 512), np.float16)
    x = np.ones((2, 512), np.float16)
    assert orc.sba_search(Wz, x, np.ones(512), 3)[0] == 0
    W, x, a = _layer(48, 1024, 4, name="sba-perm")
    p_star, bits, errs = orc.sba_search(W, x, a, 3)
    perm = np.array([5, 2, 7, 0, 3, 6, 1, 4])
    cols = np.concatenate([np.arange(128 * j, 128 * j + 128) for j in perm])
    p2, bits2, errs2 = orc.sba_search(W[:, cols], x[:, cols], a[cols], 3)
    assert p2 == p_star and (bits2 == bits[perm]).all()
    assert np.allclose(errs, errs2, rtol=1e-9, atol=0)
