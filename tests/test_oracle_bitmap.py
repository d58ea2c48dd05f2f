"""Pins for the oracle's salience ranking and bit allocation (Eq. 4 constraint, Sec. 3.2.2)."""
import numpy as np
import pytest

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl


@pytest.mark.parametrize("K", [4096, 11008, 5120, 13824, 8192, 28672])
@pytest.mark.parametrize("avg", [2, 3])
def test_budget_is_exact(K, avg):
    G = K // 128
    S = np.random.default_rng(K + avg).random(G)
    bits = orc.allocate_bits(S, avg)
    # sum_j b_j * g / K equals the target average exactly
    assert int(bits.astype(np.int64).sum()) * 128 == avg * K
    assert (bits == avg + 1).sum() == (bits == avg - 1).sum() == G // 4
    assert set(np.unique(bits)) <= {avg - 1, avg, avg + 1}


def test_llama7b_has_32_groups_and_16_candidates():
    # "only 16 iterations are needed in LLaMA-7B": search range [0, k/2] with k = m/128
    G = 4096 // 128
    assert G == 32 and G // 2 == 16
    S = np.arange(G, dtype=np.float64)
    for p in range(0, G // 2 + 1):
        bits = orc.allocate_bits(S, 2, p)
        assert bits.astype(int).sum() == 2 * G
        assert (bits == 3).sum() == p and (bits == 1).sum() == p
    # extreme cases named in App. C: uniform, and half/half without N-bit groups
    assert (orc.allocate_bits(S, 2, 0) == 2).all()
    assert set(np.unique(orc.allocate_bits(S, 2, G // 2))) == {1, 3}


def test_most_salient_get_more_bits_and_ties_break_by_index():
    S = np.array([5.0, 1.0, 9.0, 1.0, 3.0, 7.0, 0.5, 2.0])
    bits = orc.allocate_bits(S, 2)  # p = 2; groups 1 and 3 tie, the lower index counts as more salient
    assert bits.tolist() == [2, 2, 3, 1, 2, 3, 1, 2]
    S = np.ones(8)
    assert orc.allocate_bits(S, 3).tolist() == [4, 4, 3, 3, 3, 3, 2, 2]


def test_permutation_equivariance():
    rng = np.random.default_rng(7)
    S = rng.random(40)
    perm = rng.permutation(40)
    assert (orc.allocate_bits(S[perm], 3) == orc.allocate_bits(S, 3)[perm]).all()


def test_salience_matches_brute_force_and_outlier_channel_wins():
    rng = np.random.default_rng(11)
    N, K = 8, 512
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    a = np.exp(rng.standard_normal(K)).astype(np.float32)
    S = orc.group_salience(W, a)
    for j in range(K // 128):
        ref = 0.0
        for k in range(128 * j, 128 * j + 128):
            col = 0.0
            for n in range(N):
                col += float(W[n, k]) ** 2
            ref += float(a[k]) ** 2 * col
        assert S[j] == pytest.approx(ref, rel=1e-12)
    # Theorem 1: an outlier activation channel makes its group the most salient one
    a2 = np.ones(K, dtype=np.float32)
    a2[300] = 1000.0
    assert int(np.argmax(orc.group_salience(W, a2))) == 300 // 128
    # scaling a weight column by 10 raises its group's salience by 99x that column's share
    W2 = W.copy().astype(np.float64)
    S0 = orc.group_salience(W, np.ones(K))
    W2[:, 5] *= 10
    S1 = orc.group_salience(W2, np.ones(K))
    assert S1[0] - S0[0] == pytest.approx(99 * (W[:, 5].astype(np.float64) ** 2).sum(), rel=1e-9)
    assert np.allclose(S1[1:], S0[1:], rtol=0, atol=0)


def test_config_recipe_quartiles():
    seed = wl.layer_seed("llama-7b", "q", 0)
    W = wl.make_weight(seed, 256, 4096)
    a = wl.make_act_norms(seed, 4096)
    bits = orc.allocate_bits(orc.group_salience(W, a), 2)
    assert (bits == 3).sum() == 8 and (bits == 1).sum() == 8 and (bits == 2).sum() == 16
