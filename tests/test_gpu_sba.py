"""GPU parity: the SBA search (func SBA of Algorithm 2) and its two helper kernels against the oracle."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl

pytestmark = pytest.mark.gpu

# The device evaluates a candidate with the hot path itself: fp16 weights and outputs, fp32 accumulation.
# Against the oracle's fp64 outputs this perturbs a candidate's KL by a relative 1e-4 at most for the
# layers below (the KL is second order in the output noise); candidates closer than that are ties.
ERR_RTOL = 1e-3
ERR_ATOL = 1e-9


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


def _layer(N, K, M, name="sba-gpu", block=0):
    seed = wl.layer_seed("test", f"{name}-{N}x{K}", block)
    return wl.make_weight(seed, N, K), wl.make_x(seed, M, K), wl.make_act_norms(seed, K)


def test_dense_linear_against_fp64():
    slim = _slim()
    for (M, N, K) in [(1, 16, 128), (5, 80, 256), (70, 200, 1024), (64, 64, 32)]:
        rng = np.random.default_rng(M * 1000 + N)
        x = rng.normal(0, 1, (M, K)).astype(np.float16)
        W = rng.normal(0, 0.05, (N, K)).astype(np.float16)
        y = slim.dense_linear(torch.from_numpy(x).cuda(), torch.from_numpy(W).cuda()).cpu().numpy()
        ref = x.astype(np.float64) @ W.astype(np.float64).T
        assert np.abs(y - ref).max() <= 2e-6 * np.abs(ref).max() * np.sqrt(K)     # fp32 accumulation of K products


def test_softmax_kl_against_the_oracle():
    slim = _slim()
    rng = np.random.default_rng(5)
    for (M, N, spread) in [(1, 16, 1.0), (7, 333, 3.0), (33, 4096, 1.5), (3, 1000, 40.0)]:
        a = rng.normal(0, spread, (M, N)).astype(np.float32)
        b = (a + rng.normal(0, 0.2 * spread, (M, N))).astype(np.float16)
        got = slim.softmax_kl(torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()).cpu().numpy()
        want = orc.softmax_kl(a, b)
        assert np.abs(got - want).max() <= 1e-11 * max(1.0, np.abs(want).max())
    same = rng.normal(0, 1, (2, 64)).astype(np.float16)
    z = slim.softmax_kl(torch.from_numpy(same.astype(np.float32)).cuda(), torch.from_numpy(same).cuda()).cpu().numpy()
    assert np.abs(z).max() <= 1e-15


def _check_search(W, x, a, avg, include_uniform=True, g=128):
    slim = _slim()
    p_star, bits, errs = slim.sba_search(torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda(),
                                         torch.from_numpy(a.astype(np.float32)).cuda(), avg, include_uniform, g=g)
    p_ref, bits_ref, errs_ref = orc.sba_search(W, x, a.astype(np.float32), avg, g=g, include_uniform=include_uniform)
    errs_ref = np.asarray(errs_ref)
    assert errs.shape == errs_ref.shape
    assert np.abs(errs - errs_ref).max() <= ERR_RTOL * np.abs(errs_ref).max() + ERR_ATOL, (errs, errs_ref)
    first = 0 if include_uniform else 1
    # the winner is the oracle's, unless the oracle's own errors tie within the tolerance: then any of the tied
    # candidates is a valid answer
    assert errs_ref[p_star - first] <= errs_ref.min() * (1 + 2 * ERR_RTOL) + ERR_ATOL
    G = W.shape[1] // g
    assert int(bits.sum()) == avg * G and (bits == avg + 1).sum() == (bits == avg - 1).sum() == p_star
    if p_star == p_ref:
        assert (bits == bits_ref).all()
    return p_star, p_ref


@pytest.mark.parametrize("N,K,M,avg", [(256, 1024, 8, 2), (512, 1024, 32, 3), (272, 1536, 64, 2), (128, 512, 1, 3)])
def test_search_matches_the_oracle(N, K, M, avg):
    W, x, a = _layer(N, K, M, block=avg)
    _check_search(W, x, a, avg)


@pytest.mark.parametrize("g,N,K,M,avg", [(32, 128, 512, 8, 2), (64, 256, 1024, 40, 2), (256, 128, 2048, 4, 2), (512, 64, 4096, 24, 2),
                                         (32, 64, 9216, 8, 3)])
def test_search_at_the_other_group_sizes(g, N, K, M, avg):
    """Groups of 32 to 512 columns (the group-size ablation of the appendix); the last case has 288 groups, more than
    a layer of 128-column groups can have.  Its weights are scaled by 1/8 (exact in fp16): with 9216 inputs the logits
    would otherwise be large enough for the fp16 rounding of the device's outputs to show in the errors at first
    order."""
    W, x, a = _layer(N, K, M, name=f"sba-gpu-g{g}")
    if K > 4096:
        W = (W.astype(np.float32) * 0.125).astype(np.float16)
    _check_search(W, x, a, avg, g=g)


def test_search_without_the_uniform_candidate_and_constructed_optimum():
    W, x, a = _layer(256, 1024, 24, name="sba-gpu-b")
    _check_search(W, x, a, 2, include_uniform=False)
    # zero groups cost nothing at one bit: the search must pair all of them with the others
    W = W.copy()
    for j in (1, 3, 4, 6):
        W[:, 128 * j:128 * (j + 1)] = 0
    p_star, p_ref = _check_search(W, x, a, 2)
    assert p_star == p_ref == 4


def test_search_rejects_bad_arguments():
    slim = _slim()
    W, x, a = _layer(128, 256, 4)
    Wd, xd, ad = torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda(), torch.from_numpy(a.astype(np.float32)).cuda()
    with pytest.raises(slim.SlimError):
        slim.sba_search(Wd, xd, ad, 4)                              # average bit-width out of range
    with pytest.raises(slim.SlimError):
        slim.sba_search(Wd, xd, ad, 2, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    W1, x1, a1 = _layer(128, 128, 4)                                # one group: only the uniform map exists
    p, bits, errs = slim.sba_search(torch.from_numpy(W1).cuda(), torch.from_numpy(x1).cuda(),
                                    torch.from_numpy(a1.astype(np.float32)).cuda(), 2)
    assert p == 0 and list(bits) == [2] and errs.shape == (1,)
    with pytest.raises(slim.SlimError):
        slim.sba_search(torch.from_numpy(W1).cuda(), torch.from_numpy(x1).cuda(), torch.from_numpy(a1.astype(np.float32)).cuda(),
                        2, include_uniform=False)
