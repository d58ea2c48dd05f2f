"""GPU parity: salience, bit allocation and the Eq. 1 quantizer against the oracle."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


@pytest.mark.parametrize("N,K,avg", [(64, 512, 2), (1024, 4096, 2), (272, 11008, 3), (512, 5120, 3)])
def test_salience_bits_and_quantizer_match_oracle(N, K, avg):
    slim = _slim()
    seed = wl.layer_seed("test", f"quant-{N}x{K}", avg)
    W = wl.make_weight(seed, N, K)
    a = wl.make_act_norms(seed, K)
    sal_ref = orc.group_salience(W, a)
    sal = slim.group_salience(torch.from_numpy(W).cuda(), torch.from_numpy(a).cuda()).cpu().numpy()
    assert np.allclose(sal, sal_ref, rtol=1e-12, atol=0)
    bits_ref = orc.allocate_bits(sal_ref, avg)
    bits = slim.allocate_bits(sal, avg)
    # the ranking is decided in fp64 on both sides; a different map is only acceptable on a near-tie
    if not (bits == bits_ref).all():
        diff = np.flatnonzero(bits != bits_ref)
        order = np.sort(sal_ref)
        gaps = np.min(np.abs(sal_ref[diff][:, None] - np.delete(order, 0)[None, :]), axis=1)
        assert (gaps <= 1e-11 * sal_ref[diff]).all(), "bit maps differ without a salience tie"
    assert int(bits.astype(int).sum()) == avg * (K // 128)
    codes, scales, zeros = slim.quantize_minmax(torch.from_numpy(W).cuda(), bits_ref)
    c_ref, s_ref, z_ref = orc.quantize_minmax(W, bits_ref)
    assert (scales.cpu().numpy().view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.cpu().numpy().view(np.uint16) == z_ref.view(np.uint16)).all()
    assert (codes.cpu().numpy() == c_ref).all()


def test_quantizer_edge_groups():
    """All-positive, all-negative, constant-zero, huge-range and tiny-range groups."""
    slim = _slim()
    rng = np.random.default_rng(3)
    N, K = 16, 640
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    W[:, 0:128] = np.abs(W[:, 0:128])
    W[:, 128:256] = -np.abs(W[:, 128:256])
    W[:, 256:384] = 0
    W[:, 384:512] = np.clip(rng.standard_normal((N, 128)) * 3e4, -6e4, 6e4).astype(np.float16)   # range beyond fp16 for 1 bit
    W[:, 512:640] = (rng.standard_normal((N, 128)) * 1e-7).astype(np.float16)  # subnormal weights
    for bits in ([1, 2, 3, 1, 4], [4, 3, 2, 1, 1], [2, 2, 2, 2, 2]):
        bits = np.array(bits, dtype=np.uint8)
        c_ref, s_ref, z_ref = orc.quantize_minmax(W, bits)
        codes, scales, zeros = slim.quantize_minmax(torch.from_numpy(W).cuda(), bits)
        assert (scales.cpu().numpy().view(np.uint16) == s_ref.view(np.uint16)).all()
        assert (zeros.cpu().numpy().view(np.uint16) == z_ref.view(np.uint16)).all()
        assert (codes.cpu().numpy() == c_ref).all()


def test_allocate_bits_host_matches_oracle_on_ties_and_p():
    slim = _slim()
    rng = np.random.default_rng(5)
    for G in (4, 32, 86, 108, 224):
        S = rng.integers(0, 6, G).astype(np.float64)   # many ties
        for avg in (2, 3):
            assert (slim.allocate_bits(S, avg) == orc.allocate_bits(S, avg)).all()
            for p in (0, 1, G // 2):
                assert (slim.allocate_bits(S, avg, p) == orc.allocate_bits(S, avg, p)).all()


@pytest.mark.parametrize("N,K,bits", [(48, 1024, [1, 2, 3, 4, 2, 3, 1, 4]), (272, 512, [2, 3, 3, 2]), (64, 11008, None)])
def test_sqc_line_search_matches_oracle_bit_for_bit(N, K, bits):
    """slim_quantize_sqc (function SQC of Algorithm 2): codes, scales, zero points and the chosen
    candidate must equal the oracle's; both sides decide in fp64 with column-order sums."""
    slim = _slim()
    seed = wl.layer_seed("test", f"sqc-{N}x{K}", 0)
    W = wl.make_weight(seed, N, K)
    if bits is None:
        bits = orc.allocate_bits(orc.group_salience(W, wl.make_act_norms(seed, K)), 2)
    bits = np.asarray(bits, dtype=np.uint8)
    c_ref, s_ref, z_ref, t_ref, _, _ = orc.quantize_sqc(W, bits)
    codes, scales, zeros, tau = slim.quantize_sqc(torch.from_numpy(W).cuda(), bits)
    assert (tau.cpu().numpy() == t_ref).all()
    assert (scales.cpu().numpy().view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.cpu().numpy().view(np.uint16) == z_ref.view(np.uint16)).all()
    assert (codes.cpu().numpy() == c_ref).all()


def test_sqc_edge_groups_and_other_grids():
    slim = _slim()
    rng = np.random.default_rng(13)
    N, K = 16, 512
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    W[:, 0:128] = np.abs(W[:, 0:128])          # all positive
    W[:, 128:256] = 0                          # constant zero
    W[:, 256:384] = (rng.standard_normal((N, 128)) * 1e-7).astype(np.float16)   # subnormal weights
    W[:, 400] = np.float16(3.0)                # one strong outlier
    for bits, lam, n in ([[1, 2, 3, 4], 0.1, 50], [[4, 3, 2, 1], 0.25, 10], [[2, 2, 2, 2], 0.0, 1]):
        bits = np.array(bits, dtype=np.uint8)
        c_ref, s_ref, z_ref, t_ref, _, _ = orc.quantize_sqc(W, bits, lam=lam, n=n)
        codes, scales, zeros, tau = slim.quantize_sqc(torch.from_numpy(W).cuda(), bits, lam=lam, n=n)
        assert (tau.cpu().numpy() == t_ref).all()
        assert (scales.cpu().numpy().view(np.uint16) == s_ref.view(np.uint16)).all()
        assert (zeros.cpu().numpy().view(np.uint16) == z_ref.view(np.uint16)).all()
        assert (codes.cpu().numpy() == c_ref).all()


@pytest.mark.parametrize("N,K,M", [(272, 1536, 1), (512, 1024, 5), (256, 2048, 40)])
def test_eq2_one_bit_groups_end_to_end(N, K, M):
    """Eq. 2 for the one-bit groups: quantizer bit-exact against the oracle, then the packed layer through every
    entry point of the hot path (z = 1/2) against the fp64 oracle."""
    from tests.helpers import check_output
    slim = _slim()
    seed = wl.layer_seed("test", f"sign1-{N}x{K}", M)
    W, a, x = wl.make_weight(seed, N, K), wl.make_act_norms(seed, K), wl.make_x(seed, M, K)
    bits = orc.allocate_bits(orc.group_salience(W, a), 2)
    assert (bits == 1).sum() == K // 128 // 4
    codes, scales, zeros = slim.quantize_minmax(torch.from_numpy(W).cuda(), bits, one_bit="sign_alpha")
    c_ref, s_ref, z_ref = orc.quantize_minmax_sign1(W, bits)
    assert (codes.cpu().numpy() == c_ref).all()
    assert (scales.cpu().numpy().view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.cpu().numpy().view(np.uint16) == z_ref.view(np.uint16)).all()
    packed = slim.pack_weights(codes, bits)
    What = slim.dequant(packed, bits, scales, zeros, N, K).cpu().numpy()
    assert (What.view(np.uint16) == orc.dequant_f16(c_ref, s_ref, z_ref).view(np.uint16)).all()
    y_ref = orc.linear_f64(x, c_ref, s_ref, z_ref)
    xd = torch.from_numpy(x).cuda()
    layer = slim.QuantLinear(packed, bits, scales, zeros, N, K)
    ws = slim.new_workspace(M, N, K, bits)
    check_output(layer.forward(xd, ws).cpu().numpy(), y_ref, f"Eq. 2 groups, M={M}")
    slim.workspace_status(ws)
    if M <= 16:
        y = torch.empty(M, N, dtype=torch.float16, device="cuda")
        s = slim.LayerSet([(layer, xd, y)])
        s.run()
        s.check()
        check_output(y.cpu().numpy(), y_ref, f"Eq. 2 groups, layer set, M={M}")


@pytest.mark.parametrize("b", [1, 2, 3, 4])
def test_quantizer_exact_ties_round_to_even(b):
    """Weights exactly half-way between two grid points (w / s = k + 1/2): both sides must round to the even code."""
    slim = _slim()
    levels = 2 ** b - 1
    s = 2.0 ** -6
    rng = np.random.default_rng(b)
    W = np.empty((32, 256), dtype=np.float16)
    for n in range(32):
        for j in range(2):
            k = rng.integers(0, levels, 128)
            w = (k + 0.5) * s                      # exact ties
            w[0], w[1] = 0.0, levels * s           # the group's range is exactly [0, levels * s]: scale s, zero point 0
            if n % 2:                              # every other row mirrored: negative range, zero point = levels
                w = -w
            W[n, 128 * j:128 * j + 128] = w
    bits = np.array([b, b], dtype=np.uint8)
    c_ref, s_ref, z_ref = orc.quantize_minmax(W, bits)
    assert (s_ref.astype(np.float64) == s).all()
    codes, scales, zeros = slim.quantize_minmax(torch.from_numpy(W).cuda(), bits)
    assert (codes.cpu().numpy() == c_ref).all()
    assert (scales.cpu().numpy().view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.cpu().numpy().view(np.uint16) == z_ref.view(np.uint16)).all()
    # ties really occurred and went both ways
    k_plus = (c_ref[0::2, 2:128].astype(np.int64) - np.floor(W[0::2, 2:128].astype(np.float64) / s)).ravel()
    assert set(np.unique(k_plus)) <= {0, 1} and (len(set(np.unique(k_plus))) == 2 or b == 1)


def test_requantising_a_subset_of_groups():
    slim = _slim()
    seed = wl.layer_seed("test", "quant-subset", 0)
    W = wl.make_weight(seed, 272, 1024)
    bits_a = np.array([2, 2, 2, 2, 2, 2, 2, 2], dtype=np.uint8)
    bits_b = np.array([2, 3, 2, 2, 1, 2, 2, 4], dtype=np.uint8)
    Wd = torch.from_numpy(W).cuda()
    codes, scales, zeros = slim.quantize_minmax(Wd, bits_a)
    slim.quantize_minmax_groups(Wd, bits_b, [7, 1, 4], codes, scales, zeros)
    c_ref, s_ref, z_ref = orc.quantize_minmax(W, bits_b)       # groups 0, 2, 3, 5, 6 have the same width in both maps
    assert (codes.cpu().numpy() == c_ref).all()
    assert (scales.cpu().numpy().view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.cpu().numpy().view(np.uint16) == z_ref.view(np.uint16)).all()
    with pytest.raises(slim.SlimError):
        slim.quantize_minmax_groups(Wd, bits_b, [8], codes, scales, zeros)
