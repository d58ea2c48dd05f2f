"""GPU parity: the GPTQ error-compensation loop (Algorithm 1) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


def _layer(N, K, T, name="gptq-gpu", block=0):
    seed = wl.layer_seed("test", f"{name}-{N}x{K}", block)
    return wl.make_weight(seed, N, K), wl.make_calibration_x(seed, T, K)


# 384, 640 and 1408 columns: a number of 64-column blocks that is not a power of two (ragged last segments of the
# doubling inverse)
@pytest.mark.parametrize("K,T", [(128, 16), (256, 300), (384, 200), (512, 100), (640, 64), (1024, 1500), (1408, 700)])
def test_factor_against_the_library_cholesky_of_the_inverse(K, T):
    slim = _slim()
    _, x = _layer(4, K, T)
    U, dead = slim.gptq_factor(torch.from_numpy(x).cuda(), 0.01)
    U_ref, dead_ref = orc.gptq_factor(orc.gptq_hessian(x), 0.01)
    U = U.cpu().numpy()
    assert (dead.cpu().numpy().astype(bool) == dead_ref).all()
    assert np.abs(np.tril(U, -1)).max() == 0
    # fp64 on both sides, two routes to the same factor (inverse of the reversed Cholesky factor here, Cholesky of the
    # inverse there): they differ by rounding amplified by the condition number (about 1/lambda times the spread of diag H)
    assert np.abs(U - U_ref).max() <= 1e-9 * np.abs(U_ref).max()


def _check_quantize(W, x, bits, quantizer, lam=0.01, g=128):
    slim = _slim()
    codes, scales, zeros, running = slim.gptq_quantize(torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda(), bits, lam, quantizer,
                                                       return_running=True, g=g)
    c_ref, s_ref, z_ref, w_ref = orc.gptq_quantize(W, x, np.asarray(bits), lam, quantizer, g)
    codes, scales, zeros, running = codes.cpu().numpy(), scales.cpu().numpy(), zeros.cpu().numpy(), running.cpu().numpy()
    assert (scales.view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.view(np.uint16) == z_ref.view(np.uint16)).all()
    assert (codes == c_ref).all(), f"{(codes != c_ref).sum()} codes differ"
    assert np.abs(running - w_ref).max() <= 1e-9 * max(1.0, np.abs(w_ref).max())
    return codes, scales, zeros


@pytest.mark.parametrize("N,K,T,bits", [(64, 512, 128, [2, 1, 3, 2]), (272, 1024, 300, [3, 2, 4, 3, 3, 2, 4, 3]),
                                        (16, 128, 40, [2]), (130, 256, 64, [1, 3]), (48, 384, 500, [3, 2, 1]),
                                        (32, 1408, 256, [2, 3, 1, 2, 3, 2, 2, 1, 3, 2, 2])])
@pytest.mark.parametrize("quantizer", ["minmax", "sqc"])
def test_quantize_matches_the_oracle(N, K, T, bits, quantizer):
    if N % 16:
        N = N // 16 * 16 + 16
    W, x = _layer(N, K, T, block=len(bits))
    _check_quantize(W, x, bits, quantizer)


@pytest.mark.parametrize("g,N,K,T", [(32, 48, 384, 200), (32, 16, 1152, 300), (64, 80, 512, 128), (256, 64, 1024, 300), (512, 32, 1536, 400)])
@pytest.mark.parametrize("quantizer", ["minmax", "sqc"])
def test_quantize_at_the_other_group_sizes(g, N, K, T, quantizer):
    """Algorithm 1 with blocks of g columns (the group-size ablation of the appendix).  At g = 32 every other
    trailing region ends in the middle of a 64-column tile of the update."""
    rng = np.random.default_rng(g + K)
    bits = rng.integers(1, 5, K // g)
    W, x = _layer(N, K, T, block=g)
    _check_quantize(W, x, bits, quantizer, g=g)


def test_uncorrelated_inputs_and_dead_channel():
    slim = _slim()
    K = 256
    W = wl.make_weight(wl.layer_seed("test", "gptq-gpu-eye", 0), 32, K)
    x = (np.eye(K) * 3.0).astype(np.float16)
    codes, scales, zeros = _check_quantize(W, x, [2, 3], "minmax")
    q, s, z = slim.quantize_minmax(torch.from_numpy(W).cuda(), [2, 3])
    assert (codes == q.cpu().numpy()).all() and (scales == s.cpu().numpy()).all()
    W2, x2 = _layer(48, 256, 64, name="gptq-gpu-dead")
    x2 = x2.copy()
    x2[:, 5] = 0
    x2[:, 200] = 0
    codes, scales, zeros = _check_quantize(W2, x2, [3, 2], "sqc")
    assert (orc.dequant_f64(codes, scales, zeros)[:, [5, 200]] == 0).all()


def test_repeatable_and_lower_output_error():
    slim = _slim()
    W, x = _layer(256, 1024, 512, name="gptq-gpu-loss")
    bits = [2, 1, 3, 2, 3, 2, 1, 2]
    Wd, xd = torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda()
    a = slim.gptq_quantize(Wd, xd, bits, 0.01, "sqc")
    b = slim.gptq_quantize(Wd, xd, bits, 0.01, "sqc")
    for u, v in zip(a, b):
        assert torch.equal(u, v)
    with_c = orc.gptq_proxy_loss(W, orc.dequant_f64(*[t.cpu().numpy() for t in a]), x)
    plain = slim.quantize_sqc(Wd, bits)[:3]
    without = orc.gptq_proxy_loss(W, orc.dequant_f64(*[t.cpu().numpy() for t in plain]), x)
    assert with_c < 0.8 * without


def test_llama7b_layer_full_size_on_sampled_rows():
    """4096 x 4096 with 1024 calibration tokens, as the benchmark runs it.  Given the factor, the rows of the weight are
    independent problems: the oracle computes a sample of rows."""
    slim = _slim()
    N = K = 4096
    seed = wl.layer_seed("llama-7b", "q_proj", 0)
    W = wl.make_weight(seed, N, K)
    x = wl.make_calibration_x(seed, 1024, K)
    bits = orc.allocate_bits(orc.group_salience(W, wl.make_act_norms(seed, K)), 2)
    codes, scales, zeros = slim.gptq_quantize(torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda(), bits, 0.01, "minmax")
    rows = np.unique(np.concatenate([[0, 1, 15, 16, 4095], np.random.default_rng(7).integers(0, N, 27)]))
    c_ref, s_ref, z_ref, _ = orc.gptq_quantize(W[rows], x, bits, 0.01, "minmax")
    assert (scales.cpu().numpy()[:, rows].view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.cpu().numpy()[:, rows].view(np.uint16) == z_ref.view(np.uint16)).all()
    got = codes.cpu().numpy()[rows]
    assert (got == c_ref).all(), f"{(got != c_ref).sum()} codes differ"


def test_llama7b_down_projection_shape_on_sampled_rows():
    """4096 x 11008 (172 blocks of 64 columns: ragged segments at several levels of the doubling inverse), SQC."""
    slim = _slim()
    N, K = 4096, 11008
    seed = wl.layer_seed("llama-7b", "down_proj", 0)
    W = wl.make_weight(seed, N, K)
    x = wl.make_calibration_x(seed, 1024, K)
    bits = orc.allocate_bits(orc.group_salience(W, wl.make_act_norms(seed, K)), 2)
    codes, scales, zeros = slim.gptq_quantize(torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda(), bits, 0.01, "sqc")
    rows = np.array([0, 17, 2049, 4095])
    c_ref, s_ref, z_ref, _ = orc.gptq_quantize(W[rows], x, bits, 0.01, "sqc")
    assert (scales.cpu().numpy()[:, rows].view(np.uint16) == s_ref.view(np.uint16)).all()
    assert (zeros.cpu().numpy()[:, rows].view(np.uint16) == z_ref.view(np.uint16)).all()
    got = codes.cpu().numpy()[rows]
    assert (got == c_ref).all(), f"{(got != c_ref).sum()} codes differ"


def test_rejects_bad_arguments():
    slim = _slim()
    W, x = _layer(16, 256, 32)
    Wd, xd = torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda()
    with pytest.raises(slim.SlimError):
        slim.gptq_quantize(Wd, xd, [2, 2], 0.0)                         # the damping must be positive
    with pytest.raises(slim.SlimError):
        slim.gptq_quantize(Wd, xd, [2, 5])                              # bit-width out of range
    with pytest.raises(slim.SlimError):
        slim.gptq_quantize(Wd, xd, [2, 2], workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
