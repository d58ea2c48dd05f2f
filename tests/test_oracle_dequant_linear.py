"""Pins for the oracle's dequantisation (closed form, single rounding) and the fp64 linear layer."""
import os

import numpy as np
import pytest

from oracle import slim_oracle as orc
from oracle import slim_oracle_c as orc_c
from paper_2405_14917_b200 import workloads as wl


def _all_finite_f16():
    u = np.arange(0x7C00, dtype=np.uint16)
    return np.concatenate([u, u | 0x8000]).view(np.float16)


@pytest.mark.parametrize("zeros_kind", ["integer", "half"])
def test_dequant_f16_is_the_single_rounding_of_the_exact_product(zeros_kind):
    """Exhaustive: every finite fp16 scale x every code 0..15 x every zero point.

    s has an 11-bit significand and |q - z| <= 15.5 needs 5 bits, so s (q - z) is exact in fp64;
    rounding that once to fp16 is the definition the fp32 recipe must reproduce."""
    s_all = _all_finite_f16()
    G = s_all.size // 16 + 1
    for z in (range(16) if zeros_kind == "integer" else [0.5, 3.5, 7.5]):
        # layer with N = 16 rows, one group per block of 16 scales; codes 0..15 repeated along k
        n_groups = (s_all.size + 15) // 16
        s_pad = np.concatenate([s_all, np.ones(n_groups * 16 - s_all.size, np.float16)]).reshape(n_groups, 16)
        scales = s_pad
        zeros = np.full_like(scales, z)
        codes = np.tile(np.arange(128, dtype=np.uint8) % 16, (16, n_groups))
        got = orc.dequant_f16(codes, scales, zeros)
        exact = np.repeat(scales.T.astype(np.float64), 128, axis=1) * (codes.astype(np.float64) - float(z))
        with np.errstate(over="ignore"):
            want = exact.astype(np.float16)
        assert (got.view(np.uint16) == want.view(np.uint16)).all()
        if z in (0, 7, 3.5):
            assert (orc_c.dequant_f16(codes[:, :128 * 64], scales[:64], zeros[:64]).view(np.uint16)
                    == want[:, :128 * 64].view(np.uint16)).all()


def test_dequant_closed_form_on_hand_values():
    # w_hat = s (q - z): s = 0.25, z = 3 -> q = 0..7 gives -0.75 .. 1.0
    codes = np.tile(np.arange(128, dtype=np.uint8) % 8, (16, 1))
    scales = np.full((1, 16), 0.25, np.float16)
    zeros = np.full((1, 16), 3, np.float16)
    want = (np.arange(128) % 8 - 3) * 0.25
    assert (orc.dequant_f64(codes, scales, zeros) == want).all()
    assert (orc.dequant_f16(codes, scales, zeros).astype(np.float64) == want).all()
    # scales and zeros are indexed [group][row]: change one row of one group only
    codes2 = np.tile(codes, (1, 2))
    scales2 = np.full((2, 16), 0.25, np.float16)
    zeros2 = np.full((2, 16), 3, np.float16)
    scales2[1, 5] = 2.0
    zeros2[1, 5] = 1.0
    W = orc.dequant_f64(codes2, scales2, zeros2)
    assert (W[:, :128] == want).all() and (np.delete(W[:, 128:], 5, axis=0) == want).all()
    assert (W[5, 128:] == (np.arange(128) % 8 - 1) * 2.0).all()


def _small_layer(seed=3, N=32, K=512, M=3, avg=2):
    s = wl.layer_seed("unit", "t", seed)
    W = wl.make_weight(s, N, K)
    a = wl.make_act_norms(s, K)
    x = wl.make_x(s, M, K)
    bits, codes, scales, zeros = orc.make_layer(W, a, avg)
    return x, bits, codes, scales, zeros


def test_linear_special_inputs():
    x, bits, codes, scales, zeros = _small_layer()
    M, K = x.shape
    What = orc.dequant_f64(codes, scales, zeros)
    # one-hot x selects a column of W-hat
    for k in (0, 127, 128, 300, K - 1):
        e = np.zeros((1, K), dtype=np.float16)
        e[0, k] = 1.0
        assert (orc.linear_f64(e, codes, scales, zeros)[0] == What[:, k]).all()
    assert (orc.linear_f64(np.zeros((2, K), np.float16), codes, scales, zeros) == 0).all()
    # rows of x are independent; linear in x
    y = orc.linear_f64(x, codes, scales, zeros)
    for m in range(M):
        assert np.allclose(orc.linear_f64(x[m:m + 1], codes, scales, zeros)[0], y[m], rtol=1e-13, atol=1e-300)
    x2 = (x.astype(np.float32) * 2).astype(np.float16)
    assert np.allclose(orc.linear_f64(x2, codes, scales, zeros), 2 * y, rtol=1e-13)


def test_linear_matches_triple_loop_and_c_twin():
    x, bits, codes, scales, zeros = _small_layer(N=16, K=256, M=2)
    y = orc.linear_f64(x, codes, scales, zeros)
    ref = np.zeros_like(y)
    for m in range(2):
        for n in range(16):
            acc = 0.0
            for k in range(256):
                j = k // 128
                acc += float(x[m, k]) * (float(scales[j, n]) * (float(codes[n, k]) - float(zeros[j, n])))
            ref[m, n] = acc
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-15)
    yc, used = orc_c.linear_f64(x, codes, scales, zeros)
    assert used >= 1
    assert np.allclose(yc, ref, rtol=1e-12, atol=1e-15)
    rows = [3, 9, 15]
    assert np.allclose(orc.linear_rows_f64(x, codes, scales, zeros, rows), y[:, rows], rtol=1e-13)


def test_quantised_layer_error_follows_the_uniform_noise_model():
    """The whole chain (Eq. 1 -> s (q - z) -> matmul) against x W^T: for Gaussian weights the relative
    output error of a b-bit uniform quantizer is step / sqrt(12) over the weight rms (textbook noise model).
    A dropped zero point, a transposed scale table or a wrong group index breaks this by far more than 25 %."""
    s = wl.layer_seed("unit", "approx", 0)
    N, K = 64, 1024
    W = wl.make_weight(s, N, K, outlier_frac=0.0)
    x = wl.make_x(s, 4, K)
    Wd = W.astype(np.float64)
    y_fp = x.astype(np.float64) @ Wd.T
    span = Wd.reshape(N, K // 128, 128).max(2) - Wd.reshape(N, K // 128, 128).min(2)
    prev = None
    for b in (2, 3, 4):
        codes, scales, zeros = orc.quantize_minmax(W, np.full(K // 128, b, np.uint8))
        y = orc.linear_f64(x, codes, scales, zeros)
        err = np.linalg.norm(y - y_fp) / np.linalg.norm(y_fp)
        theory = np.sqrt(((span / (2**b - 1)) ** 2 / 12).mean()) / np.sqrt((Wd**2).mean())
        if b >= 3:
            assert 0.75 * theory < err < 1.25 * theory, (b, err, theory)
        assert prev is None or err < 0.6 * prev
        prev = err
    # mixed maps: more bits on average, less error
    a = wl.make_act_norms(s, K)
    e = {}
    for avg in (2, 3):
        bits, codes, scales, zeros = orc.make_layer(W, a, avg)
        e[avg] = np.linalg.norm(orc.linear_f64(x, codes, scales, zeros) - y_fp) / np.linalg.norm(y_fp)
    assert e[3] < e[2] < 1.0


def test_memory_model_matches_paper_weight_memory():
    golden = os.path.join(os.path.dirname(__file__), "golden", "paper_weight_memory.txt")
    vocab = 32000
    for line in open(golden):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        model, avg, wm = [f.strip() for f in line.split(";")]
        avg, wm = int(avg), float(wm)
        total = 0
        hidden = wl.LAYER_SETS[model][0][2]
        for (_, N, K) in wl.LAYER_SETS[model]:
            G = K // 128
            bits = orc.allocate_bits(np.arange(G, dtype=np.float64), avg)
            total += orc.packed_bytes(N, K, bits) + 2 * 2 * G * N
        total = total * wl.N_BLOCKS[model] + 2 * vocab * hidden * 2
        assert abs(total / 1e9 - wm) / wm < 0.06, (model, avg, total / 1e9, wm)
