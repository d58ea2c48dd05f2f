"""Pins for the oracle's Eq. 1 quantizer: hand-worked cases, brute force, bounds."""
import os

import numpy as np
import pytest

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "eq1_hand_cases.txt")


def _cases():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, b, ws, s, z, qs = [f.strip() for f in line.split(";")]
        out.append((name, int(b), [float(v) for v in ws.split()], float(s), float(z), [int(v) for v in qs.split()]))
    return out


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c[0])
def test_hand_worked_cases(case):
    name, b, ws, s, z, qs = case
    row = np.array([ws[i % len(ws)] for i in range(128)], dtype=np.float16)
    W = np.stack([row, row[::-1]])  # column order must not matter
    codes, scales, zeros = orc.quantize_minmax(W, np.array([b], dtype=np.uint8))
    assert scales.dtype == np.float16 and zeros.dtype == np.float16
    assert float(scales[0, 0]) == s and float(zeros[0, 0]) == z
    assert not np.signbit(zeros).any()   # the zero point is an unsigned integer: never -0
    assert float(scales[0, 1]) == s and float(zeros[0, 1]) == z
    assert codes[0].tolist() == [qs[i % len(ws)] for i in range(128)]
    assert codes[1].tolist() == codes[0].tolist()[::-1]


@pytest.mark.parametrize("b", [1, 2, 3, 4])
def test_brute_force_every_code_is_the_nearest_level(b):
    """K = 128, N = 4: the code chosen for each weight must be a nearest level among all 2^b codes."""
    rng = np.random.default_rng(100 + b)
    W = (rng.standard_normal((4, 128)) * 0.02).astype(np.float16)
    W[1] = np.abs(W[1])            # all-positive row
    W[2] = -np.abs(W[2])           # all-negative row
    W[3, ::7] *= 10                # outliers
    codes, scales, zeros = orc.quantize_minmax(W, np.array([b], dtype=np.uint8))
    levels = 2**b
    for n in range(4):
        s, z = float(scales[0, n]), float(zeros[0, n])
        assert 0 <= z <= levels - 1 and z == int(z)
        recon = [s * (q - z) for q in range(levels)]
        for k in range(128):
            w = float(W[n, k])
            errs = [abs(w - r) for r in recon]
            assert errs[int(codes[n, k])] <= min(errs) * (1 + 1e-12) + 1e-300
        # extremes hit the end codes, zero maps to the zero point (and dequantises to exactly 0)
        lo, hi = min(W[n].min(), 0), max(W[n].max(), 0)
        wn = W[n].astype(np.float64)
        if lo < 0:
            assert codes[n, int(np.argmin(wn))] == 0
        if hi > 0:
            assert codes[n, int(np.argmax(wn))] == levels - 1


@pytest.mark.parametrize("avg", [2, 3])
def test_error_bound_and_range(avg):
    rng = np.random.default_rng(5)
    N, K = 16, 1024
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    bits = orc.allocate_bits(rng.random(K // 128), avg)
    codes, scales, zeros = orc.quantize_minmax(W, bits)
    What = orc.dequant_f64(codes, scales, zeros)
    Wd = W.astype(np.float64)
    for j, b in enumerate(bits):
        sl = slice(128 * j, 128 * j + 128)
        assert codes[:, sl].max() <= 2**int(b) - 1
        s = scales[j].astype(np.float64)[:, None]
        span = (np.maximum(Wd[:, sl].max(1), 0) - np.minimum(Wd[:, sl].min(1), 0))[:, None]
        # |w - w_hat| <= s/2, plus what the fp16 rounding of s can cost at the clamped extremes
        assert (np.abs(Wd[:, sl] - What[:, sl]) <= s / 2 + span * 2.0**-10).all()
    # w = 0 is represented exactly (zero point): a zero weight dequantises to 0
    Wz = W.copy()
    Wz[:, ::5] = 0
    c2, s2, z2 = orc.quantize_minmax(Wz, bits)
    assert (orc.dequant_f64(c2, s2, z2)[:, ::5] == 0).all()


def test_monotone_and_idempotent():
    rng = np.random.default_rng(9)
    W = (rng.standard_normal((8, 256)) * 0.05).astype(np.float16)
    bits = np.array([2, 3], dtype=np.uint8)
    codes, scales, zeros = orc.quantize_minmax(W, bits)
    for n in range(8):
        for j in range(2):
            sl = slice(128 * j, 128 * j + 128)
            order = np.argsort(W[n, sl].astype(np.float64), kind="stable")
            assert (np.diff(codes[n, sl][order].astype(int)) >= 0).all()
    # quantising the fp16 dequantised weights with the same grid reproduces the codes
    W2 = orc.dequant_f16(codes, scales, zeros)
    What2 = orc.dequant_f64(*orc.quantize_minmax(W2, bits))
    assert np.abs(What2 - W2.astype(np.float64)).max() <= np.abs(W2.astype(np.float64)).max() * 2.0**-9


def test_all_equal_bit_map_is_uniform_group_quantisation():
    """p = 0 (uniform precision, App. C): quantising group by group with one width equals
    quantising each 128-column block as its own single-group layer."""
    rng = np.random.default_rng(21)
    W = (rng.standard_normal((4, 512)) * 0.02).astype(np.float16)
    for b in (2, 3):
        bits = np.full(4, b, dtype=np.uint8)
        codes, scales, zeros = orc.quantize_minmax(W, bits)
        for j in range(4):
            cj, sj, zj = orc.quantize_minmax(W[:, 128 * j:128 * j + 128], bits[:1])
            assert (cj == codes[:, 128 * j:128 * j + 128]).all()
            assert (sj[0] == scales[j]).all() and (zj[0] == zeros[j]).all()
    # and a mixed map only changes the groups whose width changed
    mixed = np.array([2, 3, 2, 1], dtype=np.uint8)
    cm, sm, zm = orc.quantize_minmax(W, mixed)
    cu, su, zu = orc.quantize_minmax(W, np.full(4, 2, dtype=np.uint8))
    for j in (0, 2):
        assert (cm[:, 128 * j:128 * j + 128] == cu[:, 128 * j:128 * j + 128]).all()
        assert (sm[j] == su[j]).all()


def test_sign_alpha_binarisation_eq2():
    W = np.zeros((2, 128), dtype=np.float16)
    W[0, :64], W[0, 64:] = 0.5, -0.25        # alpha = 0.375
    W[1, :] = -1.0
    W[1, 0] = 0.0                              # sign(0) = +1
    codes, scales, zeros = orc.quantize_sign_alpha_1bit(W)
    What = orc.dequant_f64(codes, scales, zeros)
    assert (What[0, :64] == 0.375).all() and (What[0, 64:] == -0.375).all()
    a1 = 127.0 / 128.0
    assert What[1, 0] == pytest.approx(a1, rel=2**-11) and What[1, 0] > 0
    assert (What[1, 1:] < 0).all()


def test_mixed_quantizer_takes_eq2_only_for_one_bit_groups():
    seed = wl.layer_seed("test", "sign1", 0)
    W = wl.make_weight(seed, 24, 768)
    bits = np.array([1, 2, 3, 1, 2, 1], dtype=np.uint8)
    codes, scales, zeros = orc.quantize_minmax_sign1(W, bits)
    c0, s0, z0 = orc.quantize_minmax(W, bits)
    c1, s1, z1 = orc.quantize_sign_alpha_1bit(W)
    for j, b in enumerate(bits):
        cols = slice(128 * j, 128 * j + 128)
        src = (c1, s1, z1) if b == 1 else (c0, s0, z0)
        assert (codes[:, cols] == src[0][:, cols]).all() and (scales[j] == src[1][j]).all() and (zeros[j] == src[2][j]).all()
    # Eq. 2: the dequantised one-bit groups are +-alpha with alpha = mean |w| (rounded once to fp16 as 2 alpha)
    What = orc.dequant_f64(codes, scales, zeros)
    w = W.astype(np.float64)
    for j in np.nonzero(bits == 1)[0]:
        cols = slice(128 * j, 128 * j + 128)
        alpha = np.float16(2 * np.abs(w[:, cols]).mean(axis=1)).astype(np.float64) / 2
        assert (What[:, cols] == np.where(w[:, cols] >= 0, alpha[:, None], -alpha[:, None])).all()
