"""Pins for the oracle at the group sizes of the paper's group-size ablation (appendix; g in {32, 64, 128, 256, 512}):
storage format (size, hand-worked bit positions, round trip), quantizer, dequantisation and linear layer."""
import os

import numpy as np
import pytest

from oracle import slim_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pack_positions_group_sizes.txt")
SIZES = (32, 64, 128, 256, 512)


def _positions():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = [v.strip() for v in line.split(";")]
        out.append((f[0], int(f[1]), int(f[2]), int(f[3]), [int(v) for v in f[4].split(",")]) + tuple(int(v) for v in f[5:]))
    return out


@pytest.mark.parametrize("pos", _positions(), ids=lambda p: "%s_n%d_k%d_bit%d" % (p[0], p[5], p[6], p[7]))
def test_one_hot_code_bit_lands_where_the_format_says(pos):
    _, g, N, K, bits, n, k, bit, byte, bit_in_byte = pos
    bits = np.array(bits, dtype=np.uint8)
    codes = np.zeros((N, K), dtype=np.uint8)
    codes[n, k] = 1 << bit
    packed = orc.pack(codes, bits, g)
    assert packed.size == N * g * int(bits.sum()) // 8
    expect = np.zeros(packed.size, dtype=np.uint8)
    expect[byte] = 1 << bit_in_byte
    assert (packed == expect).all()


def _random_codes(rng, N, bits, g):
    return np.concatenate([rng.integers(0, 2**int(b), (N, g), dtype=np.uint8) for b in bits], axis=1)


@pytest.mark.parametrize("g", SIZES)
@pytest.mark.parametrize("bits", [[1, 2, 3, 4], [3, 1, 4, 2, 2, 3, 1, 4]])
def test_size_round_trip_and_no_padding(g, bits):
    rng = np.random.default_rng(g + len(bits))
    bits = np.array(bits, dtype=np.uint8)
    N, K = 32, g * len(bits)
    if K % 128:
        pytest.skip("K is a multiple of 128 in every configuration")
    codes = _random_codes(rng, N, bits, g)
    packed = orc.pack(codes, bits, g)
    assert packed.size == orc.packed_bytes(N, K, bits, g) == N * g * int(bits.sum()) // 8      # = N K avg_bits / 8
    assert (orc.unpack(packed, N, K, bits, g) == codes).all()
    full = np.concatenate([np.full((N, g), 2**int(b) - 1, np.uint8) for b in bits], axis=1)
    assert (orc.pack(full, bits, g) == 0xFF).all()          # every bit of the buffer belongs to exactly one code bit


def test_every_single_bit_is_distinct_on_tiny_layers_of_small_groups():
    for g, K in ((32, 128), (64, 128)):
        for b in (1, 2, 3, 4):
            bits = np.full(K // g, b, dtype=np.uint8)
            seen = set()
            for n in (0, 1, 6, 15):
                for k in range(K):
                    for bit in range(b):
                        codes = np.zeros((16, K), dtype=np.uint8)
                        codes[n, k] = 1 << bit
                        packed = orc.pack(codes, bits, g)
                        nz = np.flatnonzero(packed)
                        assert nz.size == 1 and bin(int(packed[nz[0]])).count("1") == 1
                        key = (int(nz[0]), int(packed[nz[0]]))
                        assert key not in seen
                        seen.add(key)


def test_a_group_of_256_columns_is_two_tiles_of_its_width():
    """For g = 256 the buffer equals the g = 128 buffer of the same codes with every bit-width repeated twice."""
    rng = np.random.default_rng(256)
    bits = np.array([3, 1, 2, 4], dtype=np.uint8)
    codes = _random_codes(rng, 48, bits, 256)
    assert (orc.pack(codes, bits, 256) == orc.pack(codes, np.repeat(bits, 2), 128)).all()
    assert (orc.pack(codes[:, :512], bits[:1], 512) == orc.pack(codes[:, :512], np.repeat(bits[:1], 4), 128)).all()


@pytest.mark.parametrize("g", SIZES)
def test_quantizer_per_group_properties(g):
    """Eq. 1 at group size g: extremes map to the end codes, 0 maps to the zero point, the error stays within half a
    step (plus the fp16 rounding of the step), and every group is quantised on its own."""
    rng = np.random.default_rng(g)
    N, K = 24, 4 * g if g >= 128 else 512
    W = (rng.normal(0, 0.02, (N, K)) * (1 + 9 * (rng.random(K) < 0.02))).astype(np.float16)
    bits = rng.integers(1, 5, K // g).astype(np.uint8)
    codes, scales, zeros = orc.quantize_minmax(W, bits, g)
    assert scales.shape == zeros.shape == (K // g, N)
    What = orc.dequant_f64(codes, scales, zeros, g)
    for j in range(K // g):
        w = W[:, j * g:(j + 1) * g].astype(np.float64)
        s = scales[j].astype(np.float64)
        lo, hi = np.minimum(w.min(axis=1), 0), np.maximum(w.max(axis=1), 0)
        err = np.abs(w - What[:, j * g:(j + 1) * g])
        assert (err <= s[:, None] / 2 + ((hi - lo) * 2.0 ** -11)[:, None] + 1e-12).all()
        assert (codes[:, j * g:(j + 1) * g] <= 2 ** int(bits[j]) - 1).all()
        # the group quantised as a one-group layer gives the same codes, scale and zero point
        c1, s1, z1 = orc.quantize_minmax(W[:, j * g:(j + 1) * g], bits[j:j + 1], g)
        assert (c1 == codes[:, j * g:(j + 1) * g]).all() and (s1[0] == scales[j]).all() and (z1[0] == zeros[j]).all()


@pytest.mark.parametrize("g", SIZES)
def test_linear_layer_against_a_plain_triple_loop_and_one_hot_inputs(g):
    rng = np.random.default_rng(1000 + g)
    N, K, M = 4, 1024, 2
    bits = rng.integers(1, 5, K // g).astype(np.uint8)
    codes = _random_codes(rng, N, bits, g)
    scales = rng.uniform(0.01, 0.1, (K // g, N)).astype(np.float16)
    zeros = rng.integers(0, 2, (K // g, N)).astype(np.float16)
    x = rng.normal(0, 1, (M, K)).astype(np.float16)
    y = orc.linear_f64(x, codes, scales, zeros, g)
    ref = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                j = k // g
                acc += float(x[m, k]) * (float(scales[j, n]) * (float(codes[n, k]) - float(zeros[j, n])))
            ref[m, n] = acc
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    e = np.zeros((1, K), dtype=np.float16)
    e[0, 3 * g // 2 + 5] = 1
    col = orc.linear_f64(e, codes, scales, zeros, g)[0]
    j = (3 * g // 2 + 5) // g
    assert np.array_equal(col, scales[j].astype(np.float64) * (codes[:, 3 * g // 2 + 5] - zeros[j].astype(np.float64)))
    w16 = orc.dequant_f16(codes, scales, zeros, g)
    assert w16.dtype == np.float16 and np.array_equal(w16.astype(np.float64), (scales.astype(np.float32).T.repeat(g, axis=1) * (codes.astype(np.float32) - zeros.astype(np.float32).T.repeat(g, axis=1))).astype(np.float16).astype(np.float64))


@pytest.mark.parametrize("g", SIZES)
def test_salience_and_bit_budget(g):
    rng = np.random.default_rng(7 + g)
    N, K = 16, 16 * g if g <= 128 else 8 * g
    W = rng.normal(0, 0.02, (N, K)).astype(np.float16)
    a = np.exp(rng.normal(0, 1, K)).astype(np.float32)
    S = orc.group_salience(W, a, g)
    assert S.shape == (K // g,)
    k0 = 2 * g
    manual = sum(float(a[k]) ** 2 * float((W[:, k].astype(np.float64) ** 2).sum()) for k in range(k0, k0 + g))
    assert np.isclose(S[2], manual, rtol=1e-12)
    bits = orc.allocate_bits(S, 2)
    assert int(bits.astype(np.int64).sum()) * g == 2 * K          # the average-bit budget holds exactly


@pytest.mark.parametrize("g", (32, 64, 256))
def test_sqc_against_the_scalar_restatement_at_other_group_sizes(g):
    """Function SQC of Algorithm 2 at group size g: the 3-sigma mask, the tau grid and the two-term loss are taken
    per (row, group of g columns); a scalar restatement of the algorithm must pick the same tau, step, zero point
    and codes."""
    from tests.test_oracle_sqc import _brute_sqc_row
    rng = np.random.default_rng(300 + g)
    N, K = 2, 2 * g
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    W[0, 3] = np.float16(0.25)                       # an outlier for the mask
    W[1, g:] = -np.abs(W[1, g:])                     # an all-negative group
    bits = np.array([2, 3], np.uint8)
    codes, scales, zeros, ti, loss, loss_s = orc.quantize_sqc(W, bits, g, lam=0.1, n=10)
    for r in range(N):
        for j in range(2):
            w = [float(v) for v in W[r, g * j:g * (j + 1)]]
            L, i, delta, z, q, Ls = _brute_sqc_row(w, int(bits[j]), lam=0.1, n=10)
            assert ti[j, r] == i and float(scales[j, r]) == delta and float(zeros[j, r]) == z
            assert list(codes[r, g * j:g * (j + 1)]) == q
            assert loss[j, r] == L and loss_s[j, r] == Ls


@pytest.mark.parametrize("g", SIZES)
def test_sign_alpha_one_bit_groups_at_every_group_size(g):
    """Eq. 2 per group of g columns: codes are the signs, s (q - z) = +- mean |w| of the group."""
    rng = np.random.default_rng(500 + g)
    N, K = 4, 3 * g
    W = rng.normal(0, 0.02, (N, K)).astype(np.float16)
    bits = np.array([1, 2, 1], np.uint8)
    codes, scales, zeros = orc.quantize_minmax_sign1(W, bits, g)
    c2, s2, z2 = orc.quantize_minmax(W, bits, g)
    assert (codes[:, g:2 * g] == c2[:, g:2 * g]).all() and (scales[1] == s2[1]).all()      # the 2-bit group is Eq. 1
    for j in (0, 2):
        w = W[:, g * j:g * (j + 1)].astype(np.float64)
        assert ((codes[:, g * j:g * (j + 1)] == 1) == (w >= 0)).all()
        alpha = np.abs(w).mean(axis=1)
        assert (zeros[j] == np.float16(0.5)).all()
        assert np.array_equal(scales[j], (2 * alpha).astype(np.float16))
