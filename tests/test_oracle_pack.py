"""Pins for the oracle's storage format: size, hand-worked positions, round trip, C twin."""
import os

import numpy as np
import pytest

from oracle import slim_oracle as orc
from oracle import slim_oracle_c as orc_c

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pack_positions.txt")


def _positions():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        out.append(tuple(int(v) for v in line.split(";")))
    return out


@pytest.mark.parametrize("impl", ["numpy", "c"])
@pytest.mark.parametrize("pos", _positions(), ids=lambda p: "n%d_k%d_bit%d" % p[:3])
def test_one_hot_code_bit_lands_where_the_format_says(impl, pos):
    n, k, bit, byte, bit_in_byte = pos
    N, K, bits = 32, 256, np.array([3, 1], dtype=np.uint8)
    codes = np.zeros((N, K), dtype=np.uint8)
    codes[n, k] = 1 << bit
    packed = orc.pack(codes, bits) if impl == "numpy" else orc_c.pack(codes, bits)
    assert packed.size == 2048
    expect = np.zeros(2048, dtype=np.uint8)
    expect[byte] = 1 << bit_in_byte
    assert (packed == expect).all()


@pytest.mark.parametrize("N,K,avg", [(16, 128, 2), (48, 512, 2), (32, 1024, 3), (4096, 4096, 2)])
def test_size_is_n_k_avgbits_over_8_no_padding(N, K, avg):
    bits = orc.allocate_bits(np.random.default_rng(1).random(K // 128), avg) if K >= 512 else np.full(K // 128, avg, np.uint8)
    assert orc.packed_bytes(N, K, bits) == N * K * avg // 8
    assert orc_c.packed_bytes(N, K, bits) == N * K * avg // 8


def _random_codes(rng, N, bits):
    return np.concatenate([rng.integers(0, 2**int(b), (N, 128), dtype=np.uint8) for b in bits], axis=1)


@pytest.mark.parametrize("bits", [[1], [2], [3], [4], [1, 2, 3, 4], [3, 3, 1, 2, 4, 1], [4, 2, 3]])
def test_round_trip_and_twins_agree(bits):
    rng = np.random.default_rng(sum(bits) * 31 + len(bits))
    bits = np.array(bits, dtype=np.uint8)
    N, K = 48, 128 * len(bits)
    codes = _random_codes(rng, N, bits)
    p_np = orc.pack(codes, bits)
    p_c = orc_c.pack(codes, bits)
    assert (p_np == p_c).all()
    assert (orc.unpack(p_np, N, K, bits) == codes).all()
    assert (orc_c.unpack(p_np, N, K, bits) == codes).all()
    # all-ones codes fill every bit: the format has no padding and no overlap
    full = np.concatenate([np.full((N, 128), 2**int(b) - 1, np.uint8) for b in bits], axis=1)
    assert (orc.pack(full, bits) == 0xFF).all()


def test_every_single_bit_is_distinct_on_a_tiny_layer():
    """Brute force on K = 128, N = 16: each (n, k, bit) sets exactly one bit, all different."""
    for b in (1, 2, 3, 4):
        bits = np.array([b], dtype=np.uint8)
        seen = set()
        for n in range(16):
            for k in range(0, 128, 5):
                for bit in range(b):
                    codes = np.zeros((16, 128), dtype=np.uint8)
                    codes[n, k] = 1 << bit
                    packed = orc_c.pack(codes, bits)
                    nz = np.flatnonzero(packed)
                    assert nz.size == 1 and bin(int(packed[nz[0]])).count("1") == 1
                    key = (int(nz[0]), int(packed[nz[0]]))
                    assert key not in seen
                    seen.add(key)


def test_out_of_range_code_is_rejected():
    codes = np.full((16, 128), 2, dtype=np.uint8)
    with pytest.raises(AssertionError):
        orc.pack(codes, np.array([1], dtype=np.uint8))
    with pytest.raises(ValueError):
        orc_c.pack(codes, np.array([1], dtype=np.uint8))
