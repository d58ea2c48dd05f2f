"""CPU-only checks of the C-ABI library: it builds, loads, exports every declared symbol, and its
host-side logic (argument validation, sizes, bit allocation, launch plans) behaves as declared.
No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def slim():
    cuda_build.build()
    from paper_2405_14917_b200 import binding
    binding.lib()
    return binding


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "slim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slim_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(slim):
    names = _declared_symbols()
    assert {"slim_pack_weights", "slim_dequant", "slim_mpq_gemv", "slim_mpq_gemm"} <= set(names)
    L = ctypes.CDLL(cuda_build.LIB_PATH)
    for n in names:
        assert hasattr(L, n), f"{n} is declared in slim.h but not exported"


def test_version_and_status_strings(slim):
    assert slim.version() >> 16 == 2
    L = slim.lib()
    for code in range(0, -8, -1):
        assert L.slim_status_string(code).decode() not in ("", "unknown status")
    assert L.slim_status_string(-99).decode() == "unknown status"


def test_packed_bytes_is_unpadded(slim):
    """N*K*avg_bits/8 exactly: groups are stored back to back (App. B.2)."""
    for N, K, avg in [(4096, 4096, 2), (11008, 4096, 3), (4096, 11008, 2), (16, 128, 3)]:
        G = K // 128
        p = G // 4
        bits = np.full(G, avg, np.uint8)
        bits[:p] = avg + 1
        bits[G - p:] = avg - 1
        assert slim.packed_bytes(N, K, bits) == N * K * avg // 8 == orc.packed_bytes(N, K, bits)


def test_shape_and_argument_errors(slim):
    bits = np.array([2, 2], np.uint8)
    out = ctypes.c_size_t(0)
    L = slim.lib()
    bp = bits.ctypes.data_as(ctypes.c_void_p)
    assert L.slim_packed_bytes(16, 256, 96, bp, ctypes.byref(out)) == -2      # g not in {32, 64, 128, 256, 512}
    assert L.slim_packed_bytes(16, 256, 1024, bp, ctypes.byref(out)) == -2
    b4 = np.array([2, 3, 1, 2], np.uint8)
    assert L.slim_packed_bytes(16, 256, 64, b4.ctypes.data_as(ctypes.c_void_p), ctypes.byref(out)) == 0 and out.value == 16 * 64 * 8 // 8
    assert L.slim_packed_bytes(16, 256, 256, bp, ctypes.byref(out)) == 0 and out.value == 16 * 256 * 2 // 8
    assert L.slim_packed_bytes(16, 256, 512, bp, ctypes.byref(out)) == -2     # K % g
    assert L.slim_packed_bytes(16, 200, 128, bp, ctypes.byref(out)) == -2     # K % 128
    assert L.slim_packed_bytes(24, 256, 128, bp, ctypes.byref(out)) == -2     # N % 16
    assert L.slim_packed_bytes(16, 256, 128, None, ctypes.byref(out)) == -1   # no bit map
    bad = np.array([2, 5], np.uint8)
    assert L.slim_packed_bytes(16, 256, 128, bad.ctypes.data_as(ctypes.c_void_p), ctypes.byref(out)) == -1
    big = np.full(257, 2, np.uint8)
    assert L.slim_packed_bytes(16, 257 * 128, 128, big.ctypes.data_as(ctypes.c_void_p), ctypes.byref(out)) == -2
    # the linear entry points validate before touching the device: null pointers and M ranges
    assert L.slim_mpq_gemv(None, None, bp, None, None, None, 17, 16, 256, 128, None, 0, None) == -1
    assert L.slim_mpq_gemm(None, None, bp, None, None, None, 16, 16, 256, 128, None, 0, None) == -1
    assert L.slim_mpq_gemv(None, None, bp, None, None, None, 1, 16, 256, 128, None, 0, None) == -1   # y missing
    assert L.slim_mpq_gemv(None, None, bp, None, None, None, 0, 16, 256, 128, None, 0, None) == 0    # M = 0: no-op


def test_allocate_bits_matches_oracle_and_budget(slim):
    rng = np.random.default_rng(11)
    for G in (4, 32, 86, 108, 224):
        for avg in (2, 3):
            S = rng.lognormal(size=G)
            b = slim.allocate_bits(S, avg)
            assert (b == orc.allocate_bits(S, avg)).all()
            assert int(b.astype(int).sum()) == avg * G                       # the average-bit budget is exact
            assert (b == avg + 1).sum() == (b == avg - 1).sum() == G // 4
            T = rng.integers(0, 4, G).astype(np.float64)                     # ties: lower index ranks higher
            assert (slim.allocate_bits(T, avg) == orc.allocate_bits(T, avg)).all()


def test_gemv_plan_invariants(slim):
    rng = np.random.default_rng(3)
    for (N, K, avg, M) in [(4096, 4096, 2, 1), (11008, 4096, 2, 1), (4096, 11008, 2, 1), (1024, 8192, 2, 16),
                           (28672, 8192, 2, 1), (8192, 28672, 2, 16), (16, 128, 2, 1), (272, 1408, 3, 9), (4096, 32768, 3, 16)]:
        G = K // 128
        bits = np.full(G, avg, np.uint8)
        bits[: G // 4] = avg + 1
        bits[G - G // 4:] = avg - 1
        rng.shuffle(bits)
        pl = slim.gemv_plan(M, N, K, bits)
        assert pl["tiles_per_cta"] in (1, 2, 4, 8)
        assert 1 <= pl["k_slices"] <= min(8, G)
        assert pl["row_blocks"] * pl["tiles_per_cta"] >= N // 16
        assert pl["smem_bytes"] <= 227 * 1024
        assert pl["n_tiles"] == (1 if M <= 8 else 2)
        assert 1 <= pl["groups_per_chunk"] <= G


def _set_bytes(slim, shapes, g=128):
    """shapes: list of (M, N, K, bits).  Returns (status, plan_bytes, workspace_bytes)."""
    arr = (slim._Layer * max(len(shapes), 1))()
    keep = []
    for k, (M, N, K, bits) in enumerate(shapes):
        b = np.asarray(bits, dtype=np.uint8)
        keep.append(b)
        arr[k] = slim._Layer(0, 0, 0, 0, 0, b.ctypes.data, M, N, K)
    pb, wb = ctypes.c_size_t(0), ctypes.c_size_t(0)
    st = slim.lib().slim_gemv_set_bytes(ctypes.cast(arr, ctypes.c_void_p), len(shapes), g, ctypes.byref(pb), ctypes.byref(wb))
    return st, pb.value, wb.value


def test_layer_set_sizes_and_argument_errors(slim):
    ok = [(1, 256, 512, [2, 3, 1, 2]), (4, 144, 256, [3, 3])]
    st, pb, wb = _set_bytes(slim, ok)
    assert st == 0
    # plan: item ranges of the CTAs, one descriptor per layer, one entry per work item
    st2, pb2, _ = _set_bytes(slim, ok + [(1, 128, 128, [2])])
    assert st2 == 0 and pb2 > pb and (pb2 - pb) % 16 == 0
    # workspace: status header + per layer the sums [G][16] float2 and the fragments of every slice; the set has a
    # layer with more than one token, so every layer is staged eight tokens wide (absent tokens as zeros)
    want = 256 + (4 * 128 + (4 + 1) * 8 * 8 * 32) + (2 * 128 + (2 + 2) * 8 * 8 * 32)
    assert wb == want
    assert _set_bytes(slim, [(1, 256, 512, [2, 3, 1, 2])])[2] == 256 + (4 * 128 + (4 + 1) * 512)              # one token: 8-bit digit form
    assert _set_bytes(slim, [(9, 256, 512, [2, 3, 1, 2])])[2] == 256 + (4 * 128 + (4 + 1) * 8 * 16 * 32)     # sixteen wide
    assert _set_bytes(slim, [])[0] == -1                                  # empty set
    assert _set_bytes(slim, [(0, 256, 512, [2] * 4)])[0] == -1            # no token
    assert _set_bytes(slim, [(40, 256, 512, [2, 3, 1, 2])])[2] == 256 + (4 * 512 + (4 + 1) * 256 * 64)        # 64 wide: 8 bytes of sums per token
    assert _set_bytes(slim, [(65, 256, 512, [2] * 4)])[0] == -1           # more than 64 tokens: the batched path
    assert _set_bytes(slim, [(1, 256, 512, [2, 5, 2, 2])])[0] == -1       # bit-width out of range
    assert _set_bytes(slim, [(1, 250, 512, [2] * 4)])[0] == -2            # N not a multiple of 16
    assert _set_bytes(slim, [(1, 256, 500, [2] * 4)])[0] == -2            # K not a multiple of 128
    assert _set_bytes(slim, [(1, 256, 0, [])])[0] == -1                   # empty reduction
    assert _set_bytes(slim, ok, g=64)[0] == -2                            # group size


def test_sba_workspace_and_quantizer_argument_errors(slim):
    L = slim.lib()
    out = ctypes.c_size_t(0)
    assert L.slim_sba_workspace_bytes(128, 4096, 4096, 128, 2, ctypes.byref(out)) == 0
    # codes + scales + zeros + widest packed buffer + both outputs + one error per candidate and token, at least
    G = 32
    least = 4096 * 4096 + 2 * (G * 4096 * 2) + 4096 * 4096 * 3 // 8 + 128 * 4096 * (4 + 2) + (G // 2 + 1) * 128 * 8
    assert least <= out.value <= least + 32 * 1024 * 1024
    assert L.slim_sba_workspace_bytes(128, 4096, 4096, 128, 4, ctypes.byref(out)) == -1      # average bit-width
    assert L.slim_sba_workspace_bytes(0, 4096, 4096, 128, 2, ctypes.byref(out)) == -1        # no calibration token
    assert L.slim_sba_workspace_bytes(128, 4096, 4000, 128, 2, ctypes.byref(out)) == -2      # K not a multiple of 128
    assert L.slim_sba_workspace_bytes(128, 4096, 4096, 96, 2, ctypes.byref(out)) == -2       # group size
    assert L.slim_sba_workspace_bytes(128, 4096, 4096, 64, 2, ctypes.byref(out)) == 0
    assert L.slim_sba_workspace_bytes(128, 4096, 4096, 128, 2, None) == -1
    # nothing is launched for null pointers
    bits = np.array([2, 2], dtype=np.uint8)
    groups = np.array([0], dtype=np.int32)
    assert L.slim_quantize_minmax_groups(None, bits.ctypes.data, None, None, None, 16, 256, 128, groups.ctypes.data, 1, None) == -1
    assert L.slim_quantize_minmax_sign1(None, bits.ctypes.data, None, None, None, 16, 256, 128, None) == -1
    assert L.slim_dense_linear(None, None, None, 4, 16, 128, None) == -1
    assert L.slim_dense_linear(None, None, None, 0, 16, 128, None) == 0
    assert L.slim_softmax_kl(None, None, None, 4, 16, None) == -1


def test_gptq_workspace_and_argument_errors(slim):
    def ws_bytes(T, N, K, g=128):
        out = ctypes.c_size_t(0)
        return slim.lib().slim_gptq_workspace_bytes(T, N, K, g, ctypes.byref(out)), out.value

    st, b = ws_bytes(64, 256, 512)
    # dead flags, two K x K fp64 matrices, the fp64 running weights, one group of errors (fp64), of quantizer input
    # (fp16) and of codes, each rounded up to 256 bytes
    assert st == 0 and b == 512 + 2 * 512 * 512 * 8 + 256 * 512 * 8 + 256 * 128 * (8 + 2 + 1)
    assert ws_bytes(64, 0, 512)[1] == 512 + 2 * 512 * 512 * 8            # the factor alone
    assert ws_bytes(0, 256, 512)[0] == -1                                 # no calibration token
    assert ws_bytes(64, 256, 500)[0] == -2                                # K not a multiple of 128
    assert ws_bytes(64, 256, 512, g=96)[0] == -2                          # group size
    st64, b64 = ws_bytes(64, 256, 512, g=64)                              # the per-group buffers follow the group size
    assert st64 == 0 and b64 == b - 256 * 64 * (8 + 2 + 1)
    bits = np.array([2, 2, 2, 2], dtype=np.uint8)
    L = slim.lib()
    args = lambda lam, wsb: (256, 256, bits.ctypes.data, ctypes.c_double(lam), 1, 256, 256, 256, None, 256, 512, 64, 128, 256, wsb, None)
    assert L.slim_gptq_quantize(*args(0.0, b)) == -1                      # the damping must be positive
    assert L.slim_gptq_quantize(*args(0.01, b - 1)) == -4                 # workspace too small
    assert L.slim_gptq_factor(256, 64, 512, ctypes.c_double(0.01), None, None, 256, b, None) == -1   # no output

