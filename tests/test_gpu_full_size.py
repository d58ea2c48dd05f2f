"""GPU parity at the full sizes of the workload configurations, in the launch configurations the benchmark
times: every entry point of the hot path against the fp64 oracle on sampled output rows (the oracle computes
a row on its own, so a few hundred rows of a 28672 x 8192 layer take milliseconds).

Covered here: the LLaMA-2-70B shapes (avg 2 bits, M = 1 and 16) through slim_mpq_gemv and through one
layer-set launch that holds all seven projections of a block; the LLaMA-7B shapes at avg 3 bits through the
layer-set launch at M = 1, 4, 8, 16 with more work items than persistent CTAs; the LLaMA-13B shapes at
M = 2048 through slim_mpq_gemm and through the entry point with built-in scratch; and the single-token
fixed-point form of the layer-set launch at the inputs that are worst for it.
"""
import functools

import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from tests.helpers import check_output, oracle_layer

pytestmark = pytest.mark.gpu


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


@functools.lru_cache(maxsize=None)
def _layer(N, K, avg_bits):
    """Oracle-quantised layer of a configuration shape (cached: the 70B layers take seconds to quantise)."""
    L = oracle_layer(N, K, avg_bits, 1, seed_name="full-size")
    L["packed"] = orc.pack(L["codes"], L["bits"])
    return L


@functools.lru_cache(maxsize=None)
def _device_layer(N, K, avg_bits):
    slim = _slim()
    L = _layer(N, K, avg_bits)
    return slim.QuantLinear(torch.from_numpy(L["packed"]).cuda(), L["bits"], torch.from_numpy(L["scales"]).cuda(),
                            torch.from_numpy(L["zeros"]).cuda(), N, K)


def _sample_rows(N, rng, n=200):
    edge = [0, 1, 15, 16, 127, 128, 255, 256, N - 257, N - 256, N - 17, N - 16, N - 1]
    return np.unique(np.concatenate([[r for r in edge if 0 <= r < N], rng.integers(0, N, n)]))


def _x(rng, M, K):
    return rng.normal(0.0, 1.0, (M, K)).astype(np.float16)


LLAMA70B = [("q", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192), ("o", 8192, 8192),
            ("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)]
LLAMA7B = [(4096, 4096), (11008, 4096), (4096, 11008)]


@pytest.mark.parametrize("M", [1, 16])
@pytest.mark.parametrize("N,K", [(8192, 8192), (28672, 8192), (8192, 28672)])
def test_llama70b_shapes_single_layer_entry_point(N, K, M):
    """slim_mpq_gemv on the large LLaMA-2-70B projections (G = 64 and G = 224 groups)."""
    slim = _slim()
    L, dl = _layer(N, K, 2), _device_layer(N, K, 2)
    rng = np.random.default_rng(70 + N + K + M)
    x = _x(rng, M, K)
    ws = slim.new_workspace(M, N, K, L["bits"])
    y = slim.mpq_gemv(torch.from_numpy(x).cuda(), dl.packed, L["bits"], dl.scales, dl.zeros, N, ws)
    slim.workspace_status(ws)
    y = y.cpu().numpy()
    assert np.isfinite(y.astype(np.float64)).all()
    rows = _sample_rows(N, rng)
    check_output(y[:, rows], orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows), f"gemv {N}x{K} M={M}")


@pytest.mark.parametrize("M", [1, 4])
def test_large_layer_takes_the_ring_or_the_per_layer_kernel_by_workspace_size(M):
    """slim_mpq_gemv sends a layer of 32 MB or more through the layer-set kernels when the workspace has room for their
    plan (written by a kernel, so the call can sit in a CUDA graph) and staged activations; with a 256-byte workspace
    the same call takes the per-layer kernel.  Both against the oracle, the routed one also replayed from a graph."""
    slim = _slim()
    N, K = 28672, 8192
    L, dl = _layer(N, K, 2), _device_layer(N, K, 2)
    rng = np.random.default_rng(2800 + M)
    x = _x(rng, M, K)
    xd = torch.from_numpy(x).cuda()
    rows = _sample_rows(N, rng)
    y_ref = orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows)
    big = slim.new_workspace(M, N, K, L["bits"])
    assert big.numel() > 1 << 16                          # room for the plan, the staged x and the partial outputs
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for ws, what in ((big, "through the ring"), (small, "per-layer kernel")):
        y = slim.mpq_gemv(xd, dl.packed, L["bits"], dl.scales, dl.zeros, N, ws)
        slim.workspace_status(ws)
        check_output(y.cpu().numpy()[:, rows], y_ref, f"{what}, M={M}")
    out = torch.empty((M, N), dtype=torch.float16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        slim.mpq_gemv(xd, dl.packed, L["bits"], dl.scales, dl.zeros, N, big, out)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        slim.mpq_gemv(xd, dl.packed, L["bits"], dl.scales, dl.zeros, N, big, out)
    first = out.clone()
    for _ in range(3):
        out.fill_(float("nan"))
        graph.replay()
    torch.cuda.synchronize()
    slim.workspace_status(big)
    assert torch.equal(out, first)
    check_output(out.cpu().numpy()[:, rows], y_ref, f"replayed from a graph, M={M}")


@pytest.mark.parametrize("M", [1, 16])
def test_llama70b_block_as_one_layer_set(M):
    """All seven projections of a LLaMA-2-70B block in one layer-set launch (the benchmark's 70B configuration
    runs eight such blocks): 1024-row to 28672-row layers and 64 to 224 groups side by side."""
    slim = _slim()
    rng = np.random.default_rng(7000 + M)
    entries, meta = [], []
    for rep in range(2):                      # twice, so that the set holds more items than persistent CTAs at M = 16 too
        for name, N, K in LLAMA70B:
            L, dl = _layer(N, K, 2), _device_layer(N, K, 2)
            x = _x(rng, M, K)
            y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
            entries.append((dl, torch.from_numpy(x).cuda(), y))
            meta.append((name, L, x))
    s = slim.LayerSet(entries)
    assert s.info["n_items"] > s.info["grid"]
    s.run()
    s.check()
    for (name, L, x), (_, _, y) in zip(meta, entries):
        y = y.cpu().numpy()
        assert np.isfinite(y.astype(np.float64)).all(), name
        rows = _sample_rows(L["N"], rng, 120)
        check_output(y[:, rows], orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows),
                     f"set, 70B {name} {L['N']}x{L['K']} M={M}")


def test_projections_of_a_block_as_small_single_token_sets():
    """The small sets a decoder issues at one token.  q/k/v (three 4096 x 4096 layers on one x) fit the GPU as one
    wave of resident CTAs and run as a single launch; gate/up (two 11008 x 4096 layers) take two waves of it; six
    11008 x 4096 layers are too many CTAs for that and too few row blocks for the persistent ring as it is, so their
    row blocks are cut into parts, which the last-arriving part adds up."""
    slim = _slim()
    rng = np.random.default_rng(404)
    for shapes, resident in (([(4096, 4096)] * 3, True), ([(11008, 4096)] * 2, True), ([(11008, 4096)] * 6, False)):
        entries, xs = [], []
        for i, (N, K) in enumerate(shapes):
            x = _x(rng, 1, K) if (i == 0 or len(shapes) > 3) else xs[0]          # q/k/v and gate/up share their input
            xs.append(x)
            entries.append((_device_layer(N, K, 2 + (i & 1)), torch.from_numpy(x).cuda(),
                            torch.full((1, N), float("nan"), dtype=torch.float16, device="cuda")))
        s = slim.LayerSet(entries)
        assert (s.info["resident_pairs"] > 0) == resident
        if not resident:
            assert s.info["split"] > 1 and s.info["n_counters"] > 0
        for _ in range(2):                       # twice: the arrival counters start every launch at zero
            for (_, _, y) in entries:
                y.fill_(float("nan"))
            s.run()
            s.check()
            for i, ((N, K), (_, _, y)) in enumerate(zip(shapes, entries)):
                L = _layer(N, K, 2 + (i & 1))
                y = y.cpu().numpy()
                assert np.isfinite(y.astype(np.float64)).all()
                rows = _sample_rows(N, rng, 120)
                check_output(y[:, rows], orc.linear_rows_f64(xs[i], L["codes"], L["scales"], L["zeros"], rows), f"{N}x{K} layer {i}")


@pytest.mark.parametrize("M", [1, 4, 8, 16, 32, 64])
def test_llama7b_avg3_layer_set_all_token_counts(M):
    """LLaMA-7B shapes at avg 3 bits (bit-widths 2, 3, 4) through the layer-set launch, for every token count of
    that configuration and for the 32 and 64 tokens a set also takes: the single-token integer form and the f16 forms
    of one, two, four and eight token tiles, each with more work items than persistent CTAs so that CTAs cross item and
    layer boundaries."""
    slim = _slim()
    rng = np.random.default_rng(300 + M)
    entries, meta = [], []
    for rep in range(12):
        for N, K in LLAMA7B:
            L, dl = _layer(N, K, 3), _device_layer(N, K, 3)
            x = _x(rng, M, K)
            y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
            entries.append((dl, torch.from_numpy(x).cuda(), y))
            meta.append((L, x))
    s = slim.LayerSet(entries)
    assert s.info["max_bits"] == 4 and s.info["max_tokens"] == M
    assert s.info["n_items"] > 2 * s.info["grid"]
    s.run()
    s.check()
    for k, ((L, x), (_, _, y)) in enumerate(zip(meta, entries)):
        y = y.cpu().numpy()
        assert np.isfinite(y.astype(np.float64)).all(), f"entry {k}"
        rows = _sample_rows(L["N"], rng, 60)
        check_output(y[:, rows], orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows),
                     f"set, 7B avg3 entry {k} {L['N']}x{L['K']} M={M}")


@pytest.mark.parametrize("N,K", [(5120, 5120), (13824, 5120)])
def test_llama13b_shapes_batched_m2048(N, K):
    """slim_mpq_gemm and slim_mpq_gemm_static at M = 2048 on the LLaMA-13B attention and gate/up shapes, both
    against the oracle (the down projection at this M is in test_gpu_gemm.py)."""
    slim = _slim()
    M = 2048
    L, dl = _layer(N, K, 3), _device_layer(N, K, 3)
    rng = np.random.default_rng(13 + N + K)
    x = _x(rng, M, K)
    xd = torch.from_numpy(x).cuda()
    rows = _sample_rows(N, rng, 120)
    y_ref = orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows)
    ws = slim.new_workspace(M, N, K, L["bits"])
    y = slim.mpq_gemm(xd, dl.packed, L["bits"], dl.scales, dl.zeros, N, ws)
    slim.workspace_status(ws)
    y = y.cpu().numpy()
    assert np.isfinite(y.astype(np.float64)).all()
    check_output(y[:, rows], y_ref, f"gemm {N}x{K} M={M}")
    out = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    slim.mpq_gemm_static(xd, dl.packed, L["bits"], dl.scales, dl.zeros, N, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_output(out.cpu().numpy()[:, rows], y_ref, f"gemm with built-in scratch {N}x{K} M={M}")


def test_built_in_scratch_entry_point_against_the_oracle_on_a_stream_k_shape():
    """5120 x 13824 at M = 512 is cut across CTAs (stream-K): partial tiles and flags live in the built-in scratch."""
    slim = _slim()
    N, K, M = 5120, 13824, 512
    L, dl = _layer(N, K, 3), _device_layer(N, K, 3)
    rng = np.random.default_rng(99)
    x = _x(rng, M, K)
    out = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    rows = _sample_rows(N, rng, 120)
    y_ref = orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows)
    for call in range(2):
        out.fill_(float("nan"))
        slim.mpq_gemm_static(torch.from_numpy(x).cuda(), dl.packed, L["bits"], dl.scales, dl.zeros, N, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        check_output(out.cpu().numpy()[:, rows], y_ref, f"built-in scratch, call {call}")


# ------------------------------------------------------------------------------------------------------------------
# The single-token layer-set form rounds x, per group of 128, to fixed point relative to the group's largest |x|:
# |X 2^-S - x| <= 2^-22 max|x_group| per element.  Per output row the error is therefore bounded by
#     sum over groups of 2^-22 max|x_group| sum_k |w-hat[n, k]|
# plus the fp16 rounding of y and the fp32 rounding of the running sum.  The inputs below are the ones that come
# closest to that bound.

def _row_bound(L, x):
    What = np.abs(orc.dequant_f64(L["codes"], L["scales"], L["zeros"]))
    xa = np.abs(x.astype(np.float64))[0]
    G = L["K"] // 128
    return sum(2.0 ** -22 * xa[128 * j:128 * j + 128].max() * What[:, 128 * j:128 * j + 128].sum(axis=1) for j in range(G))


ROUTES = ("set", "per-layer")         # the layer-set launch, and slim_mpq_gemv's single-token kernel


def _run_single_token_set(L, x, route="set"):
    slim = _slim()
    dl = slim.QuantLinear(torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda(), L["bits"],
                          torch.from_numpy(L["scales"]).cuda(), torch.from_numpy(L["zeros"]).cuda(), L["N"], L["K"])
    y = torch.full((1, L["N"]), float("nan"), dtype=torch.float16, device="cuda")
    if route == "per-layer":
        ws = slim.new_workspace(1, L["N"], L["K"], L["bits"])
        dl.forward(torch.from_numpy(x).cuda(), ws, out=y)
        slim.workspace_status(ws)
        return y.cpu().numpy()
    s = slim.LayerSet([(dl, torch.from_numpy(x).cuda(), y)])
    assert s.info["max_tokens"] == 1
    s.run()
    s.check()
    return y.cpu().numpy()


def _check_row_bound(y, y_ref, bound, what):
    err = np.abs(y.astype(np.float64) - y_ref)[0]
    slack = 2.0 ** -10 * np.abs(y_ref[0]) + 1e-5 * np.abs(y_ref).max()
    worst = np.max(err - bound - slack)
    assert worst <= 0, f"{what}: a row exceeds the fixed-point bound by {worst:.3e}"


@pytest.mark.parametrize("route", ROUTES)
@pytest.mark.parametrize("ratio", [1e3, 1e4])
def test_fixed_point_form_one_dominant_activation_in_every_group(ratio, route):
    """Every group holds one activation `ratio` times the rest (which then lose their last bits to the fixed-point
    grid), and a quarter of the rows have a weight that dequantises to exactly 0 at the dominant column of every
    group, so that nothing large hides their rounding error."""
    N, K = 512, 2048
    L = dict(oracle_layer(N, K, 2, 1, seed_name="fixed-point-worst"))
    rng = np.random.default_rng(int(ratio))
    x = rng.normal(0.0, 1.0, (1, K)).astype(np.float32)
    dom = 128 * np.arange(K // 128) + rng.integers(0, 128, K // 128)
    x[0, dom] = ratio * np.sign(x[0, dom])
    x = x.astype(np.float16)
    codes = L["codes"].copy()
    zero_rows = np.arange(0, N, 4)
    zint = L["zeros"].astype(np.float64)                     # Eq. 1 zero points are integers inside the code range
    for j, k in enumerate(dom):
        codes[zero_rows, k] = zint[j, zero_rows].astype(np.uint8)     # q = z: the weight is exactly 0
    L["codes"] = codes
    assert (orc.dequant_f64(codes, L["scales"], L["zeros"])[np.ix_(zero_rows, dom)] == 0).all()
    y = _run_single_token_set(L, x, route)
    y_ref = orc.linear_f64(x, codes, L["scales"], L["zeros"])
    check_output(y, y_ref, f"dominant activation x{ratio:g}")
    _check_row_bound(y, y_ref, _row_bound(L, x), f"dominant activation x{ratio:g}")


@pytest.mark.parametrize("route", ROUTES)
def test_fixed_point_form_largest_and_smallest_fp16_activations(route):
    """A group whose largest |x| is 65504 (the fixed-point scale 2^S is then below 1), a group of fp16 subnormals
    only (2^S = 2^27), a group with one subnormal among zeros, and ordinary groups in between."""
    N, K = 256, 1024
    L = dict(oracle_layer(N, K, 2, 1, seed_name="fixed-point-range"))
    rng = np.random.default_rng(65504)
    x = rng.normal(0.0, 1.0, (1, K)).astype(np.float16)
    x[0, 128 + 17] = np.float16(65504.0)
    x[0, 128 + 90] = np.float16(-65504.0)
    sub = (rng.integers(1, 1024, 128).astype(np.uint16) | (rng.integers(0, 2, 128).astype(np.uint16) << 15)).view(np.float16)
    x[0, 384:512] = sub                                            # subnormals of both signs
    x[0, 640:768] = 0
    x[0, 700] = np.array([1], dtype=np.uint16).view(np.float16)[0]  # the smallest subnormal, alone in its group
    y = _run_single_token_set(L, x, route)
    y_ref = orc.linear_f64(x, L["codes"], L["scales"], L["zeros"])
    check_output(y, y_ref, "fp16 range")
    _check_row_bound(y, y_ref, _row_bound(L, x), "fp16 range")
    # the subnormal-only groups on their own: exact products, so only the fp16 rounding of y is left
    x2 = np.zeros_like(x)
    x2[0, 384:512] = sub
    x2[0, 700] = x[0, 700]
    y2 = _run_single_token_set(L, x2, route)
    y2_ref = orc.linear_f64(x2, L["codes"], L["scales"], L["zeros"])
    assert np.abs(y2.astype(np.float64) - y2_ref).max() <= 2.0 ** -10 * np.abs(y2_ref).max() + 2.0 ** -25
