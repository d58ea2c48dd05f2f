"""GPU parity: slim_mpq_gemm (M > 16, tcgen05 path) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from tests.helpers import check_output, oracle_layer

pytestmark = pytest.mark.gpu


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


def _run(L, x=None, scales=None, zeros=None):
    slim = _slim()
    x = L["x"] if x is None else x
    scales = L["scales"] if scales is None else scales
    zeros = L["zeros"] if zeros is None else zeros
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    ws = slim.new_workspace(x.shape[0], L["N"], L["K"], L["bits"])
    y = slim.mpq_gemm(torch.from_numpy(x).cuda(), packed, L["bits"], torch.from_numpy(scales).cuda(),
                      torch.from_numpy(zeros).cuda(), L["N"], ws)
    slim.workspace_status(ws)
    return y.cpu().numpy()


@pytest.mark.parametrize("bits", [[1, 1], [2, 2], [3, 3], [4, 4], [1, 4, 2, 3]])
def test_identity_x_returns_dequantised_weights_bit_exact(bits):
    """x = I (one token per input column): y must be W-hat^T exactly as slim_dequant defines it.
    Pins the tensor-memory operand layout, the swizzled x tiles and every decode path."""
    K = 128 * len(bits)
    L = oracle_layer(144, K, 2, 1, bits=bits)
    x = np.eye(K, dtype=np.float16)
    y = _run(L, x=x)
    want = orc.dequant_f16(L["codes"], L["scales"], L["zeros"]).T
    assert (y.view(np.uint16) == np.ascontiguousarray(want).view(np.uint16)).all()


@pytest.mark.parametrize("M", [17, 64, 128, 129, 256, 300])
@pytest.mark.parametrize("N,K,avg", [(256, 1024, 3), (272, 1408, 2)])
def test_small_layers_token_counts(N, K, avg, M):
    L = oracle_layer(N, K, avg, M)
    y = _run(L)
    check_output(y, orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"]), f"{N}x{K} avg{avg} M={M}")


def test_half_integer_zero_points_and_zero_scale():
    L = oracle_layer(128, 512, 3, 40)
    zh = (L["zeros"].astype(np.float32) + 0.5).astype(np.float16)
    check_output(_run(L, zeros=zh), orc.linear_f64(L["x"], L["codes"], L["scales"], zh), "half-integer zeros")
    s0 = L["scales"].copy()
    s0[1] = 0
    check_output(_run(L, scales=s0), orc.linear_f64(L["x"], L["codes"], s0, L["zeros"]), "zero scale group")
    assert (_run(L, x=np.zeros((40, 512), np.float16)) == 0).all()


def test_many_tiles_persistent_loop_and_determinism():
    """More tiles than SMs (persistent loop wraps), ragged row block and token tail."""
    slim = _slim()
    L = oracle_layer(2064, 512, 3, 2100)
    y1 = _run(L)
    y2 = _run(L)
    assert (y1.view(np.uint16) == y2.view(np.uint16)).all()
    rows = np.unique(np.concatenate([[0, 127, 128, 2047, 2048, 2063], np.random.default_rng(1).integers(0, 2064, 100)]))
    check_output(y1[:, rows], orc.linear_rows_f64(L["x"], L["codes"], L["scales"], L["zeros"], rows), "2064x512 M=2100")


@pytest.mark.parametrize("N,K,M", [(5120, 5120, 512), (13824, 5120, 512), (5120, 13824, 2048)])
def test_13b_shapes_full_size_sampled_rows(N, K, M):
    """Full-size layers of the batched configuration (avg 3 bits); the oracle computes sampled rows."""
    L = oracle_layer(N, K, 3, M)
    y = _run(L)
    rng = np.random.default_rng(N + K + M)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, N - 1], rng.integers(0, N, 120)]))
    check_output(y[:, rows], orc.linear_rows_f64(L["x"], L["codes"], L["scales"], L["zeros"], rows), f"{N}x{K} M={M}")
    assert np.isfinite(y.astype(np.float64)).all()


def test_stream_k_and_whole_tile_paths_agree():
    """A shape whose tile count leaves the last wave half empty takes the stream-K path when the
    workspace is large enough and whole tiles when it is not; both must match the oracle."""
    slim = _slim()
    L = oracle_layer(5120, 13824, 3, 512)         # 40 row blocks x 2 token tiles = 80 tiles on 148 SMs
    assert slim.workspace_bytes(512, 5120, 13824, L["bits"]) > 1 << 20
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    sc, zp, x = (torch.from_numpy(L[k]).cuda() for k in ("scales", "zeros", "x"))
    big = slim.new_workspace(512, 5120, 13824, L["bits"])
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    ys = []
    for ws in (big, small, big):                   # the large workspace is used twice: its flags must be reusable
        ys.append(slim.mpq_gemm(x, packed, L["bits"], sc, zp, 5120, ws).cpu().numpy())
        slim.workspace_status(ws)
    rows = np.unique(np.concatenate([[0, 127, 128, 5119], np.random.default_rng(2).integers(0, 5120, 100)]))
    y_ref = orc.linear_rows_f64(L["x"], L["codes"], L["scales"], L["zeros"], rows)
    for y in ys:
        check_output(y[:, rows], y_ref, "5120x13824 M=512")
    assert (ys[0].view(np.uint16) == ys[2].view(np.uint16)).all()
    assert np.abs(ys[0].astype(np.float64) - ys[1].astype(np.float64)).max() <= 2e-3 * np.abs(ys[1].astype(np.float64)).max()


@pytest.mark.parametrize("M", [100, 300])
def test_cut_tiles_with_many_peers(M):
    """Few tiles and a long K: the plan cuts every tile into many segments, so the pair that starts a tile adds the
    partial tiles of five to nine peers (its shared-memory ring goes round several times), with a ragged last row
    block and a ragged token tile, at 128 and at 256 tokens per tile."""
    slim = _slim()
    N, K = 2064, 13824
    L = oracle_layer(N, K, 3, M)
    assert slim.workspace_bytes(M, N, K, L["bits"]) > 1 << 20          # the tiles are cut
    y1 = _run(L)
    y2 = _run(L)
    assert (y1.view(np.uint16) == y2.view(np.uint16)).all()
    rows = np.unique(np.concatenate([[0, 127, 128, 2047, 2048, 2063], np.random.default_rng(M).integers(0, N, 100)]))
    check_output(y1[:, rows], orc.linear_rows_f64(L["x"], L["codes"], L["scales"], L["zeros"], rows), f"{N}x{K} M={M}")


def test_argument_errors_are_statuses():
    slim = _slim()
    L = oracle_layer(128, 256, 2, 1)
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    sc, zp = (torch.from_numpy(L[k]).cuda() for k in ("scales", "zeros"))
    ws = slim.new_workspace(32, 128, 256, L["bits"])
    x16 = torch.zeros((16, 256), dtype=torch.float16, device="cuda")
    with pytest.raises(slim.SlimError) as e:
        slim.mpq_gemm(x16, packed, L["bits"], sc, zp, 128, ws)
    assert e.value.status == -1
    y0 = slim.mpq_gemm(torch.zeros((0, 256), dtype=torch.float16, device="cuda"), packed, L["bits"], sc, zp, 128, ws)
    assert y0.shape == (0, 128)
