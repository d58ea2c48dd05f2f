"""GPU parity: slim_mpq_gemv (M <= 16) against the fp64 oracle, through the C ABI."""
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
    y = slim.mpq_gemv(torch.from_numpy(x).cuda(), packed, L["bits"], torch.from_numpy(scales).cuda(),
                      torch.from_numpy(zeros).cuda(), L["N"], ws)
    slim.workspace_status(ws)
    return y.cpu().numpy()


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8, 9, 16])
@pytest.mark.parametrize("N,K,avg", [(512, 1024, 2), (272, 1408, 3)])
def test_small_layers_all_token_counts(N, K, avg, M):
    L = oracle_layer(N, K, avg, M)
    y = _run(L)
    y_ref = orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"])
    check_output(y, y_ref, f"{N}x{K} avg{avg} M={M}")


@pytest.mark.parametrize("N,K", [(16, 128), (16, 2048), (48, 32768), (2064, 256), (4736, 1024)])
def test_single_token_edge_shapes(N, K):
    """One token at the edges of the single-token kernel: a single tile and a single group; a K of 256 groups whose
    digit form does not fit a CTA (the general kernel takes it); row counts that leave a CTA with one tile of its pair
    and pad the grid to whole clusters; more CTAs than one tile pair each lets be resident (several pairs per CTA)."""
    L = oracle_layer(N, K, 2, 1, seed_name="one-token-edges")
    y = _run(L)
    check_output(y, orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"]), f"{N}x{K}")


@pytest.mark.parametrize("M", [1, 4])
@pytest.mark.parametrize("as_graph", [False, True])
def test_chain_of_layers_each_reading_the_output_of_the_one_before(M, as_graph):
    """Six layers launched back to back, each taking the y of the one before as its x.  The kernels are launched with
    programmatic stream serialisation and request their weights before they wait for the kernel ahead; what they read of
    x must still be that kernel's finished output.  Checked layer by layer against the oracle fed with the device's own
    (fp16) inputs, eagerly and as a replayed CUDA graph."""
    from paper_2405_14917_b200 import binding as slim
    dims = [1024, 512, 2048, 512, 1024, 256, 768]
    layers = [oracle_layer(dims[i + 1], dims[i], 3, M, seed_name="chain", block=i) for i in range(6)]
    dev = []
    for L in layers:
        dev.append(slim.QuantLinear(torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda(), L["bits"],
                                    torch.from_numpy(L["scales"]).cuda(), torch.from_numpy(L["zeros"]).cuda(), L["N"], L["K"]))
    acts = [torch.from_numpy(layers[0]["x"]).cuda()] + [torch.zeros(M, d, dtype=torch.float16, device="cuda") for d in dims[1:]]
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    slim.workspace_init(ws)

    def run():
        for i, dl in enumerate(dev):
            dl.forward(acts[i], ws, out=acts[i + 1])
    run()
    torch.cuda.synchronize()
    if as_graph:
        for a in acts[1:]:
            a.zero_()
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g):
                run()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
    slim.workspace_status(ws)
    for i, L in enumerate(layers):
        x_in = acts[i].cpu().numpy()
        y_ref = orc.linear_f64(x_in, L["codes"], L["scales"], L["zeros"])
        check_output(acts[i + 1].cpu().numpy(), y_ref, f"layer {i} of the chain")


@pytest.mark.parametrize("bits", [[1] * 8, [2] * 8, [3] * 8, [4] * 8, [1, 4, 2, 3, 3, 1, 4, 2], [3], [2, 1]])
@pytest.mark.parametrize("M", [1, 4])
def test_adversarial_bit_maps(bits, M):
    L = oracle_layer(144, 128 * len(bits), 2, M, bits=bits)
    y = _run(L)
    check_output(y, orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"]), f"bits={bits} M={M}")


def test_one_hot_x_returns_dequantised_columns():
    L = oracle_layer(256, 1024, 2, 1)
    What = orc.dequant_f64(L["codes"], L["scales"], L["zeros"])
    for k in (0, 1, 31, 32, 127, 128, 500, 1023):
        x = np.zeros((1, 1024), dtype=np.float16)
        x[0, k] = 1.0
        y = _run(L, x=x)
        want = What[:, k].astype(np.float16)   # exact column, rounded once to fp16
        assert (y[0].view(np.uint16) == want.view(np.uint16)).all(), f"column {k}"


def test_zero_x_zero_scale_and_half_zero_points():
    L = oracle_layer(128, 512, 3, 2)
    assert (_run(L, x=np.zeros((2, 512), np.float16)) == 0).all()
    s0 = L["scales"].copy()
    s0[1] = 0
    check_output(_run(L, scales=s0), orc.linear_f64(L["x"], L["codes"], s0, L["zeros"]), "zero scale group")
    zh = (L["zeros"].astype(np.float32) + 0.5).astype(np.float16)
    check_output(_run(L, zeros=zh), orc.linear_f64(L["x"], L["codes"], L["scales"], zh), "half-integer zeros")


def test_wide_dynamic_range_activations():
    """Outlier channels 1000x the typical activation, and tiny activations."""
    L = oracle_layer(256, 2048, 2, 2)
    x = L["x"].astype(np.float32)
    x[:, ::97] *= 1000.0
    x[1] *= 1e-3
    x = x.astype(np.float16)
    check_output(_run(L, x=x), orc.linear_f64(x, L["codes"], L["scales"], L["zeros"]), "outlier x")


def test_deterministic_and_workspace_reuse():
    slim = _slim()
    L = oracle_layer(4096, 4096, 2, 1)
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    sc, zp, x = (torch.from_numpy(L[k]).cuda() for k in ("scales", "zeros", "x"))
    ws = slim.new_workspace(1, 4096, 4096, L["bits"])
    ys = [slim.mpq_gemv(x, packed, L["bits"], sc, zp, 4096, ws).clone() for _ in range(5)]
    slim.workspace_status(ws)
    for y in ys[1:]:
        assert torch.equal(y, ys[0])
    check_output(ys[0].cpu().numpy(), orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"]), "4096x4096 M=1")


@pytest.mark.parametrize("N,K,avg,M", [(4096, 4096, 2, 1), (11008, 4096, 2, 1), (4096, 11008, 2, 1),
                                       (4096, 4096, 3, 16), (11008, 4096, 3, 8), (4096, 11008, 3, 4),
                                       (1024, 8192, 2, 1), (1024, 8192, 2, 16)])
def test_config_shapes_full_size_sampled_rows(N, K, avg, M):
    """Full-size config layers in the benchmark's launch configuration; the oracle computes sampled rows."""
    slim = _slim()
    L = oracle_layer(N, K, avg, M)
    y = _run(L)
    rng = np.random.default_rng(N + K + M)
    rows = np.unique(np.concatenate([[0, 1, 15, 16, N - 1], rng.integers(0, N, 250)]))
    y_ref = orc.linear_rows_f64(L["x"], L["codes"], L["scales"], L["zeros"], rows)
    check_output(y[:, rows], y_ref, f"{N}x{K} avg{avg} M={M}")
    assert np.isfinite(y.astype(np.float64)).all()


@pytest.mark.parametrize("M", [4, 8, 16])
def test_small_workspace_stages_x_inside_the_kernel(M):
    """From four tokens on x is put into fragment order by a kernel of its own, in the workspace;
    with a 256-byte workspace every CTA stages x itself.  Both paths must match the oracle."""
    slim = _slim()
    L = oracle_layer(1024, 2048, 3, M)
    assert slim.workspace_bytes(M, 1024, 2048, L["bits"]) > 256
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    sc, zp, x = (torch.from_numpy(L[k]).cuda() for k in ("scales", "zeros", "x"))
    y_ref = orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"])
    big = slim.new_workspace(M, 1024, 2048, L["bits"])
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for ws in (big, small, big):
        y = slim.mpq_gemv(x, packed, L["bits"], sc, zp, 1024, ws).cpu().numpy()
        check_output(y, y_ref, f"M={M} workspace {ws.numel()} B")


def test_argument_errors_are_statuses():
    slim = _slim()
    L = oracle_layer(128, 256, 2, 1)
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    sc, zp, x = (torch.from_numpy(L[k]).cuda() for k in ("scales", "zeros", "x"))
    tiny = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(slim.SlimError) as e:
        slim.mpq_gemv(x, packed, L["bits"], sc, zp, 128, tiny)
    assert e.value.status == -4
    ws = slim.new_workspace(1, 128, 256, L["bits"])
    x17 = torch.zeros((17, 256), dtype=torch.float16, device="cuda")
    with pytest.raises(slim.SlimError) as e:
        slim.mpq_gemv(x17, packed, L["bits"], sc, zp, 128, ws)
    assert e.value.status == -1
    # M = 0 is a no-op
    y0 = slim.mpq_gemv(torch.zeros((0, 256), dtype=torch.float16, device="cuda"), packed, L["bits"], sc, zp, 128, ws)
    assert y0.shape == (0, 128)
