"""GPU parity at the group sizes of the paper's group-size ablation (appendix): g in {32, 64, 256, 512} next to the
default 128, for every entry point of the hot path, against the oracle run at the same group size."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from paper_2405_14917_b200 import workloads as wl
from tests.helpers import check_output

pytestmark = pytest.mark.gpu

LARGE = (256, 512)           # groups of several 128-column K-tiles: the kernels of g = 128 with shared scale rows
SMALL = (32, 64)             # K-tiles of the group's own size: kernels of their own
ALL = SMALL + (128,) + LARGE


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


def _layer(N, K, g, avg_bits, M, seed=0, bits=None):
    sd = wl.layer_seed("test", f"group-size-{g}-{N}x{K}", seed)
    W = wl.make_weight(sd, N, K)
    a = wl.make_act_norms(sd, K)
    x = wl.make_x(sd, M, K)
    if bits is None:
        bits = orc.allocate_bits(orc.group_salience(W, a, g), avg_bits)
    bits = np.asarray(bits, dtype=np.uint8)
    codes, scales, zeros = orc.quantize_minmax(W, bits, g)
    return dict(x=x, bits=bits, codes=codes, scales=scales, zeros=zeros, N=N, K=K, M=M, g=g)


def _dev(L):
    return (torch.from_numpy(orc.pack(L["codes"], L["bits"], L["g"])).cuda(), torch.from_numpy(L["scales"]).cuda(),
            torch.from_numpy(L["zeros"]).cuda())


@pytest.mark.parametrize("g", ALL)
@pytest.mark.parametrize("avg_bits", [2, 3])
def test_pack_and_dequant_bit_exact(g, avg_bits):
    slim = _slim()
    N, K = 272, 2048
    L = _layer(N, K, g, avg_bits, 1)
    want = orc.pack(L["codes"], L["bits"], g)
    assert slim.packed_bytes(N, K, L["bits"], g) == want.size == N * K * avg_bits // 8
    guard = 64
    buf = torch.full((want.size + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    packed = buf[guard:guard + want.size]
    slim.pack_weights(torch.from_numpy(L["codes"]).cuda(), L["bits"], packed, g=g)
    got = buf.cpu().numpy()
    assert (got[guard:-guard] == want).all(), "packed buffer differs from the oracle"
    assert (got[:guard] == 0xA5).all() and (got[-guard:] == 0xA5).all(), "wrote outside the packed buffer"
    sc, zp = torch.from_numpy(L["scales"]).cuda(), torch.from_numpy(L["zeros"]).cuda()
    What = slim.dequant(packed.clone(), L["bits"], sc, zp, N, K, g=g).cpu().numpy()
    assert (What.view(np.uint16) == orc.dequant_f16(L["codes"], L["scales"], L["zeros"], g).view(np.uint16)).all()


@pytest.mark.parametrize("g", ALL)
@pytest.mark.parametrize("bits_of", ["all1", "all4", "mixed"])
def test_adversarial_bit_maps_pack_dequant(g, bits_of):
    slim = _slim()
    N, K = 48, 1024
    G = K // g
    bits = {"all1": [1] * G, "all4": [4] * G, "mixed": [(1, 4, 2, 3)[j % 4] for j in range(G)]}[bits_of]
    L = _layer(N, K, g, 2, 1, bits=bits)
    packed = slim.pack_weights(torch.from_numpy(L["codes"]).cuda(), L["bits"], g=g)
    assert (packed.cpu().numpy() == orc.pack(L["codes"], L["bits"], g)).all()
    What = slim.dequant(packed, L["bits"], torch.from_numpy(L["scales"]).cuda(), torch.from_numpy(L["zeros"]).cuda(), N, K, g=g)
    assert (What.cpu().numpy().view(np.uint16) == orc.dequant_f16(L["codes"], L["scales"], L["zeros"], g).view(np.uint16)).all()


@pytest.mark.parametrize("g", ALL)
@pytest.mark.parametrize("M", [1, 5, 16])
def test_decode_path(g, M):
    slim = _slim()
    N, K = 528, 2048
    L = _layer(N, K, g, 2, M, seed=M)
    packed, sc, zp = _dev(L)
    ws = slim.new_workspace(M, N, K, L["bits"], g=g)
    y = slim.mpq_gemv(torch.from_numpy(L["x"]).cuda(), packed, L["bits"], sc, zp, N, ws, g=g)
    slim.workspace_status(ws)
    check_output(y.cpu().numpy(), orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"], g), f"gemv g={g} M={M}")


@pytest.mark.parametrize("g", ALL)
def test_decode_path_one_hot_x_returns_the_dequantised_column(g):
    slim = _slim()
    N, K = 64, 1024
    L = _layer(N, K, g, 3, 1)
    packed, sc, zp = _dev(L)
    ws = slim.new_workspace(1, N, K, L["bits"], g=g)
    What = orc.dequant_f64(L["codes"], L["scales"], L["zeros"], g)
    for k in (0, g - 1, g, 3 * g // 2 + 1, K - 1):
        x = np.zeros((1, K), dtype=np.float16)
        x[0, k] = 1.0
        y = slim.mpq_gemv(torch.from_numpy(x).cuda(), packed, L["bits"], sc, zp, N, ws, g=g).cpu().numpy()
        assert (y[0].view(np.uint16) == What[:, k].astype(np.float16).view(np.uint16)).all(), f"g={g} column {k}"


@pytest.mark.parametrize("g", ALL)
@pytest.mark.parametrize("M", [40, 300])
def test_batched_path(g, M):
    slim = _slim()
    N, K = 272, 1024
    L = _layer(N, K, g, 3, M, seed=M)
    packed, sc, zp = _dev(L)
    ws = slim.new_workspace(M, N, K, L["bits"], g=g)
    y = slim.mpq_gemm(torch.from_numpy(L["x"]).cuda(), packed, L["bits"], sc, zp, N, ws, g=g)
    slim.workspace_status(ws)
    check_output(y.cpu().numpy(), orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"], g), f"gemm g={g} M={M}")


@pytest.mark.parametrize("g", LARGE)
@pytest.mark.parametrize("Ms", [(1, 1, 1), (4, 2, 16)])
def test_layer_set_with_groups_of_several_tiles(g, Ms):
    slim = _slim()
    layers = [_layer(384, 1024, g, 2, Ms[0], seed=1), _layer(144, 2048, g, 3, Ms[1], seed=2), _layer(1040, 1024, g, 2, Ms[2], seed=3)]
    entries = []
    for L in layers:
        packed, sc, zp = _dev(L)
        y = torch.full((L["M"], L["N"]), float("nan"), dtype=torch.float16, device="cuda")
        entries.append((slim.QuantLinear(packed, L["bits"], sc, zp, L["N"], L["K"], g), torch.from_numpy(L["x"]).cuda(), y))
    s = slim.LayerSet(entries, g=g)
    s.run()
    s.check()
    for L, (_, _, y) in zip(layers, entries):
        check_output(y.cpu().numpy(), orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"], g), f"set g={g} M={L['M']}")


@pytest.mark.parametrize("g", LARGE)
def test_full_size_layer_with_large_groups(g):
    """A 4096 x 4096 layer at g = 256 / 512 through the decode path, the layer-set launch and the batched path."""
    slim = _slim()
    N = K = 4096
    L = _layer(N, K, g, 2, 1)
    packed, sc, zp = _dev(L)
    rng = np.random.default_rng(g)
    rows = np.unique(np.concatenate([[0, 15, 16, N - 1], rng.integers(0, N, 150)]))
    for M in (1, 16, 128):
        x = rng.normal(0, 1, (M, K)).astype(np.float16)
        ws = slim.new_workspace(M, N, K, L["bits"], g=g)
        fn = slim.mpq_gemv if M <= 16 else slim.mpq_gemm
        y = fn(torch.from_numpy(x).cuda(), packed, L["bits"], sc, zp, N, ws, g=g)
        slim.workspace_status(ws)
        check_output(y.cpu().numpy()[:, rows], orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows, g), f"g={g} M={M}")


def _same_bits(a, b):
    return (a.cpu().numpy().view(np.uint16) == b.view(np.uint16)).all()


@pytest.mark.parametrize("g", ALL)
@pytest.mark.parametrize("N,K", [(48, 1024), (272, 4096)])
def test_salience_and_quantizers_match_the_oracle_bit_for_bit(g, N, K):
    """Group salience, the Eq. 1 quantizer, its Eq. 2 one-bit form and SQC (Algorithm 2) at group size g."""
    slim = _slim()
    sd = wl.layer_seed("test", f"quant-group-size-{g}-{N}x{K}", 0)
    W = wl.make_weight(sd, N, K)
    a = wl.make_act_norms(sd, K)
    Wd = torch.from_numpy(W).cuda()
    sal_ref = orc.group_salience(W, a, g)
    sal = slim.group_salience(Wd, torch.from_numpy(a).cuda(), g).cpu().numpy()
    assert sal.shape == (K // g,) and np.allclose(sal, sal_ref, rtol=1e-12, atol=0)
    rng = np.random.default_rng(g + N)
    bits = rng.integers(1, 5, K // g).astype(np.uint8)
    for one_bit, ref in (("minmax", orc.quantize_minmax), ("sign_alpha", orc.quantize_minmax_sign1)):
        codes, scales, zeros = slim.quantize_minmax(Wd, bits, one_bit=one_bit, g=g)
        c_ref, s_ref, z_ref = ref(W, bits, g)
        assert _same_bits(scales, s_ref) and _same_bits(zeros, z_ref), one_bit
        assert (codes.cpu().numpy() == c_ref).all(), one_bit
    rows = 16 if K > 1024 else N                  # the oracle's tau search is slow: a slice of the rows
    codes, scales, zeros, tau = slim.quantize_sqc(Wd[:rows].contiguous(), bits, lam=0.1, n=20, g=g)
    c_ref, s_ref, z_ref, t_ref, _, _ = orc.quantize_sqc(W[:rows], bits, g, lam=0.1, n=20)
    assert (tau.cpu().numpy() == t_ref).all()
    assert _same_bits(scales, s_ref) and _same_bits(zeros, z_ref) and (codes.cpu().numpy() == c_ref).all()


@pytest.mark.parametrize("g", ALL)
def test_layer_built_on_the_device_from_a_weight(g):
    """Salience -> bit allocation -> Eq. 1 -> packing on the device at group size g, then one decode call: the result
    is the oracle's layer of the same bit map."""
    slim = _slim()
    N, K, M = 256, 2048, 3
    sd = wl.layer_seed("test", f"from-weight-{g}", 0)
    W = wl.make_weight(sd, N, K)
    a = wl.make_act_norms(sd, K)
    x = wl.make_x(sd, M, K)
    L = slim.QuantLinear.from_weight(torch.from_numpy(W).cuda(), torch.from_numpy(a).cuda(), 2, g=g)
    assert L.g == g and int(L.bits.astype(int).sum()) * g == 2 * K
    codes, scales, zeros = orc.quantize_minmax(W, L.bits, g)
    assert (L.packed.cpu().numpy() == orc.pack(codes, L.bits, g)).all()
    ws = slim.new_workspace(M, N, K, L.bits, g=g)
    y = L.forward(torch.from_numpy(x).cuda(), ws)
    slim.workspace_status(ws)
    check_output(y.cpu().numpy(), orc.linear_f64(x, codes, scales, zeros, g), f"g={g}")


def test_unsupported_group_sizes_are_statuses():
    slim = _slim()
    bits = np.full(8, 2, dtype=np.uint8)
    for g in (16, 96, 1024):
        with pytest.raises(slim.SlimError) as e:
            slim.packed_bytes(64, 1024, bits[:max(1024 // g, 1)], g)
        assert e.value.status == -2
