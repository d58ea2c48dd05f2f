"""GPU parity: the layer-set launch of the decode path (slim_gemv_set_plan / slim_mpq_gemv_set)
against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from tests.helpers import check_output, oracle_layer

pytestmark = pytest.mark.gpu


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


def _device_layer(L):
    slim = _slim()
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    return slim.QuantLinear(packed, L["bits"], torch.from_numpy(L["scales"]).cuda(), torch.from_numpy(L["zeros"]).cuda(), L["N"], L["K"])


def _run_set(layers):
    """layers: oracle dicts.  Returns the list of y (numpy) the set launch produced."""
    slim = _slim()
    entries = []
    for L in layers:
        x = torch.from_numpy(L["x"]).cuda()
        y = torch.full((L["M"], L["N"]), float("nan"), dtype=torch.float16, device="cuda")
        entries.append((_device_layer(L), x, y))
    s = slim.LayerSet(entries)
    s.run()
    s.check()
    return [y.cpu().numpy() for (_, _, y) in entries], s


def _check_all(layers, ys, what):
    for k, (L, y) in enumerate(zip(layers, ys)):
        y_ref = orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"])
        check_output(y, y_ref, f"{what}: layer {k} ({L['N']}x{L['K']} M={L['M']})")


def test_mixed_shapes_one_token():
    # several tiles, a ragged last row block (272 = 2 * 128 + 16), one to eleven groups
    layers = [oracle_layer(512, 1024, 2, 1, block=0), oracle_layer(272, 1408, 3, 1, block=1),
              oracle_layer(128, 128, 2, 1, block=2), oracle_layer(16, 256, 3, 1, block=3),
              oracle_layer(1040, 512, 2, 1, block=4)]
    ys, s = _run_set(layers)
    _check_all(layers, ys, "one token")
    # a single-token set this small runs as one launch with every CTA resident at once: whole clusters per layer,
    # 2 x resident_pairs tiles of 16 rows per CTA
    assert s.info["resident_pairs"] > 0 and s.info["resident_cluster"] in (4, 8)
    rows = 32 * s.info["resident_pairs"]
    cs = s.info["resident_cluster"]
    assert s.info["grid"] == sum(-(-(-(-L["N"] // rows)) // cs) * cs for L in layers)


def test_small_set_of_several_tokens_cuts_its_row_blocks_into_parts():
    # the same shapes with two tokens somewhere: the persistent ring, and a set this small cuts the groups of its row
    # blocks into parts (fewer for the layers with few groups)
    layers = [oracle_layer(512, 1024, 2, 2, block=0), oracle_layer(272, 1408, 3, 1, block=1),
              oracle_layer(128, 128, 2, 1, block=2), oracle_layer(16, 256, 3, 2, block=3),
              oracle_layer(1040, 512, 2, 1, block=4)]
    ys, s = _run_set(layers)
    _check_all(layers, ys, "two tokens")
    rows = 128 * s.info["tiles_per_warp"]           # rows of a work item
    assert s.info["resident_pairs"] == 0 and s.info["split"] > 1
    parts = [min(s.info["split"], max(L["K"] // 128 // 4, 1)) for L in layers]
    assert s.info["n_items"] == sum(k * -(-L["N"] // rows) for k, L in zip(parts, layers))


@pytest.mark.parametrize("Ms", [(1, 2, 3), (4, 8, 5), (16, 9, 1), (16, 16, 16), (17, 3, 1), (32, 32, 32), (5, 40, 64), (64, 64, 64), (33, 1, 24)])
def test_mixed_token_counts(Ms):
    layers = [oracle_layer(384, 768, 2, Ms[0], block=0), oracle_layer(144, 1280, 3, Ms[1], block=1),
              oracle_layer(256, 256, 2, Ms[2], block=2)]
    ys, _ = _run_set(layers)
    _check_all(layers, ys, f"Ms={Ms}")


@pytest.mark.parametrize("bits", [[1] * 8, [2] * 8, [3] * 8, [4] * 8, [1, 4, 2, 3, 3, 1, 4, 2], [3], [2, 1]])
def test_adversarial_bit_maps(bits):
    layers = [oracle_layer(144, 128 * len(bits), 2, M, bits=bits, block=M) for M in (1, 4)]
    ys, _ = _run_set(layers)
    _check_all(layers, ys, f"bits={bits}")


def test_many_layers_more_items_than_ctas_and_repeatable():
    # 60 layers x 5 or 9 row blocks: more items than CTAs, so CTAs walk across layer boundaries
    layers = [oracle_layer(1136, 384, 2 + (k & 1), 1, block=k) for k in range(60)]
    ys, s = _run_set(layers)
    _check_all(layers, ys, "many layers")
    assert s.info["n_items"] == 60 * -(-1136 // (128 * s.info["tiles_per_warp"])) >= s.info["grid"] and s.info["split"] == 1
    ys2, _ = _run_set(layers)
    for a, b in zip(ys, ys2):
        assert (a.view(np.uint16) == b.view(np.uint16)).all(), "two runs of the same set differ"


def test_one_hot_x_returns_dequantised_columns():
    L = oracle_layer(256, 1024, 2, 1)
    What = orc.dequant_f64(L["codes"], L["scales"], L["zeros"])
    layers = []
    cols = (0, 1, 31, 32, 127, 128, 500, 1023)
    for k in cols:
        Lk = dict(L)
        x = np.zeros((1, 1024), dtype=np.float16)
        x[0, k] = 1.0
        Lk["x"] = x
        layers.append(Lk)
    ys, _ = _run_set(layers)
    for k, y in zip(cols, ys):
        want = What[:, k].astype(np.float16)   # exact column, rounded once to fp16
        assert (y[0].view(np.uint16) == want.view(np.uint16)).all(), f"column {k}"


def test_half_integer_zero_points_and_zero_x():
    L = oracle_layer(128, 512, 3, 2)
    Lh = dict(L)
    Lh["zeros"] = (L["zeros"].astype(np.float32) + 0.5).astype(np.float16)
    L0 = dict(L)
    L0["x"] = np.zeros((2, 512), np.float16)
    ys, _ = _run_set([Lh, L0])
    check_output(ys[0], orc.linear_f64(Lh["x"], Lh["codes"], Lh["scales"], Lh["zeros"]), "half-integer zeros")
    assert (ys[1] == 0).all()


def test_agrees_with_the_single_layer_entry_point():
    slim = _slim()
    L = oracle_layer(4096, 4096, 2, 1, seed_name="set-vs-single")
    ys, _ = _run_set([L])
    dl = _device_layer(L)
    ws = slim.new_workspace(1, L["N"], L["K"], L["bits"])
    y1 = slim.mpq_gemv(torch.from_numpy(L["x"]).cuda(), dl.packed, L["bits"], dl.scales, dl.zeros, L["N"], ws).cpu().numpy()
    y_ref = orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"])
    check_output(ys[0], y_ref, "set launch, 4096x4096")
    # two summation orders of the same products: both within the oracle's tolerance of each other
    assert np.abs(ys[0].astype(np.float64) - y1.astype(np.float64)).max() <= 5e-3 * np.abs(y_ref).max()


def test_rejects_bad_sets():
    slim = _slim()
    L = oracle_layer(128, 256, 2, 1)
    dl = _device_layer(L)
    x = torch.from_numpy(L["x"]).cuda()
    with pytest.raises(ValueError):
        slim.LayerSet([])
    with pytest.raises(ValueError):
        slim.LayerSet([(dl, x, torch.empty(1, 64, dtype=torch.float16, device="cuda"))])
    x65 = torch.zeros(65, 256, dtype=torch.float16, device="cuda")          # a set takes up to 64 tokens per layer
    with pytest.raises(slim.SlimError):
        slim.LayerSet([(dl, x65, torch.empty(65, 128, dtype=torch.float16, device="cuda"))])


def test_llama7b_shapes_full_size_in_the_benchmark_configuration():
    """Full-size LLaMA-7B layers (q, gate, down shapes) as one set that is larger than the persistent grid, so that
    CTAs walk several items and cross layer boundaries as in the benchmark's sweep; the oracle computes sampled rows."""
    slim = _slim()
    shapes = [(4096, 4096), (11008, 4096), (4096, 11008)]
    base = [oracle_layer(N, K, 2, 1, seed_name="set-full", block=i) for i, (N, K) in enumerate(shapes)]
    dev = [_device_layer(L) for L in base]
    entries, meta = [], []
    rng = np.random.default_rng(2405)
    for rep in range(12):
        for L, dl in zip(base, dev):
            x = rng.normal(0, 1, (1, L["K"])).astype(np.float16)
            y = torch.full((1, L["N"]), float("nan"), dtype=torch.float16, device="cuda")
            entries.append((dl, torch.from_numpy(x).cuda(), y))
            meta.append((L, x))
    s = slim.LayerSet(entries)
    assert s.info["n_items"] > 2 * s.info["grid"]
    s.run()
    s.check()
    for k, ((L, x), (_, _, y)) in enumerate(zip(meta, entries)):
        y = y.cpu().numpy()
        assert np.isfinite(y.astype(np.float64)).all(), f"entry {k}"
        N = L["N"]
        rows = np.unique(np.concatenate([[0, 1, 15, 16, 255, 256, N - 1], rng.integers(0, N, 120)]))
        y_ref = orc.linear_rows_f64(x, L["codes"], L["scales"], L["zeros"], rows)
        check_output(y[:, rows], y_ref, f"entry {k}: {N}x{L['K']}")


def test_projections_that_share_one_input():
    """q/k/v (and gate/up) of a block read the same activations: one set, one x tensor, three outputs."""
    slim = _slim()
    layers = [oracle_layer(384, 1024, 2, 2, seed_name="qkv", block=i) for i in range(3)]
    x = torch.from_numpy(layers[0]["x"]).cuda()
    entries = [(_device_layer(L), x, torch.empty(2, L["N"], dtype=torch.float16, device="cuda")) for L in layers]
    s = slim.LayerSet(entries)
    s.run()
    s.check()
    for L, (_, _, y) in zip(layers, entries):
        check_output(y.cpu().numpy(), orc.linear_f64(layers[0]["x"], L["codes"], L["scales"], L["zeros"]), "shared x")


@pytest.mark.parametrize("M", [1, 2, 9])
def test_layers_that_share_input_and_bit_map_are_staged_once(M):
    """The staged form of x depends on the bit-width of each group, so layers share a staged copy when they share
    the x tensor AND the bit map.  Two such layers, one with the same x but another map in between, and one with
    its own x: the staging tasks are those of three layers, and every output still matches."""
    slim = _slim()
    K = 1024
    bits_a = np.array([2, 1, 3, 2, 2, 4, 1, 1], dtype=np.uint8)
    bits_b = np.array([3, 1, 2, 2, 1, 2, 3, 2], dtype=np.uint8)
    layers = [oracle_layer(384, K, 2, M, seed_name="share", block=0, bits=bits_a),
              oracle_layer(256, K, 2, M, seed_name="share", block=1, bits=bits_b),
              oracle_layer(512, K, 2, M, seed_name="share", block=2, bits=bits_a),
              oracle_layer(128, K, 2, M, seed_name="share", block=3, bits=bits_a)]
    x_shared = torch.from_numpy(layers[0]["x"]).cuda()
    x_own = torch.from_numpy(layers[3]["x"]).cuda()
    xs = [x_shared, x_shared, x_shared, x_own]
    entries = [(_device_layer(L), x, torch.empty(M, L["N"], dtype=torch.float16, device="cuda")) for L, x in zip(layers, xs)]
    s = slim.LayerSet(entries)
    alone = slim.LayerSet(entries[:1]).info["stage_tasks"]
    assert s.info["stage_tasks"] == 3 * alone
    s.run()
    s.check()
    for k, (L, (_, x, y)) in enumerate(zip(layers, entries)):
        check_output(y.cpu().numpy(), orc.linear_f64(x.cpu().numpy(), L["codes"], L["scales"], L["zeros"]), f"layer {k}")


@pytest.mark.parametrize("M", [1, 3])
def test_a_set_that_reads_the_outputs_of_the_set_before(M):
    """Two small sets launched back to back on one stream; the layers of the second read what the first wrote.  At
    one token both are single resident launches that fetch their weights before they wait for the launch ahead."""
    slim = _slim()
    first = [oracle_layer(512, 1024, 2, M, seed_name="set-chain", block=0), oracle_layer(768, 1024, 3, M, seed_name="set-chain", block=1)]
    second = [oracle_layer(256, 512, 2, M, seed_name="set-chain", block=2), oracle_layer(384, 768, 2, M, seed_name="set-chain", block=3)]
    x0 = torch.from_numpy(first[0]["x"]).cuda()
    mid = [torch.zeros(M, L["N"], dtype=torch.float16, device="cuda") for L in first]
    out = [torch.zeros(M, L["N"], dtype=torch.float16, device="cuda") for L in second]
    s1 = slim.LayerSet([(_device_layer(L), x0, y) for L, y in zip(first, mid)])
    s2 = slim.LayerSet([(_device_layer(L), x, y) for L, x, y in zip(second, mid, out)])
    assert (s1.info["resident_pairs"] > 0) == (M == 1)
    for _ in range(3):
        s1.run()
        s2.run()
    s1.check()
    s2.check()
    x0h = first[0]["x"]
    for L, y in zip(first, mid):
        check_output(y.cpu().numpy(), orc.linear_f64(x0h, L["codes"], L["scales"], L["zeros"]), "first set")
    for L, x, y in zip(second, mid, out):
        check_output(y.cpu().numpy(), orc.linear_f64(x.cpu().numpy(), L["codes"], L["scales"], L["zeros"]), "second set")


def test_single_token_fixed_point_with_outlier_channels():
    """Single-token sets round x per group to fixed point relative to the group's largest |x|.  Outlier channels
    (a few activations 100 x the rest, as in LLM activations) and a group of tiny activations must stay within the
    layer tolerance, and the error of a row must stay below 2^-22 max|x_group| sum|w-hat| per group."""
    L = oracle_layer(512, 1024, 2, 1, seed_name="set-outlier")
    rng = np.random.default_rng(11)
    x = rng.normal(0, 1, (1, 1024)).astype(np.float32)
    x[0, [5, 300, 301, 900]] *= 100.0                 # outlier channels in groups 0, 2 and 7
    x[0, 128:256] *= 1e-3                             # a group of small activations
    x[0, 384:512] = 0                                 # a group of zeros
    L = dict(L)
    L["x"] = x.astype(np.float16)
    ys, _ = _run_set([L])
    y_ref = orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"])
    check_output(ys[0], y_ref, "outlier channels")
    What = np.abs(orc.dequant_f64(L["codes"], L["scales"], L["zeros"]))
    xa = np.abs(L["x"].astype(np.float64))[0]
    bound = sum(2.0 ** -22 * xa[128 * j:128 * j + 128].max() * What[:, 128 * j:128 * j + 128].sum(axis=1) for j in range(8))
    err = np.abs(ys[0].astype(np.float64) - y_ref)[0]
    # + the fp16 rounding of y and the fp32 rounding of the running sum over the groups
    assert (err <= bound + 2.0 ** -10 * np.abs(y_ref[0]) + 1e-5 * np.abs(y_ref).max()).all()

