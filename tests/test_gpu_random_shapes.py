"""GPU parity on seeded random shapes: the decode path through both of its entry points (slim_mpq_gemv and the
layer-set launch) and the batched path (slim_mpq_gemm) against the fp64 oracle, over row counts, K, group sizes,
bit maps, token counts, activation scales and half-integer zero points that the hand-picked cases of the other
files do not enumerate."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from tests.helpers import check_output

pytestmark = pytest.mark.gpu


def _random_layer(rng, g, M, max_k=4096, max_tiles=160):
    from paper_2405_14917_b200 import binding as slim
    K = g * int(rng.integers(1, max(2, max_k // g) + 1))
    if K % 128:
        K = (K // 128 + 1) * 128
    N = 16 * int(rng.integers(1, max_tiles))
    bits = rng.integers(1, 5, K // g).astype(np.uint8)
    W = (rng.normal(0, 0.02, (N, K)) * (1 + 9 * (rng.random(K) < 0.01))).astype(np.float16)
    codes, scales, zeros = orc.quantize_minmax(W, bits, g)
    if rng.random() < 0.3:
        zeros = (zeros.astype(np.float32) + 0.5).astype(np.float16)            # the zero points of Eq. 2
    x = (rng.normal(0, 1, (M, K)) * (10.0 ** rng.integers(-3, 3))).astype(np.float16)
    L = slim.QuantLinear(torch.from_numpy(orc.pack(codes, bits, g)).cuda(), bits, torch.from_numpy(scales).cuda(),
                         torch.from_numpy(zeros).cuda(), N, K, g)
    return L, x, orc.linear_f64(x, codes, scales, zeros, g)


@pytest.mark.parametrize("seed", range(6))
def test_single_layers_through_both_entry_points(seed):
    from paper_2405_14917_b200 import binding as slim
    rng = np.random.default_rng(1000 + seed)
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    slim.workspace_init(ws)
    for case in range(12):
        g = int(rng.choice([32, 64, 128, 128, 256, 512]))
        M = int(rng.choice([1, 1, 1, 2, 3, 7, 16]))
        L, x, ref = _random_layer(rng, g, M)
        xd = torch.from_numpy(x).cuda()
        y = L.forward(xd, ws)
        check_output(y.cpu().numpy(), ref, f"gemv seed {seed} case {case}: {L.N}x{L.K} g={g} M={M}")
        if g >= 128:
            y2 = torch.full((M, L.N), float("nan"), dtype=torch.float16, device="cuda")
            st = slim.LayerSet([(L, xd, y2)], g=g)
            st.run()
            st.check()
            check_output(y2.cpu().numpy(), ref, f"set seed {seed} case {case}: {L.N}x{L.K} g={g} M={M}")
    slim.workspace_status(ws)


@pytest.mark.parametrize("seed", range(6))
def test_sets_of_several_layers(seed):
    """One to six layers with their own shapes, bit maps and token counts: the resident launch at one token, the
    persistent ring (with and without parts) otherwise; every set runs twice."""
    from paper_2405_14917_b200 import binding as slim
    rng = np.random.default_rng(2000 + seed)
    modes = set()
    for case in range(8):
        g = int(rng.choice([128, 128, 256]))
        m_max = int(rng.choice([1, 1, 2, 5, 16]))
        entries, refs = [], []
        for _ in range(int(rng.integers(1, 7))):
            M = 1 if m_max == 1 else int(rng.integers(1, m_max + 1))
            L, x, ref = _random_layer(rng, g, M, max_k=2048, max_tiles=100)
            entries.append((L, torch.from_numpy(x).cuda(), torch.full((M, L.N), float("nan"), dtype=torch.float16, device="cuda")))
            refs.append(ref)
        st = slim.LayerSet(entries, g=g)
        modes.add("resident" if st.info["resident_pairs"] > 0 else ("ring in parts" if st.info["split"] > 1 else "ring"))
        for _ in range(2):
            st.run()
        st.check()
        for i, ((L, _, y), ref) in enumerate(zip(entries, refs)):
            check_output(y.cpu().numpy(), ref, f"seed {seed} case {case} layer {i}: {L.N}x{L.K} g={g}")
    assert modes          # which routes a seed reaches depends on its draws; the union over the seeds is all three


@pytest.mark.parametrize("seed", range(4))
def test_batched_path_on_random_shapes(seed):
    """slim_mpq_gemm on random row counts, K, group sizes, bit maps and 17 to 700 tokens: ragged row blocks and token
    tiles (the output leaves through clipped tensor stores), whole tiles and cut ones (a long K on few tiles)."""
    from paper_2405_14917_b200 import binding as slim
    rng = np.random.default_rng(3000 + seed)
    for case in range(6):
        g = int(rng.choice([128, 128, 256, 512]))
        M = int(rng.integers(17, 701))
        long_k = case % 2 == 1                       # every other case: few row blocks, many groups
        L, x, ref = _random_layer(rng, g, M, max_k=16384 if long_k else 4096, max_tiles=24 if long_k else 160)
        ws = torch.zeros(L.workspace_bytes(M), dtype=torch.uint8, device="cuda")
        slim.workspace_init(ws)
        y = torch.full((M, L.N), float("nan"), dtype=torch.float16, device="cuda")
        for _ in range(2):                           # twice into the same workspace: its flags must come back to zero
            L.forward(torch.from_numpy(x).cuda(), ws, out=y)
        slim.workspace_status(ws)
        check_output(y.cpu().numpy(), ref, f"gemm seed {seed} case {case}: {L.N}x{L.K} g={g} M={M}")
