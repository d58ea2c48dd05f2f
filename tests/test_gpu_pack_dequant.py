"""GPU parity, bit-exact: slim_pack_weights and slim_dequant against the oracle."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from tests.helpers import oracle_layer

pytestmark = pytest.mark.gpu


def _slim():
    from paper_2405_14917_b200 import binding
    return binding


def _rand_codes(rng, N, bits):
    return np.concatenate([rng.integers(0, 2**int(b), (N, 128), dtype=np.uint8) for b in bits], axis=1)


BITMAPS = {
    "all1": [1] * 4, "all2": [2] * 4, "all3": [3] * 4, "all4": [4] * 4,
    "alternating": [1, 4, 2, 3, 1, 4, 2, 3], "head_tail": [3, 3, 2, 2, 2, 2, 1, 1],
    "single_group": [3], "ragged86": ([1, 2, 3, 2] * 22)[:86],
}


@pytest.mark.parametrize("name", list(BITMAPS))
@pytest.mark.parametrize("N", [16, 48, 272])
def test_pack_bit_exact(name, N):
    slim = _slim()
    bits = np.array(BITMAPS[name], dtype=np.uint8)
    rng = np.random.default_rng(len(bits) * 1000 + N)
    K = 128 * len(bits)
    codes = _rand_codes(rng, N, bits)
    want = orc.pack(codes, bits)
    assert slim.packed_bytes(N, K, bits) == want.size
    # guard bands around the output: nothing outside the buffer may change
    buf = torch.full((want.size + 512,), 0xA5, dtype=torch.uint8, device="cuda")
    out = buf[256:256 + want.size]
    slim.pack_weights(torch.from_numpy(codes).cuda(), bits, out)
    torch.cuda.synchronize()
    got = buf.cpu().numpy()
    assert (got[:256] == 0xA5).all() and (got[256 + want.size:] == 0xA5).all()
    assert (got[256:256 + want.size] == want).all()


@pytest.mark.parametrize("name", list(BITMAPS))
@pytest.mark.parametrize("zero_kind", ["integer", "half"])
def test_dequant_bit_exact_random_params(name, zero_kind):
    slim = _slim()
    bits = np.array(BITMAPS[name], dtype=np.uint8)
    N, K, G = 80, 128 * len(bits), len(bits)
    rng = np.random.default_rng(7 * G + (zero_kind == "half"))
    codes = _rand_codes(rng, N, bits)
    # scales over many binades incl. subnormal results; zeros integer or half-integer
    scales = (np.exp(rng.uniform(-16, 4, (G, N))) * rng.choice([-1, 1], (G, N))).astype(np.float16)
    zmax = (2.0 ** bits.astype(np.float64))[:, None]
    zeros = np.floor(rng.random((G, N)) * zmax)
    if zero_kind == "half":
        zeros = zeros + 0.5
    zeros = zeros.astype(np.float16)
    want = orc.dequant_f16(codes, scales, zeros)
    packed = torch.from_numpy(orc.pack(codes, bits)).cuda()
    got = slim.dequant(packed, bits, torch.from_numpy(scales).cuda(), torch.from_numpy(zeros).cuda(), N, K).cpu().numpy()
    assert (got.view(np.uint16) == want.view(np.uint16)).all()


@pytest.mark.parametrize("N,K,avg", [(4096, 4096, 2), (1024, 4096, 3), (256, 11008, 2)])
def test_pack_and_dequant_on_config_layers(N, K, avg):
    """Config-shaped layers (several tiles, ragged group count 86), oracle-quantised."""
    slim = _slim()
    L = oracle_layer(N, K, avg, 1)
    want_packed = orc.pack(L["codes"], L["bits"])
    assert want_packed.size == N * K * avg // 8
    packed = slim.pack_weights(torch.from_numpy(L["codes"]).cuda(), L["bits"])
    assert (packed.cpu().numpy() == want_packed).all()
    W = slim.dequant(packed, L["bits"], torch.from_numpy(L["scales"]).cuda(), torch.from_numpy(L["zeros"]).cuda(), N, K)
    want = orc.dequant_f16(L["codes"], L["scales"], L["zeros"])
    assert (W.cpu().numpy().view(np.uint16) == want.view(np.uint16)).all()
    # run-to-run identical
    W2 = slim.dequant(packed, L["bits"], torch.from_numpy(L["scales"]).cuda(), torch.from_numpy(L["zeros"]).cuda(), N, K)
    assert torch.equal(W, W2)


def test_empty_inputs_are_noops():
    slim = _slim()
    bits = np.array([2, 3], dtype=np.uint8)
    assert slim.packed_bytes(0, 256, bits) == 0
    codes = torch.empty((0, 256), dtype=torch.uint8, device="cuda")
    packed = slim.pack_weights(codes, bits)
    assert packed.numel() == 0
