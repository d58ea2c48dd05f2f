"""slim_mpq_gemm_static: the batched layer for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: a plugin callback that is only
given input/output pointers and a stream, or a serving loop whose memory was all handed out at
start-up (an allocation there would stall the device or fail).  They have no workspace to pass, so
this entry point keeps its scratch inside the library.  The test drives it through the C ABI,
twice in a row on the same data (the scratch is shared and keeps the previous call's contents),
and checks the result against slim_mpq_gemm with an ordinary workspace.
"""
import numpy as np
import pytest
import torch

from tests.helpers import FRO_REL, MAX_ABS_REL

pytestmark = pytest.mark.gpu


def _layer(slim, N, K, M, seed):
    from paper_2405_14917_b200 import workloads as wl
    W, a = wl.make_weight_and_norms_device((seed, N, K), N, K, "cuda")
    L = slim.QuantLinear.from_weight(W, a, 3)
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    x = torch.randn((M, K), generator=g, device="cuda").half()
    return L, x


# the first shape is cut across CTAs (stream-K: partial tiles and flags live in the scratch),
# the second runs whole tiles and only touches the status word
@pytest.mark.parametrize("N,K,M", [(5120, 13824, 512), (1024, 1024, 300)])
def test_static_scratch_matches_workspace_entry_point_twice(N, K, M):
    from paper_2405_14917_b200 import binding as slim
    L, x = _layer(slim, N, K, M, seed=N + K + M)
    ws = slim.new_workspace(M, N, K, L.bits)
    want = slim.mpq_gemm(x, L.packed, L.bits, L.scales, L.zeros, N, ws)
    slim.workspace_status(ws)
    want = want.cpu().numpy().astype(np.float64)

    out = torch.empty((M, N), dtype=torch.float16, device="cuda")       # caller-owned output and status word
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for call in range(2):
        out.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        slim.mpq_gemm_static(x, L.packed, L.bits, L.scales, L.zeros, N, out, status)
        torch.cuda.synchronize()
        if call == 1:       # the first call on a device may make the driver load the module that holds the array
            assert torch.cuda.mem_get_info()[0] >= free_before, "the call took device memory"
        assert int(status.item()) == 0, f"call {call}: a device-side wait gave up"
        got = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all(), f"call {call}"
        assert np.abs(got - want).max() <= MAX_ABS_REL * np.abs(want).max(), f"call {call}"
        assert np.linalg.norm(got - want) <= FRO_REL * np.linalg.norm(want), f"call {call}"


def test_static_entry_point_validates_like_the_ordinary_one():
    from paper_2405_14917_b200 import binding as slim
    L, x = _layer(slim, 128, 256, 16, seed=5)
    out = torch.empty((16, 128), dtype=torch.float16, device="cuda")
    with pytest.raises(slim.SlimError) as e:                              # M <= 16 belongs to the decode path
        slim.mpq_gemm_static(x, L.packed, L.bits, L.scales, L.zeros, 128, out)
    assert e.value.status == -1
