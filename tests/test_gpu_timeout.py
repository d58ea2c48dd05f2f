"""GPU test of the device-side time-out path: a bounded wait that runs out is reported through the workspace
status word as SLIM_ERR_TIMEOUT, the word is cleared by the query, and the workspace and the context stay usable.
The wait that runs out belongs to a kernel made for this (slim_selftest_wait_timeout: a barrier that nothing
signals, a limit of a millisecond); no kernel of the hot path is starved or broken to get there."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as orc
from tests.helpers import check_output, oracle_layer

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_is_reported_once():
    from paper_2405_14917_b200 import binding as slim
    L = oracle_layer(256, 512, 2, 1)
    ws = slim.new_workspace(1, 256, 512, L["bits"])
    slim.workspace_status(ws)                                  # clean to begin with
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    slim.selftest_wait_timeout(ws, limit_us=1000)
    t1.record()
    with pytest.raises(slim.SlimError) as e:
        slim.workspace_status(ws)
    assert e.value.status == -6                                # SLIM_ERR_TIMEOUT
    assert 0.9 <= t0.elapsed_time(t1) <= 50.0                  # the kernel waited about the limit, then returned by itself
    slim.workspace_status(ws)                                  # reported once: the word is cleared
    # the same workspace serves an ordinary call afterwards
    packed = torch.from_numpy(orc.pack(L["codes"], L["bits"])).cuda()
    y = slim.mpq_gemv(torch.from_numpy(L["x"]).cuda(), packed, L["bits"], torch.from_numpy(L["scales"]).cuda(),
                      torch.from_numpy(L["zeros"]).cuda(), 256, ws)
    slim.workspace_status(ws)
    check_output(y.cpu().numpy(), orc.linear_f64(L["x"], L["codes"], L["scales"], L["zeros"]), "after a time-out")


def test_selftest_arguments_are_validated():
    from paper_2405_14917_b200 import binding as slim
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for bad in (0, 100001):
        with pytest.raises(slim.SlimError) as e:
            slim.selftest_wait_timeout(ws, limit_us=bad)
        assert e.value.status == -1
    with pytest.raises(slim.SlimError) as e:
        slim.selftest_wait_timeout(torch.zeros(64, dtype=torch.uint8, device="cuda"), limit_us=10)
    assert e.value.status == -4
