"""The expiry branch of the library's bounded device-side wait, exercised without starving any real pipeline:
a dedicated one-CTA kernel waits on a barrier that nothing arms, with nothing in flight, under a short limit."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import paper_2410_09687_b200 as moin
from gpu_util import DEV, assert_layer_close, oracle_layer, run_layer

pytestmark = pytest.mark.gpu


def test_wait_that_cannot_be_satisfied_gives_up_and_reports():
    moin.device_status_reset()
    assert moin.device_status()["timeout_flag"] == 0
    got = moin.selftest_bounded_wait(200)
    assert got["first_wait_returned_ok"] == 0          # the wait ran out instead of hanging
    assert got["second_wait_returned_ok"] == 0         # the other waiter left through the abort flag
    assert 200 <= got["waited_us"] < 200000            # it waited for the limit, not for the default 2 s
    st = moin.device_status()
    assert st["timeout_flag"] == 1 and st["timeout_site"] == 99
    # the context is intact: reset the flag, then a normal call through the same pipeline code is correct
    moin.device_status_reset()
    assert moin.device_status()["timeout_flag"] == 0
    case = mi.tiny_layer(seed=0)
    y, _ = run_layer(case, moin.PLAN_TILES)
    assert_layer_close(y, oracle_layer(case), "layer after an expired wait")
    assert moin.device_status()["timeout_flag"] == 0


def test_selftest_argument_checks():
    with pytest.raises(moin.MoinError, match="INVALID_ARG"):
        moin.selftest_bounded_wait(0)
    with pytest.raises(moin.MoinError, match="INVALID_ARG"):
        moin.selftest_bounded_wait(2_000_000)
