"""The bounded-wait path of the tensor-core kernels, taken on purpose without harming the GPU.

Every device-side wait (TMA / MMA barriers, the grid barrier, hand-over flags) gives up after a
limit, after which the kernel frees what it holds, returns normally and reports DC_ERR_TIMEOUT in
status[b].  The test hook DC_OPT_TEST_STALL_LMHEAD makes the LM-head kernel skip every load: no
copy and no MMA is in flight, every wait of the kernel is one that nothing will ever satisfy, and
with the limit lowered to 50 ms the step comes back at once.  Nothing traps, faults or spins without
a bound; the context must work again on the next call."""
import time

import numpy as np
import pytest

from paper_2604_15750_b200 import inputs
from paper_2604_15750_b200.binding import (DC_ERR_TIMEOUT, DC_OPT_TEST_STALL_LMHEAD,
                                           DC_OPT_WAIT_LIMIT_US, DepCapError)

from parity import Case

pytestmark = pytest.mark.gpu


def test_expired_wait_reports_timeout_and_the_context_stays_usable():
    wl = inputs.Workload("wait_limit", 2, 256, 2, 2, 128, 512, 2048, "bf16", 2, 40, 64, 16, 32, 64, 31337)
    case = Case(wl, steer="decay")
    eng = case.make_engine()
    ref = case.run_gpu(eng)                                   # a clean step first
    assert list(ref["status"][:2]) == [0, 0]
    try:
        eng.set_option(DC_OPT_WAIT_LIMIT_US, 50_000)
        eng.set_option(DC_OPT_TEST_STALL_LMHEAD, 1)
        t0 = time.perf_counter()
        out = case.run_gpu(eng)
        dt = time.perf_counter() - t0
        assert list(out["status"][:2]) == [DC_ERR_TIMEOUT, DC_ERR_TIMEOUT]
        assert dt < 5.0, dt                                   # 50 ms per wait, not the default 2 s
        # ids stay inside the vocabulary whatever the aborted kernel left behind
        W = wl.win_len
        assert ((out["pred_id"][:2, :W] >= 0) & (out["pred_id"][:2, :W] < wl.vocab)).all()
    finally:
        eng.set_option(DC_OPT_TEST_STALL_LMHEAD, 0)
        eng.set_option(DC_OPT_WAIT_LIMIT_US, 2_000_000)
    again = case.run_gpu(eng)                                 # same context, next call: clean
    assert list(again["status"][:2]) == [0, 0]
    for k in ref:
        if k == "sel_idx":      # only the first sel_count entries of a row are written
            for b in range(2):
                n = int(ref["sel_count"][b])
                assert np.array_equal(ref[k][b, :n], again[k][b, :n])
        else:
            assert np.array_equal(ref[k], again[k]), k
    with pytest.raises(DepCapError):
        eng.set_option(DC_OPT_WAIT_LIMIT_US, 5)               # below the allowed range
    with pytest.raises(DepCapError):
        eng.set_option(99, 1)
    eng.close()
