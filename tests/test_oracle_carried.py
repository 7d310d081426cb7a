"""Pins of the carried-prev reading (p_prev from rows kept from an earlier pass)."""
import numpy as np

from oracle import adapters
from oracle import depcap_oracle as O
from paper_2604_15750_b200 import inputs

from parity import Case

TINY = inputs.WORKLOADS["tiny_f32"]


def _run(case, **kw):
    b = 0
    P, Lb, W = case.len["ctx_len"][b], case.len["last_len"][b], case.len["win_len"][b]
    return O.step(case.ocfg, case.ow, adapters.to_np(case.k_log[:, b]), adapters.to_np(case.v_log[:, b]),
                  P, case.last_ids[b, :Lb].numpy(), case.win_ids[b, :W].numpy(),
                  case.len["remain_len"][b], **kw)


def test_carrying_the_recomputed_rows_reproduces_the_recomputed_step():
    """If the carried rows are exactly the prev variant's LM-head inputs of this very step, the
    carried step is the recomputed step: same influence, scores, block length, subset."""
    case = Case(TINY, ctx_from_oracle=True)
    W = case.len["win_len"][0]
    ref = _run(case, influence=True)
    got = _run(case, carried=(ref["h_prev"], W))
    for key in ("influence", "entropy", "conf", "score", "xlogp"):
        assert np.array_equal(got[key], ref[key]), key
    assert got["block_len"] == ref["block_len"] and got["selected"] == ref["selected"]
    assert np.array_equal(got["pred"], ref["pred"])


def test_positions_without_a_carried_row_have_no_influence():
    case = Case(TINY, ctx_from_oracle=True)
    ref = _run(case, influence=True)
    n = 10
    got = _run(case, carried=(ref["h_prev"], n))
    assert np.array_equal(got["influence"][:n], ref["influence"][:n])
    assert np.all(got["influence"][n:] == 0)
    # S_k = -lambda * H~_k < 0 from position n on: the block cannot reach beyond it
    assert got["block_len"] <= max(n, case.ocfg.L_min)
    cold = _run(case, carried=(ref["h_prev"], 0))
    assert np.all(cold["influence"] == 0) and cold["block_len"] == case.ocfg.L_min
