"""GPU parity of DC_STEP_CARRIED_PREV: p_prev from rows carried over from an earlier step (one
variant through the stack), and of the h_out rows a step hands to the next."""
import numpy as np
import pytest
import torch

from oracle import adapters
from oracle import depcap_oracle as O
from paper_2604_15750_b200 import DepCapError, inputs
from paper_2604_15750_b200.binding import DC_IMPL_SIMT

from parity import Case, compare

pytestmark = pytest.mark.gpu

TINY = inputs.WORKLOADS["tiny_f32"]


def _oracle(case, b=0, **kw):
    P, Lb, W = case.len["ctx_len"][b], case.len["last_len"][b], case.len["win_len"][b]
    kc = adapters.to_np(case.k_log[:, b]) if case.k_log is not None else None
    vc = adapters.to_np(case.v_log[:, b]) if case.v_log is not None else None
    return O.step(case.ocfg, case.ow, kc, vc, P, case.last_ids[b, :Lb].numpy(),
                  case.win_ids[b, :W].numpy(), case.len["remain_len"][b], n_layers=case.n_layers, **kw)


def _gpu(case, eng, di, **kw):
    out = eng.step(**di, **kw)
    sel = eng.select(di["win_ids"], di["win_len"])
    eng.synchronize()
    res = {k_: v_.cpu().numpy() for k_, v_ in out.items()}
    res.update({k_: v_.cpu().numpy() for k_, v_ in sel.items()})
    return res


@pytest.mark.parametrize("n_prev", [32, 10, 0])
def test_carried_prev_fp32(n_prev):
    case = Case(TINY, ctx_from_oracle=True)
    ref_full = _oracle(case, influence=True)
    rows = ref_full["h_prev"]                                   # what an earlier pass would have left
    ora = _oracle(case, carried=(rows, n_prev))
    eng = case.make_engine()
    di = case.device_inputs(eng)
    di.pop("h_final")
    hp = torch.zeros((1, eng.max_window, TINY.d_model), dtype=torch.float32)
    hp[0, :rows.shape[0]] = torch.from_numpy(rows.astype(np.float32))
    h_out = torch.full((1, eng.max_window, TINY.d_model), float("nan"), dtype=torch.float32, device=eng.device)
    gpu = _gpu(case, eng, di, carried=(hp.to(eng.device), [n_prev]), h_out=h_out)
    near, _ = compare(case, gpu, {0: ora})
    assert near == dict(pred=0, block_len=0, subset=0)
    W = case.len["win_len"][0]
    assert np.all(gpu["influence"][0, n_prev:W] <= 1e-6)
    # the rows handed on are this step's curr LM-head inputs
    assert np.abs(h_out[0, :W].cpu().numpy() - ora["h_curr"]).max() <= 1e-4
    assert torch.isnan(h_out[0, W:]).all()
    eng.close()


@pytest.mark.parametrize("impl", [0, DC_IMPL_SIMT])
def test_carried_prev_bf16_rows_from_an_earlier_gpu_step(impl):
    """LLaDA widths, two layers: step 1 hands its rows out (h_out); step 2 - the next boundary
    step after a block of L = 8 - takes rows L.. as its p_prev.  96 rows through the fused chain
    (one variant) instead of 192."""
    wl = inputs.Workload("llada_carry", 2, 4096, 32, 32, 128, 12288, 4096, "bf16", 1, 64, 64, 32, 64,
                         256, 6061)
    case = Case(wl)
    eng = case.make_engine(impl=impl, max_ctx=128)
    dev = eng.device
    di = case.device_inputs(eng)
    di.pop("h_final")
    h_out = torch.zeros((1, eng.max_window, wl.d_model), dtype=torch.bfloat16, device=dev)
    eng.step(**di, influence=False, boundary=False, h_out=h_out)
    eng.synchronize()
    ora1 = _oracle(case, influence=False)
    err = np.abs(h_out[0, :64].float().cpu().numpy() - ora1["h_curr"]).max() / max(np.abs(ora1["h_curr"]).max(), 1.0)
    assert err <= 2e-2
    L, n_prev = 8, 64 - 8
    carried_gpu = torch.zeros_like(h_out)
    carried_gpu[0, :n_prev] = h_out[0, L:L + n_prev]
    # the oracle gets the same (GPU-made, bf16) rows: the comparison is of this step alone
    rows = carried_gpu[0, :n_prev].float().cpu().numpy().astype(np.float64)
    ora = _oracle(case, carried=(rows, n_prev))
    gpu = _gpu(case, eng, di, carried=(carried_gpu, [n_prev]))
    near, worst = compare(case, gpu, {0: ora})
    # random-init logits are nearly flat: a few of the 64 argmaxes are decided by a gap inside the
    # tolerance (compare() has checked each such gap) and follow the rounding order of the kernels
    assert near["pred"] <= 3
    if impl == 0:
        _, launches = eng.step_profiled(**di, carried=(carried_gpu, [n_prev]))
        assert launches["dense"] == 3          # the fused chain, on half the rows
    eng.close()


def test_carried_prev_argument_errors():
    case = Case(TINY, ctx_from_oracle=False)
    eng = case.make_engine()
    di = case.device_inputs(eng)
    di.pop("h_final")
    hp = torch.zeros((1, eng.max_window, TINY.d_model), dtype=torch.float32, device=eng.device)
    with pytest.raises(DepCapError) as e:
        eng.step(**di, carried=(hp, [33]))
    assert "prev_len" in str(e.value)
    eng.close()
