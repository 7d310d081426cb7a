"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import depcap_oracle as O
from paper_2604_15750_b200 import DepCap, DepCapError, Hyper, inputs

from parity import Case, compare

pytestmark = pytest.mark.gpu

TINY = inputs.WORKLOADS["tiny_f32"]
# small bf16 transformer whose shapes only the CUDA-core kernels take (head_dim 64)
SMALL_BF16 = inputs.Workload("small_bf16", 2, 128, 4, 2, 64, 384, 1000, "bf16", 3, 40, 100, 12, 24,
                             64, 777)


def test_tiny_f32_whole_step_raw():
    """Configuration 1: fp32, context cache made by the oracle's own prefix pass."""
    case = Case(TINY, ctx_from_oracle=True)
    eng = case.make_engine()
    gpu, ora = case.run_gpu(eng), case.run_oracle()
    near, worst = compare(case, gpu, ora)
    assert near == dict(pred=0, block_len=0, subset=0)
    # full logits of both variants agree too (debug entry of the CUDA-core LM head)
    for v, key in ((0, "logits"), (1, "logits_prev")):
        z = eng.debug_logits(v).cpu().numpy()[0, :TINY.win_len]
        ref = ora[0][key]
        keep = np.isfinite(ref)
        assert np.abs(z[keep] - ref[keep]).max() <= 1e-4
    eng.close()


@pytest.mark.parametrize("profile", ["decay", "bimodal"])
def test_tiny_f32_steered_decisions(profile):
    case = Case(TINY, ctx_from_oracle=True, steer=profile)
    eng = case.make_engine()
    gpu, ora = case.run_gpu(eng), case.run_oracle()
    near, worst = compare(case, gpu, ora)
    assert near["pred"] == 0
    # steering must exercise the decisions: confident positions exist and more than one commits
    assert (ora[0]["conf"] > 0.9).any() and len(ora[0]["selected"]) > 1
    eng.close()


def test_small_bf16_ragged_batch_grouped_heads_mid_block():
    """bf16 path, batch 3 with different context / last-block / window lengths, grouped KV heads,
    some window positions already decoded."""
    lengths = dict(ctx_len=[100, 40, 77], last_len=[12, 5, 0], win_len=[24, 17, 9],
                   remain_len=[64, 17, 30])
    case = Case(SMALL_BF16, lengths=lengths, n_decoded=4)
    eng = case.make_engine()
    gpu, ora = case.run_gpu(eng, poison=True), case.run_oracle()
    near, worst = compare(case, gpu, ora)
    assert int(gpu["block_len"][2]) == min(8, 9)          # sequence 2 has no last block
    assert np.all(gpu["influence"][2, :9] == 0)
    eng.close()


def test_small_bf16_steered():
    case = Case(SMALL_BF16, steer="decay")
    eng = case.make_engine()
    gpu, ora = case.run_gpu(eng), case.run_oracle()
    compare(case, gpu, ora)
    eng.close()


def test_without_influence_flag_and_without_context():
    wl = inputs.scaled(SMALL_BF16, batch=2, ctx_min=0, ctx_max=0)
    case = Case(wl)
    eng = case.make_engine(max_ctx=0)
    gpu = case.run_gpu(eng, influence=False)
    ora = case.run_oracle(influence=False)
    compare(case, gpu, ora)
    assert np.all(gpu["influence"][:, :wl.win_len] == 0)
    assert list(gpu["block_len"][:2]) == [8, 8]            # cold start: L = L_min
    eng.close()


def test_capacity_larger_than_the_step_and_window_of_one():
    wl = inputs.scaled(SMALL_BF16, batch=2)
    lengths = dict(ctx_len=[64, 1], last_len=[1, 12], win_len=[1, 24], remain_len=[1, 200])
    case = Case(wl, lengths=lengths)
    eng = case.make_engine(max_batch=5, max_window=48, max_last=16, max_ctx=128)
    gpu, ora = case.run_gpu(eng), case.run_oracle()
    compare(case, gpu, ora)
    assert int(gpu["block_len"][0]) == 1 and int(gpu["sel_count"][0]) == 1
    eng.close()


def test_two_identical_steps_are_bit_identical():
    case = Case(SMALL_BF16, steer="decay")
    eng = case.make_engine()
    a = case.run_gpu(eng)
    b = case.run_gpu(eng)
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    eng.close()


def test_argument_errors_are_reported_on_the_host_and_leave_outputs_untouched():
    case = Case(SMALL_BF16)
    eng = case.make_engine()
    di = case.device_inputs(eng)
    eng.out["pred_id"].fill_(-7)
    bad = dict(di); bad["win_len"] = [33, 24, 24]           # > max_window (32)
    with pytest.raises(DepCapError) as e:
        eng.step(**bad)
    assert e.value.code == 2 and "win_len" in str(e.value)
    bad = dict(di); bad["ctx_len"] = [100, 40, 10_000]
    with pytest.raises(DepCapError) as e:
        eng.step(**bad)
    assert e.value.code == 2
    bad = dict(di); bad["k_cache"] = None
    with pytest.raises(DepCapError) as e:
        eng.step(**bad)
    assert e.value.code == 1
    eng.synchronize()
    assert int(eng.out["pred_id"].min()) == -7 and int(eng.out["pred_id"].max()) == -7
    eng.step(**di)                                          # the context is still usable
    eng.synchronize()
    assert int(eng.out["status"].abs().max()) == 0
    eng.close()


def test_out_of_range_token_id_sets_the_status_word():
    case = Case(SMALL_BF16)
    eng = case.make_engine()
    di = case.device_inputs(eng)
    di["win_ids"][1, 3] = SMALL_BF16.vocab + 5
    eng.step(**di)
    eng.synchronize()
    st = eng.out["status"].cpu().numpy()
    assert st[1] == 7 and st[0] == 0 and st[2] == 0
    eng.close()


@pytest.mark.parametrize("tc", [False, True])
def test_non_finite_hidden_row_sets_the_status_word_and_keeps_the_id_in_range(tc):
    """A NaN LM-head input row (made on the host) has no finite logit: its argmax is undefined.
    The step must say so in status[b] and report an id inside the vocabulary (mask_id) instead of
    the argmax sentinel, which the cross log-prob kernel would otherwise use as a row index.
    Runs without the cross log-probs first, then with them; both CUDA-core and tensor-core LM head."""
    wl = inputs.Workload("nan_row", 1, 256, 2, 2, 128, 256, 3000, "bf16", 3, 32, 64, 16, 32, 64, 99) \
        if tc else SMALL_BF16
    case = Case(wl, steer="decay")
    eng = case.make_engine()
    di = case.device_inputs(eng)
    di["h_final"][1, 0, 5, :] = float("nan")
    for want in (False, True):
        eng.step(**di, want_xlogp=want)
        eng.synchronize()
        st = eng.out["status"].cpu().numpy()
        assert st[1] == 8 and st[0] == 0 and st[2] == 0
        pred = eng.out["pred_id"].cpu().numpy()
        assert pred[1, 5] == wl.mask_id
        for b in range(wl.batch):
            w = case.len["win_len"][b]
            assert ((pred[b, :w] >= 0) & (pred[b, :w] < wl.vocab)).all()
    # the context stays usable and clean inputs give a clean status
    clean = case.device_inputs(eng)
    eng.step(**clean)
    eng.synchronize()
    assert int(eng.out["status"].abs().max()) == 0
    eng.close()


def test_create_rejects_bad_configurations():
    case = Case(SMALL_BF16)
    with pytest.raises(DepCapError):
        case.make_engine(max_window=20)                     # not a multiple of 16
    with pytest.raises(DepCapError):
        case.make_engine(max_batch=64)
