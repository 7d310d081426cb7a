"""Parity at the full model widths of the benchmark configurations, in the launch configuration
bench.py times (fused dense chain at batch 1, per-op kernels at larger batches).

The oracle cannot run 32 layers of an 8B model in seconds, so the checks are split the way the
path factors:
  * the transformer stack: full widths and head counts, full context length, but 1-2 layers, every
    output against the oracle;
  * the LM head + signals + decisions at the full vocabulary: steered LM-head inputs, every
    position against the oracle (the oracle needs only the LM-head matrix for that);
  * the whole 32-layer step: properties that hold at any size (finite, in range, reproducible).
"""
import math

import numpy as np
import pytest
import torch

from paper_2604_15750_b200 import inputs

from parity import Case, compare

pytestmark = pytest.mark.gpu

LLADA = inputs.WORKLOADS["llada8b_b1"]
DREAM = inputs.WORKLOADS["dream7b_b4"]


def test_llada_widths_two_layers_match_the_oracle():
    """d 4096, 32 heads, MLP 12288, ctx 512, 96 rows per variant: the dense chain's real shapes
    (32 / 96 weight tiles, 4 K-splits, 5 key tiles); vocabulary cut to 8192 to keep the oracle's
    LM head short."""
    wl = inputs.scaled(LLADA, n_layers=2, vocab=8192)
    case = Case(wl)
    eng = case.make_engine()
    _, launches = eng.step_profiled(**case.device_inputs(eng))
    assert launches["dense"] == 3                      # the fused chain is what runs
    gpu, ora = case.run_gpu(eng), case.run_oracle()
    compare(case, gpu, ora)
    eng.close()


def test_dream_widths_grouped_heads_one_layer_chain_and_per_op():
    """d 3584, 28 query / 4 KV heads, MLP 18944 (148 tiles): batch 1 takes the chain, batch 4
    (768 rows, three column blocks) the per-op kernels."""
    for batch, fused in ((1, True), (4, False)):
        wl = inputs.scaled(DREAM, n_layers=1, vocab=4096, batch=batch, ctx_min=200, ctx_max=256)
        case = Case(wl)
        eng = case.make_engine()
        _, launches = eng.step_profiled(**case.device_inputs(eng))
        assert (launches["dense"] > 0) == fused
        gpu, ora = case.run_gpu(eng), case.run_oracle(seqs=[0, batch - 1])
        compare(case, gpu, ora)
        eng.close()


@pytest.mark.parametrize("batch,impl", [(1, 0), (4, 0), (2, 1)])
def test_qkv_projection_biases_chain_per_op_and_cuda_core(batch, impl):
    """Dream widths with biases on the q / k / v projections (added before the rotation): the
    fused chain (batch 1), the per-op tensor-core kernels (batch 4) and the CUDA-core kernels."""
    wl = inputs.scaled(inputs.WORKLOADS["dream7b_b4_bias"], n_layers=2 if batch == 1 else 1, vocab=4096,
                       batch=batch, ctx_min=100, ctx_max=128)
    case = Case(wl)
    assert "bq" in case.weights["layers"][0] and len(case.ow.bq) == case.n_layers
    eng = case.make_engine(impl=impl)
    _, launches = eng.step_profiled(**case.device_inputs(eng))
    assert (launches["dense"] > 0) == (batch == 1 and impl == 0)
    seqs = [0, batch - 1]
    ora = case.run_oracle(seqs=seqs)
    near, worst = compare(case, case.run_gpu(eng), ora,
                          label=f"dream widths, q/k/v biases, batch {batch}, impl {impl}")
    eng.close()
    # the biases matter at this scale: the oracle without them is far from the one with them
    ow = case.ow
    saved = (ow.bq, ow.bk, ow.bv)
    ow.bq, ow.bk, ow.bv = [], [], []
    o0 = case.run_oracle(seqs=[0])[0]
    ow.bq, ow.bk, ow.bv = saved
    assert np.abs(o0["lse"] - ora[0]["lse"]).max() > 1e-3


def test_full_vocabulary_lm_head_signals_and_decisions_match_the_oracle():
    """V = 126464, d = 4096, 64 positions x 2 variants, steered so that the distributions are
    shaped: every signal and the decisions against the oracle."""
    wl = inputs.scaled(LLADA, n_layers=1, ctx_min=64, ctx_max=64)   # one layer: the stack still runs
    case = Case(wl, steer="decay")
    eng = case.make_engine()
    _, launches = eng.step_profiled(**case.device_inputs(eng))
    assert launches["lmhead"] == 2 and launches["dense"] > 0     # tensor-core LM head + combine
    gpu, ora = case.run_gpu(eng), case.run_oracle()
    near, worst = compare(case, gpu, ora)
    assert (ora[0]["conf"] > 0.9).any()
    eng.close()


def test_influence_tolerance_tensor_core_accumulator_against_fp32_fma():
    """The same steered LM-head inputs (d_model 4096, logits up to about 15) through both LM heads:
    the CUDA-core one accumulates each logit with fp32 FMAs and must hold I_k to 1e-3 absolute; the
    tensor-core one is allowed the accumulator term d_model * 2^-24 * max |z| on top (its fp32
    accumulator drops the bits of every product below the running sum's last place)."""
    wl = inputs.scaled(LLADA, n_layers=1, vocab=8192, ctx_min=64, ctx_max=64, batch=2, win_len=128)
    case = Case(wl, steer="decay")
    errs = {}
    for impl in (1, 0):
        eng = case.make_engine(impl=impl)
        gpu = case.run_gpu(eng)
        eng.close()
        ora = case.run_oracle()
        errs[impl] = max(float(np.abs(gpu["influence"][b, :wl.win_len] - ora[b]["influence"]).max())
                         for b in range(wl.batch))
    zmax = max(float(np.abs(ora[b]["logits"][np.isfinite(ora[b]["logits"])]).max()) for b in range(wl.batch))
    assert errs[1] <= 1e-3, errs                                   # fp32 FMA accumulation
    assert errs[0] <= 1e-3 + wl.d_model * 2.0 ** -24 * zmax, (errs, zmax)
    import parity
    parity.REPORT.append(dict(label="I_k error, same steered inputs: CUDA-core vs tensor-core LM head",
                              seqs=wl.batch, near={}, worst=dict(cuda_core=float(f"{errs[1]:.3g}"),
                                                                 tensor_core=float(f"{errs[0]:.3g}"),
                                                                 max_logit=float(f"{zmax:.3g}"))))


def test_whole_32_layer_step_properties():
    """The benchmark's configuration itself: outputs are finite and in range, the step is
    reproducible bit for bit, the status word is clean."""
    wl = LLADA
    dev = torch.device("cuda:0")
    weights = inputs.make_weights(wl, device=dev)
    from paper_2604_15750_b200 import DepCap, pack_kv_cache
    eng = DepCap.from_workload(wl, weights)
    k_log, v_log = inputs.make_ctx_kv(wl, device=dev)
    kc, vc = pack_kv_cache(k_log, v_log, eng.max_batch, eng.max_ctx)
    toks = inputs.make_tokens(wl)
    lens = {k: [int(x) for x in v] for k, v in inputs.make_lengths(wl).items()}
    kw = dict(k_cache=kc, v_cache=vc, ctx_len=lens["ctx_len"], last_ids=toks["last_ids"].to(dev),
              last_len=lens["last_len"], win_ids=toks["win_ids"].to(dev), win_len=lens["win_len"],
              remain_len=lens["remain_len"])
    runs = []
    for _ in range(2):
        out = eng.step(**kw)
        sel = eng.select(kw["win_ids"], kw["win_len"])
        eng.synchronize()
        runs.append({k: v.cpu().numpy().copy() for k, v in {**out, **sel}.items()})
    a, b = runs
    W = wl.win_len
    for k in a:
        assert np.array_equal(a[k], b[k]), k                       # reproducible
    assert a["status"][0] == 0
    for k in ("conf", "entropy", "influence", "lse", "score"):
        assert np.isfinite(a[k][0, :W]).all(), k
    assert ((a["conf"][0, :W] > 0) & (a["conf"][0, :W] <= 1.0 + 1e-6)).all()
    assert (a["entropy"][0, :W] <= math.log(wl.vocab - 1) + 1e-3).all()
    assert (a["entropy"][0, :W] >= -1e-4).all() and (a["influence"][0, :W] >= 0).all()
    assert ((a["pred_id"][0, :W] >= 0) & (a["pred_id"][0, :W] < wl.vocab - 1)).all()   # never [MASK]
    assert 8 <= a["block_len"][0] <= W and 1 <= a["sel_count"][0] <= a["block_len"][0]
    # log p_i(yhat_i) = log c_i on the diagonal of the cross log-probabilities
    d = np.diagonal(a["xlogp"][0, :W, :W])
    assert np.abs(d - np.log(a["conf"][0, :W])).max() < 2e-2
    eng.close()
