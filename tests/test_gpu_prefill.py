"""GPU parity of dc_prefill: the K / V a prompt leaves in the caches against the oracle's, on the
fp32 model, on the fused-chain path and on the per-op tensor-core path, and a block-step that then
runs over the GPU-made cache."""
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


def _unpack(kc, vc, b, n0, n1):
    """logical [L, nkv, n, hd] views of keys n0..n1 of sequence b from the packed caches"""
    k = kc[:, b, :, n0:n1, :].float().cpu().numpy()
    v = np.transpose(vc[:, b, :, :, n0:n1].float().cpu().numpy(), (0, 1, 3, 2))
    return k, v


def _relerr(got, ref):
    return np.abs(got - ref).max() / max(np.abs(ref).max(), 1.0)


def test_prefill_fp32_then_a_step_over_the_gpu_made_cache():
    case = Case(TINY, ctx_from_oracle=True)            # oracle-made cache: the expected values
    eng = case.make_engine(max_last=64, max_ctx=128)
    dev = eng.device
    L, nkv, hd = TINY.n_layers, TINY.n_kv_heads, TINY.head_dim
    dt = torch.float32
    kc = torch.full((L, 1, nkv, 128, hd), float("nan"), dtype=dt, device=dev)
    vc = torch.full((L, 1, nkv, hd, 128), float("nan"), dtype=dt, device=dev)
    ids = torch.zeros((1, eng.max_last), dtype=torch.int32)
    ids[0, :64] = case.prompt[0, :64]
    st = eng.prefill(kc, vc, ids.to(dev), [64])
    eng.synchronize()
    assert int(st[0]) == 0
    k, v = _unpack(kc, vc, 0, 0, 64)
    assert np.abs(k - adapters.to_np(case.k_log[:, 0])).max() <= 1e-4
    assert np.abs(v - adapters.to_np(case.v_log[:, 0])).max() <= 1e-4
    assert torch.isnan(kc[:, :, :, 64:]).all() and torch.isnan(vc[..., 64:]).all()   # nothing else written
    # the block-step of configuration 1 over this cache
    di = case.device_inputs(eng)
    di["k_cache"], di["v_cache"] = kc, vc
    out = eng.step(influence=True, boundary=True, **di)
    sel = eng.select(di["win_ids"], di["win_len"])
    eng.synchronize()
    gpu = {k_: v_.cpu().numpy() for k_, v_ in out.items()}
    gpu.update({k_: v_.cpu().numpy() for k_, v_ in sel.items()})
    near, _ = compare(case, gpu, case.run_oracle())
    assert near == dict(pred=0, block_len=0, subset=0)
    eng.close()


@pytest.mark.parametrize("impl,n_ids", [(0, [200, 137]), (0, [96, 64]), (DC_IMPL_SIMT, [40, 17])])
def test_prefill_bf16_ragged_batch_behind_a_context(impl, n_ids):
    """LLaDA widths, two layers, two sequences with different prompt lengths, 64 keys of context
    already cached: 337 rows take the per-op kernels, 160 rows the fused chain."""
    wl = inputs.Workload("llada_prefill", 2, 4096, 32, 32, 128, 12288, 4096, "bf16", 2, 64, 64,
                         max(n_ids), 16, 256, 5150)
    case = Case(wl)
    eng = case.make_engine(impl=impl, max_ctx=320, max_last=max(n_ids))
    dev = eng.device
    di = case.device_inputs(eng)
    kc, vc = di["k_cache"], di["v_cache"]
    k0, v0 = kc.clone(), vc.clone()
    g = torch.Generator().manual_seed(11)
    ids = torch.randint(0, wl.vocab - 1, (2, eng.max_last), dtype=torch.int32, generator=g)
    st = eng.prefill(kc, vc, ids.to(dev), n_ids, ctx_len=[64, 64])
    eng.synchronize()
    assert st.cpu().tolist()[:2] == [0, 0]
    for b in range(2):
        n = n_ids[b]
        k_ref, v_ref = O.prefill(case.ocfg, case.ow, ids[b, :n].numpy().astype(np.int64),
                                 adapters.to_np(case.k_log[:, b]), adapters.to_np(case.v_log[:, b]), 64)
        k, v = _unpack(kc, vc, b, 64, 64 + n)
        assert _relerr(k, k_ref) <= 2e-2 and _relerr(v, v_ref) <= 2e-2
        # the context and everything behind the prompt are untouched
        assert torch.equal(kc[:, b, :, :64], k0[:, b, :, :64]) and torch.equal(kc[:, b, :, 64 + n:], k0[:, b, :, 64 + n:])
        assert torch.equal(vc[:, b, :, :, :64], v0[:, b, :, :, :64]) and torch.equal(vc[:, b, :, :, 64 + n:], v0[:, b, :, :, 64 + n:])
    eng.close()


def test_prefill_rejects_what_does_not_fit():
    case = Case(TINY, ctx_from_oracle=False)
    eng = case.make_engine(max_last=32, max_ctx=64)
    dev = eng.device
    di = case.device_inputs(eng)
    ids = torch.zeros((1, 32), dtype=torch.int32, device=dev)
    with pytest.raises(DepCapError) as e:
        eng.prefill(di["k_cache"], di["v_cache"], ids, [33])
    assert "max_last" in str(e.value)
    with pytest.raises(DepCapError) as e:
        eng.prefill(di["k_cache"], di["v_cache"], ids, [32], ctx_len=[40])
    assert "max_ctx" in str(e.value)
    eng.close()


@pytest.mark.parametrize("tc", [False, True])
def test_dual_cache_suffix_rows_prefilled_at_their_own_positions(tc):
    """Prefix keys, then the still masked suffix behind the window prefilled with pos0 = P + W
    (cache slots P .. P + S - 1, positions P + W ...): the cache rows match the oracle's prefill
    with the same position argument, and a step over the window with that cache matches the
    oracle's step over [prefix ; suffix] context rows."""
    if tc:
        wl = inputs.Workload("dual_tc", 2, 256, 4, 2, 128, 512, 2048, "bf16", 1, 40, 40, 0, 32, 64, 4711)
        tol = 2e-2
    else:
        wl = inputs.scaled(TINY, last_len=0)
        tol = 1e-4
    P, Wn, S = 40, wl.win_len, 24
    case = Case(inputs.scaled(wl, ctx_min=P, ctx_max=P), lengths=dict(ctx_len=[P], last_len=[0]))
    eng = case.make_engine(max_last=64, max_ctx=128)
    dev = eng.device
    L, nkv, hd = wl.n_layers, wl.n_kv_heads, wl.head_dim
    dt = wl.torch_dtype
    kc = torch.zeros((L, 1, nkv, 128, hd), dtype=dt, device=dev)
    vc = torch.zeros((L, 1, nkv, hd, 128), dtype=dt, device=dev)
    prompt = case.prompt[0, :P]
    ids = torch.zeros((1, eng.max_last), dtype=torch.int32)
    ids[0, :P] = prompt
    eng.prefill(kc, vc, ids.to(dev), [P])
    suffix = torch.full((1, eng.max_last), wl.mask_id, dtype=torch.int32)
    st = eng.prefill(kc, vc, suffix.to(dev), [S], ctx_len=[P], pos0=[P + Wn])
    eng.synchronize()
    assert int(st[0]) == 0
    # oracle: the same two prefills
    k0, v0 = O.prefill(case.ocfg, case.ow, prompt.numpy(), n_layers=L)
    k1, v1 = O.prefill(case.ocfg, case.ow, np.full(S, wl.mask_id), k0, v0, ctx_len=P, n_layers=L, pos0=P + Wn)
    kg, vg = _unpack(kc, vc, 0, P, P + S)
    assert _relerr(kg, k1) <= tol and _relerr(vg, v1) <= tol
    # a step over the window whose context is prefix + suffix rows
    case.k_log = torch.from_numpy(np.concatenate([k0, k1], axis=2)[:, None]).to(dt)
    case.v_log = torch.from_numpy(np.concatenate([v0, v1], axis=2)[:, None]).to(dt)
    case.len["ctx_len"] = [P + S]
    di = case.device_inputs(eng)
    di["k_cache"], di["v_cache"] = kc, vc
    # the window sits at positions P ... (right behind the prefix), not behind all P + S cached keys
    out = eng.step(influence=False, boundary=True, pos0=[P], **di)
    sel = eng.select(di["win_ids"], di["win_len"])
    eng.synchronize()
    gpu = {k_: v_.cpu().numpy() for k_, v_ in out.items()}
    gpu.update({k_: v_.cpu().numpy() for k_, v_ in sel.items()})
    ora = case.run_oracle(influence=False, pos0=[P])
    compare(case, gpu, ora, label="dual cache: prefix + suffix context rows")
    # and the position does matter: the oracle with the default position is somewhere else
    off = case.run_oracle(influence=False)
    assert np.abs(off[0]["lse"] - ora[0]["lse"]).max() > 1e-4
    eng.close()
