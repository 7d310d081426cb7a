"""GPU parity of the decoding loop around the step: K / V export into the cache, the Eq. (2)
commit, and whole generations (tokens, block lengths, forward count) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import adapters
from oracle import depcap_oracle as O
from paper_2604_15750_b200 import DepCap, DepCapError, Hyper, inputs
from paper_2604_15750_b200.binding import DC_IMPL_SIMT

from parity import Case

pytestmark = pytest.mark.gpu

TINY = inputs.WORKLOADS["tiny_f32"]
LLADA = inputs.WORKLOADS["llada8b_b1"]


def _peaked(wl, hyper, scale=25.0, n_layers=None, **kw):
    case = Case(wl, ctx_from_oracle=(wl.dtype == "f32"), hyper=hyper, n_layers=n_layers, **kw)
    case.weights["lm_head"] = case.weights["lm_head"] * scale
    case.ow = adapters.weights_from_torch(case.weights)
    return case


def test_commit_matches_eq2_bit_exactly():
    case = Case(TINY, ctx_from_oracle=False)
    eng = case.make_engine(max_batch=3, max_window=32)
    g = torch.Generator().manual_seed(5)
    B, MW, mask = 3, 32, TINY.mask_id
    win = torch.randint(0, 100, (B, MW), dtype=torch.int32, generator=g)
    win[torch.rand((B, MW), generator=g) < 0.6] = mask
    pred = torch.randint(100, 200, (B, MW), dtype=torch.int32, generator=g)
    sel = (torch.rand((B, MW), generator=g) < 0.5).to(torch.uint8)
    blk = torch.tensor([9, 32, 0], dtype=torch.int32)
    win_len = [20, 32, 7]
    d = eng.device
    win_d = win.to(d)
    rem = eng.commit(win_d, win_len, pred.to(d), sel.to(d), blk.to(d))
    eng.synchronize()
    exp = win.clone()
    left = []
    for b in range(B):
        L = min(int(blk[b]), win_len[b])
        for i in range(L):
            if exp[b, i] == mask and sel[b, i]:
                exp[b, i] = pred[b, i]
        left.append(int((exp[b, :L] == mask).sum()))
    assert torch.equal(win_d.cpu(), exp)
    assert rem.cpu().tolist() == left
    eng.close()


@pytest.mark.parametrize("impl", [0, DC_IMPL_SIMT])
def test_export_kv_appends_the_last_block_to_the_cache(impl):
    """bf16, two layers of the LLaDA-8B shape: fused-chain path and CUDA-core path."""
    wl = inputs.Workload("llada_small_ctx", 2, 4096, 32, 32, 128, 12288, 4096, "bf16", 1, 64, 64,
                         32, 64, 256, 4242)
    case = Case(wl)
    eng = case.make_engine(impl=impl, max_ctx=128)
    di = case.device_inputs(eng)
    k0, v0 = di["k_cache"].clone(), di["v_cache"].clone()
    eng.step(influence=True, boundary=True, export_kv=True, **di)
    eng.synchronize()
    kc, vc = di["k_cache"].float().cpu().numpy(), di["v_cache"].float().cpu().numpy()
    # untouched outside keys [64, 96)
    assert torch.equal(di["k_cache"][:, :, :, :64], k0[:, :, :, :64])
    assert torch.equal(di["k_cache"][:, :, :, 96:], k0[:, :, :, 96:])
    assert torch.equal(di["v_cache"][..., :64], v0[..., :64])
    assert torch.equal(di["v_cache"][..., 96:], v0[..., 96:])
    ora = O.step(case.ocfg, case.ow, adapters.to_np(case.k_log[:, 0]),
                 adapters.to_np(case.v_log[:, 0]), 64, case.last_ids[0, :32].numpy(),
                 case.win_ids[0, :64].numpy(), 256, return_kv=True)
    for l in range(2):
        k_ref, v_ref = ora["kv_last"][l]                       # [32, nkv, hd]
        k_gpu = np.transpose(kc[l, 0, :, 64:96, :], (1, 0, 2))
        v_gpu = np.transpose(vc[l, 0, :, :, 64:96], (2, 0, 1))
        for got, ref in ((k_gpu, k_ref), (v_gpu, v_ref)):
            err = np.abs(got - ref).max() / max(np.abs(ref).max(), 1.0)
            assert err <= 2e-2, (l, err)
    if impl == 0:       # the fused dense chain ran: one launch to start plus one per layer
        _, launches = eng.step_profiled(export_kv=True, **di)
        assert launches["dense"] == 3
    eng.close()


def test_export_kv_rejects_a_full_cache():
    case = Case(TINY, ctx_from_oracle=False)
    eng = case.make_engine()            # max_ctx 64 = ctx_len: no room for the last block
    di = case.device_inputs(eng)
    with pytest.raises(DepCapError) as e:
        eng.step(influence=True, boundary=True, export_kv=True, **di)
    assert "max_ctx" in str(e.value)
    eng.close()


@pytest.mark.parametrize("lam,norm", [(0.8, 2), (0.3, 1)])
def test_generation_fp32_matches_the_oracle(lam, norm):
    """Whole generations on the fp32 model: identical tokens, block lengths and forward count."""
    hy = Hyper(tau_low=0.3, tau_high=0.6, lam=lam, norm_mode=norm, L_min=4, L_max=16)
    case = _peaked(TINY, hy)
    N = 48
    ref = O.generate(case.ocfg, case.ow, adapters.to_np(case.k_log[:, 0]),
                     adapters.to_np(case.v_log[:, 0]), 64, N, 32)
    assert len(set(ref["block_lens"])) > 1 and ref["nfe"] < N     # adaptive and parallel
    eng = case.make_engine(max_ctx=128, max_last=16, max_window=32)
    di = case.device_inputs(eng)
    tok, blocks, nfe = eng.generate(di["k_cache"], di["v_cache"], [64], N)
    assert blocks[0] == ref["block_lens"]
    assert tok[0].tolist() == ref["tokens"].tolist()
    assert nfe == ref["nfe"]
    eng.close()


@pytest.mark.parametrize("lam,norm", [(0.02, 2), (0.3, 1)])
def test_generation_with_carried_prev_matches_the_oracle(lam, norm):
    """The same generations with p_prev carried from boundary step to boundary step (one variant
    through the stack): identical tokens, block lengths and forward count."""
    hy = Hyper(tau_low=0.3, tau_high=0.6, lam=lam, norm_mode=norm, L_min=4, L_max=16)
    case = _peaked(TINY, hy)
    N = 48
    ref = O.generate(case.ocfg, case.ow, adapters.to_np(case.k_log[:, 0]),
                     adapters.to_np(case.v_log[:, 0]), 64, N, 32, carried=True)
    assert len(set(ref["block_lens"])) > 1
    eng = case.make_engine(max_ctx=128, max_last=16, max_window=32)
    di = case.device_inputs(eng)
    tok, blocks, nfe = eng.generate(di["k_cache"], di["v_cache"], [64], N, carried_prev=True)
    assert blocks[0] == ref["block_lens"]
    assert tok[0].tolist() == ref["tokens"].tolist()
    assert nfe == ref["nfe"]
    eng.close()


def test_generation_batch_of_independent_sequences():
    """Two sequences with different contexts advance independently: each equals its own
    single-sequence oracle run; NFE is the longer of the two."""
    hy = Hyper(tau_low=0.3, tau_high=0.6, lam=0.8, norm_mode=2, L_min=4, L_max=16)
    wl = inputs.Workload("tiny_f32_b2", 2, 256, 4, 4, 64, 1024, 4096, "f32", 2, 40, 64, 16, 32, 32,
                         TINY.seed + 50)
    case = _peaked(wl, hy)
    N = 32
    ctx = case.len["ctx_len"]
    refs = [O.generate(case.ocfg, case.ow, adapters.to_np(case.k_log[:, b]),
                       adapters.to_np(case.v_log[:, b]), ctx[b], N, 32) for b in range(2)]
    eng = case.make_engine(max_ctx=128, max_last=16, max_window=32)
    di = case.device_inputs(eng)
    tok, blocks, nfe = eng.generate(di["k_cache"], di["v_cache"], ctx, N)
    for b in range(2):
        assert blocks[b] == refs[b]["block_lens"]
        assert tok[b].tolist() == refs[b]["tokens"].tolist()
    assert nfe == max(r["nfe"] for r in refs)
    eng.close()


def test_generation_on_the_fused_chain_equals_the_same_steps_called_one_by_one():
    """bf16 LLaDA-8B shape (4 layers): dc_generate against a loop of dc_step / dc_select /
    dc_commit driven from Python - the same kernels, so the ids are identical - and the
    invariants of a generation."""
    hy = Hyper(tau_low=0.3, tau_high=0.6, lam=0.8, norm_mode=2, L_min=8, L_max=32)
    wl = inputs.Workload("llada_gen", 4, 4096, 32, 32, 128, 12288, 8192, "bf16", 1, 64, 64, 32, 64,
                         256, 777)
    case = _peaked(wl, hy, scale=8.0)
    N = 64
    eng = case.make_engine(max_ctx=128, max_last=32, max_window=64)
    di = case.device_inputs(eng)
    k1, v1 = di["k_cache"].clone(), di["v_cache"].clone()
    tok, blocks, nfe = eng.generate(di["k_cache"], di["v_cache"], [64], N)
    _, launches = eng.step_profiled(k1, v1, [64], torch.zeros((1, eng.max_last), dtype=torch.int32,
                                    device=eng.device), [0], torch.full((1, eng.max_window),
                                    wl.mask_id, dtype=torch.int32, device=eng.device), [64], [N])
    assert launches["dense"] == 5
    assert sum(blocks[0]) == N and not np.any(tok[0] == wl.mask_id)
    assert len(blocks[0]) <= nfe <= N
    # the same loop from Python
    dev, MW = eng.device, eng.max_window
    cache, done, last, steps, out, bl = 64, 0, [], 0, [], []
    win = torch.full((1, MW), wl.mask_id, dtype=torch.int32, device=dev)
    last_d = torch.zeros((1, eng.max_last), dtype=torch.int32, device=dev)
    while done < N:
        W = min(hy.L_max, MW, N - done)
        win[:] = wl.mask_id
        last_d[0, :len(last)] = torch.tensor(last, dtype=torch.int32, device=dev) if last else 0
        o = eng.step(k1, v1, [cache], last_d, [len(last)], win, [W], [N - done], influence=True,
                     boundary=True, export_kv=True)
        steps += 1
        eng.select(win, [W])
        rem = eng.commit(win, [W])
        eng.synchronize()
        L = int(o["block_len"][0])
        bl.append(L)
        cache += len(last)
        blk_len = o["block_len"].clone()
        while int(rem[0]) > 0:
            o = eng.step(k1, v1, [cache], last_d, [0], win, [L], [N - done], influence=False,
                         boundary=False)
            steps += 1
            eng.select(win, [L], block_len=blk_len)
            rem = eng.commit(win, [L], block_len=blk_len)
            eng.synchronize()
        last = win[0, :L].cpu().tolist()
        out += last
        done += L
    assert bl == blocks[0] and out == tok[0].tolist() and steps == nfe
    assert torch.equal(k1, di["k_cache"]) and torch.equal(v1, di["v_cache"])
    eng.close()
