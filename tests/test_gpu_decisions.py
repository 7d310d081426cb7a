"""Decision kernels fed exactly the floats the oracle gets: results must be bit-identical."""
import numpy as np
import pytest
import torch

from oracle import depcap_oracle as O
from paper_2604_15750_b200 import Hyper, inputs

from parity import Case

pytestmark = pytest.mark.gpu

WL = inputs.scaled(inputs.WORKLOADS["tiny_f32"], n_layers=0, batch=1)


def _engine(hyper, max_batch=32, max_window=128):
    case = Case(inputs.scaled(WL, ctx_min=0, ctx_max=0), n_layers=0, hyper=hyper)
    return case.make_engine(max_batch=max_batch, max_window=max_window, max_ctx=0)


def _ocfg(hp):
    return O.OracleConfig(n_layers=0, d_model=1, n_q_heads=1, n_kv_heads=1, head_dim=1, d_ff=1,
                          vocab=2, mask_id=1, lam=hp.lam, L_min=hp.L_min, L_max=hp.L_max,
                          smooth_radius=hp.smooth_radius, norm_mode=hp.norm_mode,
                          boundary_mode=hp.boundary_mode, cap_mode=hp.cap_mode)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("norm", [0, 1, 2])
@pytest.mark.parametrize("radius", [0, 1, 3])
def test_boundary_bit_exact(mode, norm, radius):
    hp = Hyper(boundary_mode=mode, norm_mode=norm, smooth_radius=radius, lam=1.2)
    eng = _engine(hp)
    r = np.random.default_rng(100 + 10 * mode + 3 * norm + radius)
    W, B = 128, 32
    for rep in range(8):
        win = r.integers(1, W + 1, B)
        remain = r.integers(1, 300, B)
        have = (r.random(B) < 0.9).astype(np.int32)
        I = (np.abs(r.standard_normal((B, W))) * np.exp(-np.arange(W) / r.uniform(2, 40))
             ).astype(np.float32)
        H = (r.random((B, W)) * r.uniform(0.1, 11)).astype(np.float32)
        if rep == 0:                       # adversarial: exact zeros, ties, tiny values
            I[:4] = 0.0
            H[4:8] = H[4:8, :1]
            I[8:12] *= 1e-30
            I[12:16] = H[12:16] * np.float32(1.2)
        out = eng.boundary(torch.from_numpy(I).cuda(), torch.from_numpy(H).cuda(), list(win),
                           list(remain), list(have))
        eng.synchronize()
        g = {k: v.cpu().numpy() for k, v in out.items()}
        for b in range(B):
            L, score, ci, cs = O.boundary(I[b], H[b], int(win[b]), int(remain[b]), bool(have[b]),
                                          _ocfg(hp))
            n = len(score)
            assert int(g["block_len"][b]) == L, (rep, b)
            assert np.array_equal(g["score"][b, :n].view(np.uint32), score.view(np.uint32))
            assert np.array_equal(g["cum_influence"][b, :n].view(np.uint32), ci.view(np.uint32))
            assert np.array_equal(g["cum_score"][b, :n].view(np.uint32), cs.view(np.uint32))
    eng.close()


@pytest.mark.parametrize("cap_mode", [0, 1])
def test_select_bit_exact(cap_mode):
    hp = Hyper(cap_mode=cap_mode)
    eng = _engine(hp)
    r = np.random.default_rng(7 + cap_mode)
    W, B = 128, 32
    mask_id = WL.mask_id
    total = 0
    for rep in range(12):
        win = r.integers(1, W + 1, B)
        blk = np.array([r.integers(0, w + 1) for w in win]).astype(np.int32)
        conf = r.random((B, W)).astype(np.float32)
        if rep % 3 == 0:
            conf = (0.6 + 0.4 * r.random((B, W))).astype(np.float32)          # big pools
        if rep % 4 == 1:
            conf = np.round(conf, 1).astype(np.float32)                        # many ties
            conf[:, ::7] = np.float32(0.8); conf[:, ::11] = np.float32(0.95)   # on thresholds
        x = (r.standard_normal((B, W, W)) * 6 - 9).astype(np.float32)
        if rep % 4 == 2:
            x[:, :, :] = np.float32(-8.0)                                      # D == gamma exactly
        ids = np.where(r.random((B, W)) < 0.8, mask_id, 5).astype(np.int32)
        out = eng.select(torch.from_numpy(ids).cuda(), list(win),
                         conf=torch.from_numpy(conf).cuda(), xlogp=torch.from_numpy(x).cuda(),
                         block_len=torch.from_numpy(blk).cuda())
        eng.synchronize()
        g = {k: v.cpu().numpy() for k, v in out.items()}
        for b in range(B):
            w = int(win[b])
            want = O.cap_select(conf[b, :w], ids[b, :w] == mask_id, x[b, :w, :w], int(blk[b]),
                                hp.tau_low, hp.tau_high, hp.gamma, cap_mode)
            n = int(g["sel_count"][b])
            assert list(g["sel_idx"][b, :n]) == want, (rep, b)
            assert [i for i in range(w) if g["sel_mask"][b, i]] == want
            total += n
    assert total > 500
    eng.close()


def test_select_threshold_override_reduces_to_the_baselines():
    eng = _engine(Hyper())
    r = np.random.default_rng(3)
    W, B = 64, 4
    conf = r.random((B, 128)).astype(np.float32)
    x = (r.standard_normal((B, 128, 128)) * 6 - 9).astype(np.float32)
    ids = np.full((B, 128), WL.mask_id, dtype=np.int32)
    blk = np.full(B, W, dtype=np.int32)
    args = dict(conf=torch.from_numpy(conf).cuda(), xlogp=torch.from_numpy(x).cuda(),
                block_len=torch.from_numpy(blk).cuda())
    # tau_low above 1: one token per step, the most confident one
    g = eng.select(torch.from_numpy(ids).cuda(), [W] * B, thresholds=(1.5, 2.0, -16.0), **args)
    eng.synchronize()
    assert list(g["sel_count"].cpu().numpy()[:B]) == [1] * B
    assert list(g["sel_idx"][:B, 0].cpu().numpy()) == list(conf[:, :W].argmax(axis=1))
    # gamma = +inf: plain confidence thresholding at 0.9
    g = eng.select(torch.from_numpy(ids).cuda(), [W] * B, thresholds=(0.9, 0.95, float("inf")),
                   **args)
    eng.synchronize()
    m = g["sel_mask"].cpu().numpy()[:B, :W]
    assert np.array_equal(m.astype(bool), conf[:, :W] >= np.float32(0.9))
    eng.close()


def test_batched_decisions_8192_sequences_bit_exact_on_a_sample():
    """dc_boundary_batched / dc_select_batched over 8192 sequences with device-side length
    arrays (the shape bench.py --mode decisions times): 96 sampled sequences, bit for bit."""
    hp = Hyper()
    eng = _engine(hp, max_batch=1, max_window=128)
    r = np.random.default_rng(2024)
    W, B = 128, 8192
    mask_id = WL.mask_id
    win = r.integers(1, W + 1, B).astype(np.int32)
    remain = r.integers(1, 300, B).astype(np.int32)
    have = (r.random(B) < 0.9).astype(np.int32)
    I = (np.abs(r.standard_normal((B, W))) * np.exp(-np.arange(W) / 16.0)).astype(np.float32)
    H = (r.random((B, W)) * 8).astype(np.float32)
    conf = np.where(r.random((B, W)) < 0.5, 0.9 + 0.1 * r.random((B, W)), r.random((B, W))).astype(np.float32)
    x = (r.standard_normal((B, W, W)) * 6 - 12).astype(np.float32)
    ids = np.where(r.random((B, W)) < 0.8, mask_id, 5).astype(np.int32)
    dev = eng.device
    t = lambda a: torch.from_numpy(a).to(dev)
    bo = dict(score=torch.zeros((B, W), device=dev), cum_influence=torch.zeros((B, W), device=dev),
              cum_score=torch.zeros((B, W), device=dev),
              block_len=torch.zeros((B,), dtype=torch.int32, device=dev))
    eng.boundary_batched(t(I), t(H), t(win), t(remain), bo, have_prev=t(have))
    so = dict(sel_mask=torch.zeros((B, W), dtype=torch.uint8, device=dev),
              sel_idx=torch.zeros((B, W), dtype=torch.int32, device=dev),
              sel_count=torch.zeros((B,), dtype=torch.int32, device=dev))
    eng.select_batched(t(conf), t(ids), t(x), bo["block_len"], t(win), so)
    eng.synchronize()
    g = {k: v.cpu().numpy() for k, v in {**bo, **so}.items()}
    picked = 0
    for b in list(range(32)) + list(r.integers(0, B, 62)) + [B - 2, B - 1]:
        L, score, ci, cs = O.boundary(I[b], H[b], int(win[b]), int(remain[b]), bool(have[b]), _ocfg(hp))
        n = len(score)
        assert int(g["block_len"][b]) == L, b
        assert np.array_equal(g["score"][b, :n].view(np.uint32), score.view(np.uint32))
        assert np.array_equal(g["cum_score"][b, :n].view(np.uint32), cs.view(np.uint32))
        w = int(win[b])
        want = O.cap_select(conf[b, :w], ids[b, :w] == mask_id, x[b, :w, :w], L, hp.tau_low,
                            hp.tau_high, hp.gamma, hp.cap_mode)
        cnt = int(g["sel_count"][b])
        assert list(g["sel_idx"][b, :cnt]) == want, b
        picked += cnt
    assert picked > 96
    eng.close()
