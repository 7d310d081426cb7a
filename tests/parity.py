"""Shared harness of the GPU parity tests: runs one block-step through the C-ABI binding and
through the CPU oracle on the same seeded inputs and compares them.

Tolerances (bf16 path: every GEMM input is rounded to bf16, fp32 accumulation on the GPU, fp64
in the oracle; fp32 path: no rounding):
  logit-like values (lse, xlogp), confidence, entropy : max relative error 2e-2 (bf16) / 1e-4 (f32)
                                                         with denominator max(|ref|, 1)
  influence I_k                                         : 1e-3 absolute where the LM-head inputs
      are the same bits on both sides (fp32 model, or steered LM-head input): then only the fp32
      accumulation of the KL sum differs.  Through a bf16 stack the logits themselves differ
      (they are allowed 2e-2 relative), and I_k, a difference of two log-probability sets,
      inherits that: 1e-3 + 2e-2 * max_k I_k.
Integer outputs (token ids, block length, selected subset) must be identical unless the deciding
score lies within the float tolerance of its threshold; those cases are counted and returned.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import adapters
from oracle import depcap_oracle as O
from paper_2604_15750_b200 import DepCap, Hyper, inputs, pack_kv_cache


def oracle_cfg(wl, hyper: Hyper, n_layers=None):
    return adapters.config_from_workload(
        wl, n_layers=wl.n_layers if n_layers is None else n_layers, lam=hyper.lam,
        L_min=hyper.L_min, L_max=hyper.L_max, tau_low=hyper.tau_low, tau_high=hyper.tau_high,
        gamma=hyper.gamma, smooth_radius=hyper.smooth_radius, norm_mode=hyper.norm_mode,
        boundary_mode=hyper.boundary_mode, cap_mode=hyper.cap_mode,
        forbid_mask_pred=hyper.forbid_mask_pred)


def oracle_prefix_kv(ocfg, ow, prompt_ids):
    """Context cache made by the oracle's own forward over the prompt alone (bidirectional)."""
    return O.prefill(ocfg, ow, np.asarray(prompt_ids))


class Case:
    """Inputs of one step for a workload, on CPU (torch) with numpy views for the oracle."""

    def __init__(self, wl, n_layers=None, lengths=None, n_decoded=0, ctx_from_oracle=False,
                 steer=None, hyper=Hyper(), device="cpu"):
        self.wl, self.hyper = wl, hyper
        self.n_layers = wl.n_layers if n_layers is None else n_layers
        self.weights = inputs.make_weights(wl, device=device, n_layers=self.n_layers)
        self.ow = adapters.weights_from_torch(self.weights)
        self.ocfg = oracle_cfg(wl, hyper, self.n_layers)
        L = inputs.make_lengths(wl)
        if lengths:
            for k_, v_ in lengths.items():
                L[k_] = torch.tensor(v_, dtype=torch.int32)
        self.len = {k_: [int(x) for x in v_] for k_, v_ in L.items()}
        toks = inputs.make_tokens(wl, n_decoded)
        self.last_ids, self.win_ids, self.prompt = toks["last_ids"], toks["win_ids"], toks["prompt"]
        B = wl.batch
        if wl.ctx_max == 0:
            self.k_log = self.v_log = None
        elif ctx_from_oracle:
            ks, vs = [], []
            for b in range(B):
                k, v = oracle_prefix_kv(self.ocfg, self.ow, self.prompt[b, :wl.ctx_max].numpy())
                ks.append(k); vs.append(v)
            dt = wl.torch_dtype
            self.k_log = torch.from_numpy(np.stack(ks, 1)).to(dt)      # [L, B, nkv, P, hd]
            self.v_log = torch.from_numpy(np.stack(vs, 1)).to(dt)
        else:
            self.k_log, self.v_log = inputs.make_ctx_kv(wl, device=device, n_layers=self.n_layers)
        self.steer = None
        if steer:
            self.steer = inputs.make_steering(wl, self.weights["lm_head"], profile=steer)

    # ---- oracle side ------------------------------------------------------------------
    def run_oracle(self, influence=True, seqs=None):
        outs = {}
        for b in (range(self.wl.batch) if seqs is None else seqs):
            P, Lb, W = self.len["ctx_len"][b], self.len["last_len"][b], self.len["win_len"][b]
            kc = vc = None
            if self.k_log is not None:
                kc = adapters.to_np(self.k_log[:, b])
                vc = adapters.to_np(self.v_log[:, b])
            hf = None
            if self.steer is not None:
                hf = (adapters.to_np(self.steer[b, 0, :W]), adapters.to_np(self.steer[b, 1, :W]))
            outs[b] = O.step(self.ocfg, self.ow, kc, vc, P, self.last_ids[b, :Lb].numpy(),
                             self.win_ids[b, :W].numpy(), self.len["remain_len"][b],
                             influence=influence, h_final=hf, n_layers=self.n_layers)
        return outs

    # ---- GPU side ---------------------------------------------------------------------
    def make_engine(self, impl=0, max_batch=None, max_window=None, max_last=None, max_ctx=None):
        dev = torch.device("cuda:0")
        wd = dict(embed=self.weights["embed"].to(dev), lm_head=self.weights["lm_head"].to(dev),
                  final_norm=self.weights["final_norm"].to(dev),
                  layers=[{k_: v_.to(dev) for k_, v_ in lw.items()}
                          for lw in self.weights["layers"]])
        eng = DepCap.from_workload(self.wl, wd, n_layers=self.n_layers, hyper=self.hyper,
                                   impl=impl, max_batch=max_batch, max_window=max_window,
                                   max_last=max_last if max_last is not None
                                   else max(self.wl.last_len, 1), max_ctx=max_ctx)
        return eng

    def device_inputs(self, eng, poison=False):
        dev = eng.device
        B = self.wl.batch
        kc = vc = None
        if self.k_log is not None:
            kc, vc = pack_kv_cache(self.k_log.to(dev), self.v_log.to(dev), eng.max_batch,
                                   eng.max_ctx)
            if poison:      # the cache beyond ctx_len may hold anything, NaN included
                for b in range(B):
                    P = self.len["ctx_len"][b]
                    kc[:, b, :, P:, :] = float("nan")
                    vc[:, b, :, :, P:] = float("nan")
                kc[:, B:] = float("nan"); vc[:, B:] = float("nan")
        last = torch.zeros((B, eng.max_last), dtype=torch.int32)
        last[:, :self.last_ids.shape[1]] = self.last_ids
        win = torch.full((B, eng.max_window), self.wl.mask_id, dtype=torch.int32)
        win[:, :self.win_ids.shape[1]] = self.win_ids
        hf = None
        if self.steer is not None:
            hf = torch.zeros((B, 2, eng.max_window, self.wl.d_model), dtype=self.wl.torch_dtype)
            hf[:, :, :self.steer.shape[2]] = self.steer
            hf = hf.to(dev)
        return dict(k_cache=kc, v_cache=vc, ctx_len=self.len["ctx_len"], last_ids=last.to(dev),
                    last_len=self.len["last_len"], win_ids=win.to(dev),
                    win_len=self.len["win_len"], remain_len=self.len["remain_len"], h_final=hf)

    def run_gpu(self, eng, influence=True, boundary=True, poison=False):
        di = self.device_inputs(eng, poison)
        out = eng.step(influence=influence, boundary=boundary, **di)
        sel = eng.select(di["win_ids"], di["win_len"])
        eng.synchronize()
        res = {k_: v_.cpu().numpy() for k_, v_ in out.items()}
        res.update({k_: v_.cpu().numpy() for k_, v_ in sel.items()})
        return res


def _rel(got, ref):
    return np.abs(got - ref) / np.maximum(np.abs(ref), 1.0)


def compare(case: Case, gpu: dict, ora: dict, rtol=None, check_boundary=True):
    """Element-wise comparison; returns counts of near-threshold disagreements."""
    wl, hp = case.wl, case.hyper
    rtol = rtol if rtol is not None else (1e-4 if wl.dtype == "f32" else 2e-2)
    near = dict(pred=0, block_len=0, subset=0)
    worst = dict(conf=0.0, entropy=0.0, lse=0.0, influence=0.0, xlogp=0.0)
    for b, o in ora.items():
        W = case.len["win_len"][b]
        assert gpu["status"][b] == 0
        z = o["logits"]
        # ---- token ids: identical unless the top-2 logits are within tolerance
        for k in range(W):
            gp, op = int(gpu["pred_id"][b, k]), int(o["pred"][k])
            if gp != op:
                gap = z[k, op] - z[k, gp]
                assert gap <= rtol * max(1.0, abs(z[k, op])), (b, k, gp, op, gap)
                near["pred"] += 1
        same = gpu["pred_id"][b, :W] == o["pred"]
        for name in ("conf", "entropy", "lse"):
            # conf/entropy/lse depend on the whole distribution, not on which of two near-tied
            # ids won, so they are compared everywhere
            e = _rel(gpu[name][b, :W], o[name]).max()
            worst[name] = max(worst[name], float(e))
            assert e <= rtol, (name, b, e)
        e = np.abs(gpu["influence"][b, :W] - o["influence"]).max()
        worst["influence"] = max(worst["influence"], float(e))
        same_inputs = wl.dtype == "f32" or case.steer is not None
        itol = 1e-3 if same_inputs else 1e-3 + rtol * float(np.max(o["influence"]))
        assert e <= itol, ("influence", b, e, itol)
        xg, xo = gpu["xlogp"][b, :W, :W], o["xlogp"]
        cols = np.where(same)[0]
        if len(cols):
            ex = xg[:, cols] - xo[:, cols]
            finite = np.isfinite(xo[:, cols])
            e = (np.abs(ex[finite]) / np.maximum(np.abs(xo[:, cols][finite]), 1.0)).max()
            worst["xlogp"] = max(worst["xlogp"], float(e))
            assert e <= rtol, ("xlogp", b, e)
        # ---- block length
        if check_boundary and len(o["score"]):
            # The score divides I and H by their window maxima, so an input error dI becomes
            # dI / max(I) in the score (random-init weights give I ~ 1e-5, where fp32 rounding of
            # the KL sum is already visible).  Bound the score error by the observed input errors.
            n = len(o["score"])
            dI = np.abs(gpu["influence"][b, :n] - o["influence"][:n]).max()
            dH = np.abs(gpu["entropy"][b, :n] - o["entropy"][:n]).max()
            Imax = max(float(np.max(o["influence"][:n])), 1e-8)
            Hmax = max(float(np.max(o["entropy"][:n])), 1e-8)
            if hp.norm_mode == 2:
                Imax = Hmax = 1.0
            sbound = 4.0 * (dI / Imax + hp.lam * dH / Hmax) + 1e-5
            Lg, Lo = int(gpu["block_len"][b]), int(o["block_len"])
            if Lg != Lo:
                lo, hi = min(Lg, Lo), max(Lg, Lo)
                s_ = o["score"][:hi + 1]
                assert np.abs(s_[lo:]).min() <= sbound or \
                    np.abs(o["cum_score"][lo:hi + 1]).min() <= sbound * max(1, hi), (b, Lg, Lo)
                near["block_len"] += 1
            elif o["influence"][:n].max() > 0:
                assert np.abs(gpu["score"][b, :n] - o["score"]).max() <= sbound, \
                    (b, np.abs(gpu["score"][b, :n] - o["score"]).max(), sbound)
        # ---- selected subset
        cnt = int(gpu["sel_count"][b])
        sel_g = sorted(int(i) for i in gpu["sel_idx"][b, :cnt])
        assert sel_g == [i for i in range(W) if gpu["sel_mask"][b, i]]
        # the oracle's subset for the GPU's block length (the subset depends on it)
        Lsel = int(gpu["block_len"][b])
        masked = case.win_ids[b, :W].numpy() == wl.mask_id
        sel_o = O.cap_select(o["conf"], masked, o["xlogp"], Lsel, hp.tau_low, hp.tau_high,
                             hp.gamma, hp.cap_mode)
        if sel_g != sel_o:
            c = o["conf"][:Lsel]
            D = (o["xlogp"] + o["xlogp"].T)[:Lsel, :Lsel]
            close_tau = min(np.abs(c - hp.tau_low).min() / hp.tau_low,
                            np.abs(c - hp.tau_high).min() / hp.tau_high) <= rtol
            close_gamma = np.abs(D[np.isfinite(D)] - hp.gamma).min() <= 2 * rtol
            cs = np.sort(c)
            close_sort = len(cs) > 1 and (np.diff(cs) / np.maximum(cs[1:], 1e-30)).min() <= rtol
            assert close_tau or close_gamma or close_sort or near["pred"] > 0, (b, sel_g, sel_o)
            near["subset"] += 1
        # structural checks that hold whatever the rounding did
        assert all(masked[i] and i < Lsel for i in sel_g)
        if masked[:Lsel].any():
            assert cnt >= 1
    return near, worst
