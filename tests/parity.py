"""Shared harness of the GPU parity tests: runs one block-step through the C-ABI binding and
through the CPU oracle on the same seeded inputs and compares them.

Tolerances (bf16 path: every GEMM input is rounded to bf16, fp32 accumulation on the GPU, fp64
in the oracle; fp32 path: no rounding):
  logit-like values (lse, xlogp), confidence, entropy : max relative error 2e-2 (bf16) / 1e-4 (f32)
                                                         with denominator max(|ref|, 1)
  influence I_k                                         : 1e-3 absolute where the LM-head inputs
      are the same bits on both sides (fp32 model, or steered LM-head input) and the logits are
      accumulated by fp32 FMAs (the CUDA-core LM head): then only the fp32 accumulation of the
      KL sum differs.  The tensor-core LM head accumulates d_model products per logit in the
      tensor core's fp32 accumulator, which aligns every product to the running sum and drops the
      bits below its last place instead of rounding: a logit z comes out low by up to about
      d_model * 2^-24 * |z| (measured: 2e-4 relative at d_model 4096), and I_k, a difference of
      logits and log-sum-exps, inherits up to that much of the largest logit:
      1e-3 + d_model * 2^-24 * max |z|.  Through a bf16 stack the logits themselves differ (they
      are allowed 2e-2 relative), and I_k inherits that: 1e-3 + 2e-2 * max_k I_k.
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
    def run_oracle(self, influence=True, seqs=None, pos0=None):
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
                             influence=influence, h_final=hf, n_layers=self.n_layers,
                             pos0=None if pos0 is None else pos0[b])
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


# One record per compare() call; tests/conftest.py prints them in the terminal summary so that the
# near-threshold counts and the worst errors are visible in a quiet run too.
REPORT: list[dict] = []


def _tc_lmhead(wl):
    """True when the tensor-core LM head serves this model shape (the library's own rule)."""
    return wl.dtype == "bf16" and wl.head_dim == 128 and wl.d_model % 128 == 0 and wl.d_ff % 128 == 0


def _tc_accumulator_term(wl, o):
    """What the tensor core's truncating fp32 accumulator may take off the largest logit (see the
    module docstring); 0 for the CUDA-core LM head."""
    if not _tc_lmhead(wl):
        return 0.0
    zmax = float(np.max(np.abs(o["logits"][np.isfinite(o["logits"])])))
    if o["logits_prev"] is not None:
        zmax = max(zmax, float(np.max(np.abs(o["logits_prev"][np.isfinite(o["logits_prev"])]))))
    return wl.d_model * 2.0 ** -24 * zmax


def _score_tolerance(case, o, n, itol, rtol):
    """How far S_k may move when I_k and H_k move by their own tolerances (itol absolute,
    rtol * max(H, 1)): smoothing averages, so it does not amplify; dividing by the window maximum
    (or the max - min range) turns an input error e into at most 2 e / denominator."""
    hp = case.hyper
    I, H = o["influence"][:n], o["entropy"][:n]
    htol = rtol * max(float(np.max(H)), 1.0)
    if hp.norm_mode == 2:
        dI = dH = 1.0
    elif hp.norm_mode == 1:
        dI = max(float(np.max(I) - np.min(I)), 1e-8)
        dH = max(float(np.max(H) - np.min(H)), 1e-8)
    else:
        dI = max(float(np.max(I)), 1e-8)
        dH = max(float(np.max(H)), 1e-8)
    return 2.0 * (itol / dI + hp.lam * htol / dH) + 1e-5


def compare(case: Case, gpu: dict, ora: dict, rtol=None, check_boundary=True, label=None):
    """Element-wise comparison of one step with the oracle.

    Floats: within the tolerances of the module docstring.  Integers (ids, block length, subset):
    two checks.  (1) In situ: the oracle's decision rules applied to the GPU's own float outputs
    must reproduce the GPU's decisions bit for bit - the decision kernels inside the whole step.
    (2) End to end against the oracle's decisions: identical unless the deciding score of THAT
    sequence lies within its tolerance of the threshold; such cases are counted in `near`.
    Returns (near, worst); also appended to REPORT."""
    wl, hp = case.wl, case.hyper
    rtol = rtol if rtol is not None else (1e-4 if wl.dtype == "f32" else 2e-2)
    near = dict(pred=0, block_len=0, subset=0)
    worst = dict(conf=0.0, entropy=0.0, lse=0.0, influence=0.0, influence_tol=0.0, xlogp=0.0,
                 score_tol=0.0)
    for b, o in ora.items():
        W = case.len["win_len"][b]
        assert gpu["status"][b] == 0
        z = o["logits"]
        # ---- token ids: identical unless the top-2 logits are within tolerance
        near_pos = []
        for k in range(W):
            gp, op = int(gpu["pred_id"][b, k]), int(o["pred"][k])
            if gp != op:
                gap = z[k, op] - z[k, gp]
                assert gap <= rtol * max(1.0, abs(z[k, op])), (b, k, gp, op, gap)
                near["pred"] += 1
                near_pos.append(k)
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
        itol = 1e-3 + _tc_accumulator_term(wl, o)
        if not same_inputs:
            itol += rtol * float(np.max(o["influence"]))
        worst["influence_tol"] = max(worst["influence_tol"], itol)
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
        have_prev = o["logits_prev"] is not None
        if check_boundary and len(o["score"]):
            n = len(o["score"])
            Lg, Lo = int(gpu["block_len"][b]), int(o["block_len"])
            # (1) in situ: the boundary rule on the GPU's own I_k, H_k, bit for bit
            Li, si, ci, csi = O.boundary(gpu["influence"][b, :W], gpu["entropy"][b, :W], W,
                                         case.len["remain_len"][b], have_prev, case.ocfg)
            assert Li == Lg, ("block_len in situ", b, Lg, Li)
            assert np.array_equal(si, gpu["score"][b, :n]), ("score in situ", b)
            assert np.array_equal(ci, gpu["cum_influence"][b, :n]), ("cum_influence in situ", b)
            assert np.array_equal(csi, gpu["cum_score"][b, :n]), ("cum_score in situ", b)
            # (2) against the oracle's own decision
            if have_prev:
                stol = _score_tolerance(case, o, n, itol, rtol)
                worst["score_tol"] = max(worst["score_tol"], stol)
                cum = hp.boundary_mode == 1
                dec_o = o["cum_score"] if cum else o["score"]
                dec_g = gpu["cum_score"][b, :n] if cum else gpu["score"][b, :n]
                if Lg != Lo:
                    # the first position where the two sides disagree on "negative" decides
                    flips = np.where((dec_o < 0) != (dec_g < 0))[0]
                    assert len(flips), (b, Lg, Lo)
                    kd = int(flips[0])
                    assert abs(float(dec_o[kd])) <= stol * ((kd + 1) if cum else 1), \
                        ("block_len", b, Lg, Lo, kd, float(dec_o[kd]), stol)
                    near["block_len"] += 1
                else:
                    e = np.abs(gpu["score"][b, :n] - o["score"]).max()
                    assert e <= stol, ("score", b, e, stol)
            else:
                assert Lg == Lo, (b, Lg, Lo)
        # ---- selected subset
        cnt = int(gpu["sel_count"][b])
        sel_g = sorted(int(i) for i in gpu["sel_idx"][b, :cnt])
        assert sel_g == [i for i in range(W) if gpu["sel_mask"][b, i]]
        Lsel = int(gpu["block_len"][b])
        masked = case.win_ids[b, :W].numpy() == wl.mask_id
        # (1) in situ: Algorithm 1 on the GPU's own c_i and cross log-probs, bit for bit
        sel_i = O.cap_select(gpu["conf"][b, :W], masked, gpu["xlogp"][b, :W, :W], Lsel, hp.tau_low,
                             hp.tau_high, hp.gamma, hp.cap_mode)
        assert sel_g == sel_i, ("subset in situ", b, sel_g, sel_i)
        # (2) against the oracle's subset for the same block length (the subset depends on it)
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
            # a near-tied id inside this sequence's block changes a column of its D matrix
            tied_id = any(k < Lsel for k in near_pos)
            assert close_tau or close_gamma or close_sort or tied_id, (b, sel_g, sel_o)
            near["subset"] += 1
        # structural checks that hold whatever the rounding did
        assert all(masked[i] and i < Lsel for i in sel_g)
        if masked[:Lsel].any():
            assert cnt >= 1
    REPORT.append(dict(label=label or wl.name, seqs=len(ora), near=dict(near),
                       worst={k: float(f"{v:.3g}") for k, v in worst.items()}))
    return near, worst


def lm_stage_strict(case: Case, eng, seqs=None):
    """The LM-head stage alone at the strict tolerances, on rows a real stack produced.

    Three GPU steps on the case's inputs: (A) the last block masked, one variant: its h_out rows
    are the prev variant's LM-head inputs; (B) one variant with the last block decoded and A's
    rows carried in as p_prev: the LM head of B sees exactly (h_out of B, h_out of A), both known
    bit for bit; (C) the ordinary two-variant step.  The oracle's signals on those same rows must
    match B: ids identical up to near-ties, c / H / lse within rtol, I_k within 1e-3 absolute plus
    the tensor-core accumulator term (tiny on these rows: random-init logits are below 1).  Returns the worst errors of B against the oracle
    and the largest |I_k(C) - I_k(B)| (what running both variants in one pass changes)."""
    wl = case.wl
    rtol = 2e-2
    di = case.device_inputs(eng)
    di.pop("h_final")
    B, MW, d = wl.batch, eng.max_window, wl.d_model
    dev = eng.device
    mask_last = torch.full_like(di["last_ids"], wl.mask_id)
    hA = torch.zeros((B, MW, d), dtype=wl.torch_dtype, device=dev)
    eng.step(**{**di, "last_ids": mask_last}, influence=False, boundary=False, h_out=hA)
    hB = torch.zeros_like(hA)
    outB = {k: v.clone() for k, v in
            eng.step(**di, boundary=False, carried=(hA, di["win_len"]), h_out=hB).items()}
    outC = {k: v.clone() for k, v in eng.step(**di, influence=True, boundary=False).items()}
    eng.synchronize()
    worst = dict(conf=0.0, entropy=0.0, lse=0.0, influence=0.0, influence_two_variant=0.0, near_pred=0)
    for b in (range(B) if seqs is None else seqs):
        W = case.len["win_len"][b]
        hc = adapters.to_np(hB[b, :W].cpu())
        hp_ = adapters.to_np(hA[b, :W].cpu())
        z = O.logits_of(hc, case.ow.lm_head, case.ocfg)
        zp = O.logits_of(hp_, case.ow.lm_head, case.ocfg)
        pred, conf, ent, infl, lse, _ = O.signals_from_logits(z, zp)
        g = {k: outB[k][b, :W].cpu().numpy() for k in ("pred_id", "conf", "entropy", "influence", "lse")}
        for k in range(W):
            if int(g["pred_id"][k]) != int(pred[k]):
                gap = z[k, pred[k]] - z[k, int(g["pred_id"][k])]
                assert gap <= rtol * max(1.0, abs(z[k, pred[k]])), (b, k, gap)
                worst["near_pred"] += 1
        for name, ref in (("conf", conf), ("entropy", ent), ("lse", lse)):
            e = float(_rel(g[name], ref).max())
            worst[name] = max(worst[name], e)
            assert e <= rtol, (name, b, e)
        e = float(np.abs(g["influence"] - infl).max())
        worst["influence"] = max(worst["influence"], e)
        itol = 1e-3 + _tc_accumulator_term(wl, dict(logits=z, logits_prev=zp))
        worst["influence_tol"] = max(worst.get("influence_tol", 0.0), itol)
        assert e <= itol, ("influence, LM-head stage", b, e, itol)
        e2 = float(np.abs(outC["influence"][b, :W].cpu().numpy() - g["influence"]).max())
        worst["influence_two_variant"] = max(worst["influence_two_variant"], e2)
    REPORT.append(dict(label=(wl.name + " / LM-head stage on stack rows"), seqs=B,
                       near=dict(pred=worst["near_pred"]),
                       worst={k: float(f"{v:.3g}") for k, v in worst.items() if k != "near_pred"}))
    return worst
