#!/usr/bin/env python
"""Benchmark of the DepCap block-step on B200.

One "step" = one whole pass of the hot path over one batch of synthetic input:
dc_step (embedding, transformer stack over the cached context for the curr and prev variants,
LM head with the streaming softmax statistics, cross log-probs, block boundary) followed by
dc_select (CAP-Decoding).  Metric: committed tokens per second = sum_b |S_b| / step time, with
the block-step latency as ms_per_step.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

N > 1 runs N independent replicas (one process per GPU, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_15750_b200 import inputs, replicas  # noqa: E402

METRIC = "committed_tokens_per_s"
UNIT = "tokens/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def _kernel_hash():
    import hashlib
    h = hashlib.sha256()
    for f in ("tc_chain.cuh", "tc_ptx.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2604_15750_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def _traffic_record(workload):
    """DRAM traffic of one k_dense_chain launch (dram__bytes_read.sum + dram__bytes_write.sum of an
    ncu capture), read from the tracked summary of that capture: a line
    `bench-traffic: workload=<name> dram_bytes_per_launch=<bytes> kernel_sha256=<hash>` in
    profiles/dense_chain_<workload>.md.  None when there is no such line or the kernel sources
    have changed since the counters were taken."""
    import re
    path = os.path.join(ROOT, "profiles", f"dense_chain_{workload}.md")
    if not os.path.exists(path):
        return None
    m = re.search(r"bench-traffic:\s*workload=(\S+)\s+dram_bytes_per_launch=([0-9.eE+]+)\s+kernel_sha256=([0-9a-f]+)",
                  open(path).read())
    if not m or m.group(1) != workload or m.group(3) != _kernel_hash():
        return None
    return float(m.group(2))


def _layer_param_count(wl):
    hq, hkv = wl.n_q_heads * wl.head_dim, wl.n_kv_heads * wl.head_dim
    return wl.d_model * (hq + 2 * hkv) + hq * wl.d_model + 3 * wl.d_model * wl.d_ff


class ClockSampler:
    def __init__(self, index):
        self.path = f"/tmp/dc_clocks_{os.getpid()}.csv"
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.f = open(self.path, "w")
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                       "-i", str(index), "-lms", "50"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            out = dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


def _oracle_sample(wl, weights_dev, k_log, v_log, toks, lens, steer, n_head_pos=16, budget_s=None, prompt=None):
    """Times the CPU oracle, as it stands, on a bounded sample of the step for sequence 0:
    one transformer layer (curr and prev variants) over the first n_rows active rows and the LM
    head + signals on the first n_head_pos window positions; the full-step time is extrapolated
    (the layer cost is linear in the rows, the head cost in the positions).  budget_s shrinks the
    sample so that one call takes about that long (a full sample is about 5 s)."""
    import numpy as np
    from oracle import adapters
    from oracle import depcap_oracle as O
    one = dict(embed=weights_dev["embed"], lm_head=weights_dev["lm_head"],
               final_norm=weights_dev["final_norm"], layers=weights_dev["layers"][:1])
    ow = adapters.weights_from_torch(one)
    ocfg = adapters.config_from_workload(wl, n_layers=1)
    P, Lb, W = lens["ctx_len"][0], lens["last_len"][0], lens["win_len"][0]
    R = Lb + W
    n_rows = R
    if budget_s is not None:
        frac = min(1.0, budget_s / 5.0)
        n_rows = max(4, min(R, int(R * frac)))
        n_head_pos = max(2, min(n_head_pos, int(n_head_pos * frac)))
    kc = adapters.to_np(k_log[:1, 0]) if k_log is not None else None
    vc = adapters.to_np(v_log[:1, 0]) if v_log is not None else None
    if prompt is not None and P > 0:
        # the context cache of the sampled layer from the oracle's own prefill of the prompt (an
        # input of the step: not timed)
        kc, vc = O.prefill(ocfg, ow, prompt[0, :P].numpy(), n_layers=1)
    last = toks["last_ids"][0, :Lb].numpy()
    win = toks["win_ids"][0, :W].numpy()
    tok_curr = np.concatenate([last, win]).astype(np.int64)
    tok_prev = tok_curr.copy(); tok_prev[:Lb] = wl.mask_id
    t0 = time.perf_counter()
    O.forward(ocfg, ow, tok_curr[:n_rows], P, kc[:, :, :P] if kc is not None else None,
              vc[:, :, :P] if vc is not None else None, n_layers=1)
    O.forward(ocfg, ow, tok_prev[:n_rows], P, kc[:, :, :P] if kc is not None else None,
              vc[:, :, :P] if vc is not None else None, n_layers=1)
    t_layer = (time.perf_counter() - t0) * (R / n_rows)
    n = min(n_head_pos, W)
    hf = (adapters.to_np(steer[0, 0, :n]), adapters.to_np(steer[0, 1, :n]))
    t0 = time.perf_counter()
    O.step(ocfg, ow, None, None, 0, last, win[:n], lens["remain_len"][0], h_final=hf)
    t_head = time.perf_counter() - t0
    est = wl.n_layers * t_layer + t_head * (W / n)
    return dict(t_layer=t_layer, t_head=t_head, est_step_s=est * wl.batch,
                sample=f"sequence 0: 1 of {wl.n_layers} layers (curr+prev variants) on {n_rows} of {R} "
                       f"active rows + LM head/signals/decisions on {n} of {W} window positions; "
                       f"extrapolated to {wl.n_layers} layers, {R} rows, {W} positions, batch {wl.batch}")


def _oracle_committed(wl, weights_dev, toks, lens, steer, decisions=None):
    """Committed tokens of the full steered step by the oracle's decisions (not timed): the
    steering replaces the stack's output, so this needs the LM head only."""
    from oracle import adapters
    from oracle import depcap_oracle as O
    one = dict(embed=weights_dev["embed"][:1], lm_head=weights_dev["lm_head"],
               final_norm=weights_dev["final_norm"], layers=[])
    ow = adapters.weights_from_torch(one)
    ocfg = adapters.config_from_workload(wl, n_layers=0)
    total = 0
    per_seq = []
    for b in range(wl.batch):
        Lb, W = lens["last_len"][b], lens["win_len"][b]
        hf = (adapters.to_np(steer[b, 0, :W]), adapters.to_np(steer[b, 1, :W]))
        o = O.step(ocfg, ow, None, None, 0, toks["last_ids"][b, :Lb].numpy(),
                   toks["win_ids"][b, :W].numpy(), lens["remain_len"][b], h_final=hf)
        total += len(o["selected"])
        per_seq.append(dict(pred=o["pred"], block_len=int(o["block_len"]), selected=list(o["selected"])))
    if decisions is not None:
        decisions.extend(per_seq)
    return total


def _config(wl, n_layers, variants="curr+prev", ctx="prefill"):
    """The workload description; both arms print exactly this."""
    return dict(workload=wl.name, batch=wl.batch, ctx=wl.ctx_max, last_block=wl.last_len,
                window=wl.win_len, layers=n_layers, variants=variants, steering="decay",
                context=("K / V of the seeded prompt made by the model's own bidirectional prefill"
                         if ctx == "prefill" else "seeded N(0,1) K / V"),
                l2="inputs larger than L2 (weights streamed every step)")


def _setup(wl, dev, n_layers, noise_ctx=True):
    weights = inputs.make_weights(wl, device=dev, n_layers=n_layers)
    k_log, v_log = inputs.make_ctx_kv(wl, device=dev, n_layers=n_layers) if noise_ctx else (None, None)
    toks = inputs.make_tokens(wl)
    lens = {k: [int(x) for x in v] for k, v in inputs.make_lengths(wl).items()}
    steer = inputs.make_steering(wl, weights["lm_head"], profile="decay")
    return weights, k_log, v_log, toks, lens, steer


def run_reference(args, wl, rank, world):
    """The reference arm: the CPU oracle, as it stands, timed on the host cores."""
    if rank != 0:
        return
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    n_layers = args.layers or wl.n_layers
    wl1 = inputs.scaled(wl, n_layers=n_layers)
    weights = inputs.make_weights(wl, device=dev, n_layers=1)
    k_log, v_log = inputs.make_ctx_kv(inputs.scaled(wl, n_layers=1), device=dev, n_layers=1)
    toks = inputs.make_tokens(wl)
    lens = {k: [int(x) for x in v] for k, v in inputs.make_lengths(wl).items()}
    steer = inputs.make_steering(wl, weights["lm_head"], profile="decay")
    committed = _oracle_committed(wl, weights, toks, lens, steer)
    times = []
    sample = None
    budget = 150.0 / (args.warmup + args.steps)      # the whole run ends within a few minutes
    for i in range(args.warmup + args.steps):
        s = _oracle_sample(wl1, weights, k_log, v_log, toks, lens, steer, budget_s=budget,
                           prompt=toks["prompt"] if args.ctx == "prefill" else None)
        sample = s["sample"]
        if i >= args.warmup:
            times.append(s["est_step_s"])
    t = sum(times) / len(times)
    value = committed / t
    cores = torch.get_num_threads()
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=t * 1e3, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=_config(wl, n_layers, ctx=args.ctx), committed_per_step=committed,
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample,
                                  extrapolated=True),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def run_generate(args, wl, dev):
    """Block-wise generation of --gen-len tokens per sequence behind the workload's context
    (dc_generate: boundary step + denoising steps per block, host read-back every step)."""
    import time
    from paper_2604_15750_b200 import DepCap, pack_kv_cache
    n_layers = args.layers or wl.n_layers
    weights = inputs.make_weights(wl, device=dev, n_layers=n_layers)
    weights["lm_head"] = weights["lm_head"] * args.lm_scale
    k_log, v_log = inputs.make_ctx_kv(wl, device=dev, n_layers=n_layers)
    lens = {k: [int(x) for x in v] for k, v in inputs.make_lengths(wl).items()}
    N = args.gen_len
    max_ctx = (wl.ctx_max + N + 63) // 64 * 64
    eng = DepCap.from_workload(wl, weights, n_layers=n_layers, max_ctx=max_ctx,
                               max_last=max(wl.win_len, 16), max_window=(wl.win_len + 15) // 16 * 16)
    kc, vc = pack_kv_cache(k_log, v_log, eng.max_batch, eng.max_ctx)
    eng.generate(kc, vc, lens["ctx_len"], min(N, 32))           # warm-up
    eng.synchronize()
    t0 = time.perf_counter()
    tok, blocks, nfe = eng.generate(kc, vc, lens["ctx_len"], N)
    eng.synchronize()
    dt = time.perf_counter() - t0
    nb = [len(b) for b in blocks]
    print(json.dumps(dict(metric="generated_tokens_per_s", value=wl.batch * N / dt, unit="tokens/s",
                          n_gpus=1, mode="generate", ms=dt * 1e3, nfe=nfe,
                          device_ms=eng.last_generate_device_ms, host_gap_ms=dt * 1e3 - eng.last_generate_device_ms,
                          tokens_per_forward=wl.batch * N / nfe, ms_per_forward=dt * 1e3 / nfe,
                          blocks_per_sequence=nb, mean_block_len=float(N * wl.batch / max(sum(nb), 1)),
                          dtype="bf16" if wl.dtype == "bf16" else "f32", data="synthetic",
                          config=dict(workload=wl.name, batch=wl.batch, ctx=wl.ctx_max, gen_len=N,
                                      layers=n_layers, lm_head_scale=args.lm_scale,
                                      timing="wall clock around dc_generate, host read-back every step"))),
          flush=True)
    eng.close()


def run_prefill(args, wl, dev):
    """dc_prefill of --prompt-len tokens per sequence (one bidirectional pass, K / V export)."""
    from paper_2604_15750_b200 import DepCap
    n_layers = args.layers or wl.n_layers
    weights = inputs.make_weights(wl, device=dev, n_layers=n_layers)
    P = args.prompt_len
    max_ctx = (P + 63) // 64 * 64
    eng = DepCap.from_workload(wl, weights, n_layers=n_layers, max_ctx=max_ctx, max_last=P,
                               max_window=16)
    B, nkv, hd = wl.batch, wl.n_kv_heads, wl.head_dim
    kc = torch.zeros((n_layers, B, nkv, max_ctx, hd), dtype=wl.torch_dtype, device=dev)
    vc = torch.zeros((n_layers, B, nkv, hd, max_ctx), dtype=wl.torch_dtype, device=dev)
    g = torch.Generator().manual_seed(wl.seed)
    ids = torch.randint(0, wl.vocab - 1, (B, P), dtype=torch.int32, generator=g).to(dev)
    for _ in range(args.warmup):
        eng.prefill(kc, vc, ids, [P] * B)
    eng.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = min(args.steps, 20)
    e0.record(eng.stream)
    for _ in range(steps):
        eng.prefill(kc, vc, ids, [P] * B)
    e1.record(eng.stream)
    eng.synchronize()
    ms = e0.elapsed_time(e1) / steps
    # all layers but the last run in full; the last stops after its QKV projection
    qkv = wl.d_model * (wl.n_q_heads + 2 * wl.n_kv_heads) * wl.head_dim
    flops = 2.0 * B * P * ((n_layers - 1) * _layer_param_count(wl) + qkv)
    flops += 4.0 * B * (n_layers - 1) * wl.n_q_heads * wl.head_dim * P * P      # attention
    peaks = _peaks()
    print(json.dumps(dict(metric="prefill_tokens_per_s", value=B * P / (ms * 1e-3), unit="tokens/s",
                          n_gpus=1, mode="prefill", ms=ms, tflops=flops / (ms * 1e-3) / 1e12,
                          frac_of_bf16_peak=flops / (ms * 1e-3) / 1e12 / peaks["bf16_sustained"],
                          peak_source=peaks["source"], dtype="bf16" if wl.dtype == "bf16" else "f32",
                          data="synthetic",
                          config=dict(workload=wl.name, batch=B, prompt_len=P, layers=n_layers))),
          flush=True)
    eng.close()


def run_decisions(args, wl, dev):
    """The decision kernels alone over 8192 synthetic sequences with windows of 128 positions
    (dc_boundary_batched, dc_select_batched: device-side length arrays): at the sizes of a step
    they are bound by launch and dependency latency, here their memory traffic is large enough to
    time.  Algorithmic bytes: boundary 2 W floats in, 3 W floats + 1 int out per sequence; select
    W floats + W ints + W^2 floats + 1 int in, W bytes + W ints + 1 int out."""
    import numpy as np
    from paper_2604_15750_b200 import DepCap
    tiny = inputs.scaled(inputs.WORKLOADS["tiny_f32"], n_layers=0, ctx_min=0, ctx_max=0)
    weights = inputs.make_weights(tiny, device=dev, n_layers=0)
    eng = DepCap.from_workload(tiny, weights, n_layers=0, max_batch=1, max_window=128, max_ctx=0)
    B, W = 8192, 128
    g = torch.Generator(device=dev).manual_seed(1234)
    rnd = lambda *s: torch.rand(s, device=dev, generator=g)
    I = (torch.randn((B, W), device=dev, generator=g).abs() * torch.exp(-torch.arange(W, device=dev) / 16.0)).contiguous()
    H = rnd(B, W) * 8
    conf = torch.where(rnd(B, W) < 0.5, 0.9 + 0.1 * rnd(B, W), rnd(B, W))
    x = torch.randn((B, W, W), device=dev, generator=g) * 6 - 12
    ids = torch.where(rnd(B, W) < 0.8, tiny.mask_id, 5).to(torch.int32)
    win = torch.full((B,), W, dtype=torch.int32, device=dev)
    remain = torch.full((B,), 256, dtype=torch.int32, device=dev)
    bo = dict(score=torch.zeros((B, W), device=dev), cum_influence=torch.zeros((B, W), device=dev),
              cum_score=torch.zeros((B, W), device=dev), block_len=torch.zeros((B,), dtype=torch.int32, device=dev))
    so = dict(sel_mask=torch.zeros((B, W), dtype=torch.uint8, device=dev),
              sel_idx=torch.zeros((B, W), dtype=torch.int32, device=dev),
              sel_count=torch.zeros((B,), dtype=torch.int32, device=dev))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than L2
    peaks = _peaks()
    res = {}
    # the whole window is the block, so that Algorithm 1 sees pools of about 50 positions; it reads
    # D_ij only for pairs of pool members (both halves of Eq. 6): bytes touched are counted from
    # the inputs, the nominal figure is the whole W x W matrix
    blk = torch.full((B,), W, dtype=torch.int32, device=dev)
    pool = ((ids == tiny.mask_id) & (conf >= 0.8)).sum(dim=1).double()
    sel_touched = float((2.0 * pool * (pool - 1) * 4).sum().item()) + B * (W * 4.0 + W * 4 + 8 + W + W * 4 + 4)
    for name, fn, nbytes, nominal in (
            ("k_boundary", lambda: eng.boundary_batched(I, H, win, remain, bo), B * (5.0 * W * 4 + 12),
             B * (5.0 * W * 4 + 12)),
            ("k_select", lambda: eng.select_batched(conf, ids, x, blk, win, so), sel_touched,
             B * (W * 4.0 + W * 4 + W * W * 4 + 8 + W + W * 4 + 4))):
        for _ in range(3):
            fn()
        times = []
        for _ in range(max(5, min(args.steps, 20))):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(eng.stream); fn(); e1.record(eng.stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = float(np.median(times))
        ach = nbytes / (ms * 1e-3) / 1e9
        res[name] = dict(ms=ms, algorithmic_bytes=nbytes, nominal_bytes=nominal, achieved=ach, unit="GB/s",
                         peak=peaks["hbm"], frac=ach / peaks["hbm"], bound="hbm")
    committed = int(so["sel_count"].sum().item())
    print(json.dumps(dict(metric="decision_kernels_GBps", mode="decisions", n_gpus=1, sequences=B, window=W,
                          committed=committed, rooflines=res, peak_source=peaks["source"],
                          l2="flushed between timed launches (256 MiB fill)", data="synthetic", dtype="f32")),
          flush=True)
    eng.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b_b1", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="debug: run fewer layers (invalid as a result)")
    ap.add_argument("--batch", type=int, default=0,
                    help="debug: run fewer sequences of the workload (invalid as a result; for profiler captures)")
    ap.add_argument("--kernels", default="auto", choices=["auto", "simt"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-coop", action="store_true",
                    help="profiling: launch the fused dense kernel without the cooperative attribute "
                         "(ncu cannot replay cooperative cluster launches); same grid, same work")
    ap.add_argument("--mode", default="step", choices=["step", "generate", "prefill", "decisions"],
                    help="step: the bench line; generate / prefill: measurements of the decoding "
                         "loop and of dc_prefill on the same model shape (one GPU, own JSON line)")
    ap.add_argument("--prev", default="recomputed", choices=["recomputed", "carried"],
                    help="step mode: p_prev from a second variant in the pass (the bench line) or from "
                         "rows carried in (DC_STEP_CARRIED_PREV: half the rows through the stack)")
    ap.add_argument("--ctx", default="prefill", choices=["prefill", "noise"],
                    help="step mode: the context cache comes from dc_prefill over the seeded prompt "
                         "(default) or is seeded N(0,1) noise")
    ap.add_argument("--gen-len", type=int, default=256)
    ap.add_argument("--prompt-len", type=int, default=1024)
    ap.add_argument("--lm-scale", type=float, default=8.0,
                    help="generate: factor on the random-init LM head so that predictions are peaked")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl = inputs.WORKLOADS[args.workload]
    if args.batch:
        wl = inputs.scaled(wl, batch=args.batch)
    if args.impl == "reference":
        run_reference(args, wl, rank, world)
        return

    from paper_2604_15750_b200 import DepCap, pack_kv_cache, STAGE_NAMES
    from paper_2604_15750_b200 import build as _build
    _build.build()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU path"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if args.mode != "step":
        if rank == 0:
            dict(generate=run_generate, prefill=run_prefill, decisions=run_decisions)[args.mode](args, wl, dev)
        return
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    n_layers = args.layers or wl.n_layers
    # each replica draws its own sequences (seed offset by rank); weights are the same model
    wl_r = inputs.scaled(wl, seed=replicas.replica_seed(wl.seed, rank)) if rank else wl
    weights, k_log, v_log, toks, lens, steer = _setup(wl, dev, n_layers, noise_ctx=args.ctx != "prefill")
    if rank:
        toks = inputs.make_tokens(wl_r)
        steer = inputs.make_steering(wl_r, weights["lm_head"], profile="decay")
    eng = DepCap.from_workload(wl, weights, n_layers=n_layers, impl=1 if args.kernels == "simt" else 0,
                               max_last=max(wl.last_len, wl.ctx_max) if args.ctx == "prefill" else None)
    if args.no_coop:
        eng.set_option(1, 0)
    B, W = wl.batch, eng.max_window
    if args.ctx == "prefill":
        # the context cache as the model itself makes it: one bidirectional pass over the prompt
        kc = torch.zeros((n_layers, eng.max_batch, wl.n_kv_heads, eng.max_ctx, wl.head_dim),
                         dtype=wl.torch_dtype, device=dev)
        vc = torch.zeros((n_layers, eng.max_batch, wl.n_kv_heads, wl.head_dim, eng.max_ctx),
                         dtype=wl.torch_dtype, device=dev)
        ids = torch.zeros((B, eng.max_last), dtype=torch.int32)
        ids[:, :wl.ctx_max] = toks["prompt"]
        eng.prefill(kc, vc, ids.to(dev), lens["ctx_len"])
        eng.synchronize()
        assert int(eng.out["status"][:B].abs().max().item()) == 0
    else:
        kc, vc = pack_kv_cache(k_log, v_log, eng.max_batch, eng.max_ctx)
    last_h = torch.zeros((B, eng.max_last), dtype=torch.int32).pin_memory()
    last_h[:, :wl.last_len] = toks["last_ids"]
    win_h = torch.full((B, W), wl.mask_id, dtype=torch.int32).pin_memory()
    win_h[:, :wl.win_len] = toks["win_ids"]
    hf_h = torch.zeros((B, 2, W, wl.d_model), dtype=wl.torch_dtype).pin_memory()
    hf_h[:, :, :wl.win_len] = steer.cpu()
    last_d, win_d, hf_d = last_h.to(dev), win_h.to(dev), hf_h.to(dev)
    step_kw = dict(k_cache=kc, v_cache=vc, ctx_len=lens["ctx_len"], last_len=lens["last_len"],
                   win_len=lens["win_len"], remain_len=lens["remain_len"])
    if args.prev == "carried":
        step_kw["carried"] = (hf_d[:, 1].contiguous(), lens["win_len"])
    stream = eng.stream

    def one_step():
        eng.step(last_ids=last_d, win_ids=win_d, h_final=hf_d, **step_kw)
        eng.select(win_d, lens["win_len"])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        one_step()
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    committed = int(eng.sel["sel_count"][:B].sum().item())
    status_bad = int(eng.out["status"][:B].abs().max().item())

    # ---- end to end through the public API with host buffers ------------------------------
    out_h = dict(pred=torch.zeros((B, W), dtype=torch.int32).pin_memory(),
                 conf=torch.zeros((B, W), dtype=torch.float32).pin_memory(),
                 blk=torch.zeros((B,), dtype=torch.int32).pin_memory(),
                 mask=torch.zeros((B, W), dtype=torch.uint8).pin_memory(),
                 cnt=torch.zeros((B,), dtype=torch.int32).pin_memory())

    def one_step_e2e():
        with torch.cuda.stream(stream):
            last_d.copy_(last_h, non_blocking=True)
            win_d.copy_(win_h, non_blocking=True)
            hf_d.copy_(hf_h, non_blocking=True)
            one_step()
            out_h["pred"].copy_(eng.out["pred_id"][:B], non_blocking=True)
            out_h["conf"].copy_(eng.out["conf"][:B], non_blocking=True)
            out_h["blk"].copy_(eng.out["block_len"][:B], non_blocking=True)
            out_h["mask"].copy_(eng.sel["sel_mask"][:B], non_blocking=True)
            out_h["cnt"].copy_(eng.sel["sel_count"][:B], non_blocking=True)
        stream.synchronize()          # the host needs the subset before it can commit tokens

    h2d = last_h.numel() * 4 + win_h.numel() * 4 + hf_h.numel() * hf_h.element_size()
    d2h = sum(t.numel() * t.element_size() for t in out_h.values())
    e2e_steps = max(3, min(args.steps, 10))
    one_step_e2e()
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record(stream)
    for _ in range(e2e_steps):
        one_step_e2e()
    e3.record(stream)
    barrier()
    e2e_ms = e2.elapsed_time(e3) / e2e_steps
    committed_e2e = int(out_h["cnt"].sum().item())

    # ---- per-stage device time, live, for the roofline of the dominant kernel --------------
    stage_ms = {n: 0.0 for n in STAGE_NAMES}
    launches = {}
    reps = 3
    for _ in range(reps):
        ms, launches = eng.step_profiled(last_ids=last_d, win_ids=win_d, h_final=hf_d, **step_kw)
        for n in STAGE_NAMES:
            stage_ms[n] += ms[n] / reps
    gpu_launches = (sum(launches.values()) + 1) * args.steps      # + dc_select

    # ---- reduce over ranks --------------------------------------------------------------------
    ms_step = ms_total / args.steps
    (ms_step, e2e_ms), (committed, committed_e2e) = replicas.combine(
        dist, [ms_step, e2e_ms], [committed, committed_e2e], device=dev)
    if rank != 0:
        eng.close()
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = _peaks()
    src = peaks["source"] + (" (of measured)" if peaks["source"] == "measured" else " (of fallback)")
    nv = 1 if args.prev == "carried" else 2
    Rcap = (wl.last_len + wl.win_len + 15) // 16 * 16
    M = nv * wl.batch * Rcap
    fused = launches.get("dense", 0) > 0

    def roof_entry(kernel, ms, nbytes, flops, launches_per_step):
        """Roofline of one kernel group over a step: the binding resource is the one whose floor
        (bytes / measured copy bandwidth, flops / measured sustained bf16 rate) is larger."""
        t_hbm = nbytes / (peaks["hbm"] * 1e9)
        t_tensor = flops / (peaks["bf16_sustained"] * 1e12)
        if ms <= 0:
            return None
        if t_hbm >= t_tensor:
            ach = nbytes / (ms * 1e-3) / 1e9
            r = dict(bound="hbm", achieved=ach, peak=peaks["hbm"], unit="GB/s", frac=ach / peaks["hbm"])
        else:
            ach = flops / (ms * 1e-3) / 1e12
            r = dict(bound="tensor", achieved=ach, peak=peaks["bf16_sustained"], unit="TFLOP/s",
                     frac=ach / peaks["bf16_sustained"])
        r.update(kernel=kernel, ms_per_step=round(ms, 4), launches_per_step=launches_per_step,
                 algorithmic_bytes=nbytes, algorithmic_flops=flops, traffic=None, peak_source=src)
        return r

    # dense layers: every weight byte once per step; 2 flops per parameter and activation row
    gemm_ms = sum(stage_ms[n] for n in ("qkv", "oproj", "gateup", "down", "dense"))
    w_bytes = 2.0 * _layer_param_count(wl) * n_layers
    dense_name = ("k_dense_chain: O projection, norms, gate/up + SwiGLU, down projection, QKV + RoPE of the "
                  "next layer in one persistent launch per layer" if fused else
                  "k_gemm_tc: per-op QKV + RoPE, O projection, gate/up + SwiGLU, down projection")
    roof = roof_entry(dense_name, gemm_ms, w_bytes, w_bytes * M,
                      sum(launches.get(n, 0) for n in ("qkv", "oproj", "gateup", "down", "dense")))
    # DRAM traffic of the dense chain from the ncu capture summarised under profiles/ (one launch =
    # one layer), scaled to the launches of one step (traffic grows with the weights streamed)
    if fused:
        per_layer = _traffic_record(wl.name)
        if per_layer is not None:
            first = per_layer * (wl.d_model * (wl.n_q_heads + 2 * wl.n_kv_heads) * wl.head_dim) / _layer_param_count(wl)
            roof["traffic"] = per_layer * n_layers + first
    roof["stage_ms"] = {k: round(v, 4) for k, v in stage_ms.items()}
    # attention: per sequence and layer the context K / V once plus q, k, v, o of the active rows
    # (both variants); 4 flops per (query row, key, head-dim element)
    nkv_b = wl.n_kv_heads * wl.head_dim * 2.0
    att_bytes = sum(n_layers * 2.0 * (P + nv * Rcap) * nkv_b for P in lens["ctx_len"])
    att_flops = sum(4.0 * n_layers * wl.n_q_heads * wl.head_dim * nv * Rcap * (P + Rcap) for P in lens["ctx_len"])
    rooflines = [roof,
                 roof_entry("k_attn_tc: bidirectional block attention (one CTA per query tile; row tiles of 64 rows or fewer carry both variants over one staged context)",
                            stage_ms["attn"], att_bytes, att_flops, launches.get("attn", 0)),
                 roof_entry("k_lmhead_tc + k_lm_combine: LM head with streaming softmax / entropy / KL",
                            stage_ms["lmhead"], 2.0 * wl.vocab * wl.d_model,
                            2.0 * (2 * wl.batch * wl.win_len) * wl.vocab * wl.d_model, launches.get("lmhead", 0))]
    # decision kernels: (5 W + W^2) floats per sequence; at these sizes they are bound by launch
    # and dependency latency, not by bytes (bench.py --mode decisions gives their bandwidth number)
    dec_bytes = wl.batch * (5.0 * wl.win_len + wl.win_len ** 2) * 4.0
    e4, e5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e4.record(stream)
    for _ in range(20):
        eng.select(win_d, lens["win_len"])
    e5.record(stream)
    torch.cuda.synchronize()
    sel_ms = e4.elapsed_time(e5) / 20
    for name, ms_ in (("k_xlogp: cross log-probs (Eq. 6 halves)", stage_ms["xlogp"]),
                      ("k_boundary: smoothing, S_k, prefix sums, cut", stage_ms["boundary"]),
                      ("k_select: CAP-Decoding", sel_ms)):
        r = roof_entry(name, ms_, dec_bytes, 0.0, 1)
        if r:
            r["bound"] = "latency"
            rooflines.append(r)
    rooflines = [r for r in rooflines if r]

    cpu = None
    parity = None
    if not args.no_cpu_baseline:
        s = _oracle_sample(inputs.scaled(wl, n_layers=n_layers), weights,
                           k_log, v_log, toks, lens, steer,
                           prompt=toks["prompt"] if args.ctx == "prefill" else None)
        dec = []
        oc = _oracle_committed(wl, weights, toks, lens, steer, decisions=dec)
        cpu = dict(value=oc / s["est_step_s"], unit=UNIT, cores=torch.get_num_threads(),
                   kind="oracle", sample=s["sample"], est_step_ms=s["est_step_s"] * 1e3,
                   committed=oc, extrapolated=True)
        # the step's decisions against the oracle's on the same steered inputs (rank 0's sequences)
        pred_g = eng.out["pred_id"][:B].cpu().numpy()
        blk_g = eng.out["block_len"][:B].cpu().numpy()
        mask_g = eng.sel["sel_mask"][:B].cpu().numpy()
        parity = dict(positions=0, pred_mismatch=0, block_len_mismatch=0, subset_mismatch=0)
        for b, o in enumerate(dec):
            Wb = lens["win_len"][b]
            parity["positions"] += Wb
            parity["pred_mismatch"] += int((pred_g[b, :Wb] != o["pred"]).sum())
            parity["block_len_mismatch"] += int(int(blk_g[b]) != o["block_len"])
            parity["subset_mismatch"] += int([i for i in range(Wb) if mask_g[b, i]] != o["selected"])

    line = dict(metric=METRIC, value=committed / (ms_step * 1e-3), unit=UNIT, n_gpus=world,
                steps=args.steps, warmup=args.warmup, ms_per_step=ms_step, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="bf16" if wl.dtype == "bf16" else "f32",
                data="synthetic",
                config=_config(wl, n_layers, "curr + carried prev rows" if args.prev == "carried" else "curr+prev",
                               ctx=args.ctx),
                committed_per_step=committed, kernels=args.kernels, status=status_bad,
                clocks=clocks,
                e2e=dict(value=committed_e2e / (e2e_ms * 1e-3), unit=UNIT, ms_per_step=e2e_ms,
                         h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h),
                gpu_launches=gpu_launches, roofline=roof, rooflines=rooflines, cpu_baseline=cpu,
                decisions_vs_oracle=parity)
    print(json.dumps(line))
    eng.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
