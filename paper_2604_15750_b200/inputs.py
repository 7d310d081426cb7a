"""Seeded synthetic inputs for the DepCap block-step (weights, tokens, context K/V, steering).

This module is the only code that both the CUDA path's tests/benchmark and the CPU oracle's
callers use.  It holds none of the method's arithmetic: it only draws random tensors with
the shapes and value distributions of the workloads (random-init backbones shaped like
LLaDA-8B and Dream-7B, uniform-random prompts, all-masked windows) and builds the optional
LM-head steering input that makes the decisions non-degenerate.

Every tensor has its own generator seeded from (workload seed, tensor name, layer), so a
single layer can be drawn without drawing the others.
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    dtype: str            # "f32" | "bf16"
    batch: int
    ctx_min: int          # context lengths are uniform in [ctx_min, ctx_max]
    ctx_max: int
    last_len: int         # Lb: length of the last decoded block
    win_len: int          # W: candidate window
    gen_len: int          # L_remain handed to the boundary rule
    seed: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    qkv_bias: bool = False    # biases on the q / k / v projections (the Dream backbone has them)

    @property
    def mask_id(self) -> int:
        return self.vocab - 1

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


_BASE_SEED = 20260415

WORKLOADS = {
    # 1: tiny fp32 transformer, the case the oracle finishes in a fraction of a second
    "tiny_f32": Workload("tiny_f32", 2, 256, 4, 4, 64, 1024, 4096, "f32", 1, 64, 64, 16, 32,
                         32, _BASE_SEED + 1),
    # 2: LLaDA-8B shape, batch 1 (the configuration the headline metric is quoted on)
    "llada8b_b1": Workload("llada8b_b1", 32, 4096, 32, 32, 128, 12288, 126464, "bf16", 1, 512,
                           512, 32, 64, 256, _BASE_SEED + 2),
    # 3: LLaDA-8B shape, batch 8, ragged prompts
    "llada8b_b8": Workload("llada8b_b8", 32, 4096, 32, 32, 128, 12288, 126464, "bf16", 8, 768,
                           1024, 32, 128, 512, _BASE_SEED + 3),
    # 4: Dream-7B shape (grouped KV heads), batch 4
    "dream7b_b4": Workload("dream7b_b4", 28, 3584, 28, 4, 128, 18944, 152064, "bf16", 4, 768,
                           768, 32, 64, 512, _BASE_SEED + 4),
    # LLaDA-1.5 (the paper's third backbone) has LLaDA-8B's architecture: same shapes, own seed
    "llada15_b1": Workload("llada15_b1", 32, 4096, 32, 32, 128, 12288, 126464, "bf16", 1, 512,
                           512, 32, 64, 256, _BASE_SEED + 6),
    # Dream-7B shape with the biases its q / k / v projections carry
    "dream7b_b4_bias": Workload("dream7b_b4_bias", 28, 3584, 28, 4, 128, 18944, 152064, "bf16", 4,
                                768, 768, 32, 64, 512, _BASE_SEED + 4, qkv_bias=True),
    # 5: long-context stress, LLaDA-8B shape, batch 16
    "llada8b_long": Workload("llada8b_long", 32, 4096, 32, 32, 128, 12288, 126464, "bf16", 16,
                             4096, 4096, 32, 128, 1024, _BASE_SEED + 5),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (fewer layers, smaller vocab, ...)."""
    return replace(w, **kw)


def _gen(w: Workload, name: str, layer: int = -1, device="cpu") -> torch.Generator:
    h = hashlib.sha256(f"{w.seed}/{name}/{layer}".encode()).digest()
    g = torch.Generator(device=device)
    g.manual_seed(int.from_bytes(h[:8], "little") >> 1)
    return g


def _normal(w: Workload, name, layer, shape, std, device, dtype=None):
    g = _gen(w, name, layer, device)
    t = torch.empty(shape, dtype=torch.float32, device=device).normal_(0.0, std, generator=g)
    return t.to(dtype or w.torch_dtype)


def layer_weights(w: Workload, layer: int, device="cpu") -> dict:
    """Weights of one transformer layer, N(0, 0.02), row-major [out, in]; norm gains 1."""
    d, hq, hkv, F = w.d_model, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.d_ff
    mk = lambda n, s: _normal(w, n, layer, s, 0.02, device)
    lw = dict(wq=mk("wq", (hq, d)), wk=mk("wk", (hkv, d)), wv=mk("wv", (hkv, d)),
              wo=mk("wo", (d, hq)), w_gate=mk("w_gate", (F, d)), w_up=mk("w_up", (F, d)),
              w_down=mk("w_down", (d, F)),
              norm1=torch.ones(d, dtype=w.torch_dtype, device=device),
              norm2=torch.ones(d, dtype=w.torch_dtype, device=device))
    if w.qkv_bias:   # N(0, 0.5): large against the projections of a random-init model, so that a
        # dropped or misplaced bias cannot hide inside the tolerance
        mb = lambda n, k: _normal(w, n, layer, (k,), 0.5, device)
        lw.update(bq=mb("bq", hq), bk=mb("bk", hkv), bv=mb("bv", hkv))
    return lw


def make_weights(w: Workload, device="cpu", n_layers: int | None = None) -> dict:
    """{'embed','lm_head','final_norm', 'layers': [layer dicts]}."""
    n = w.n_layers if n_layers is None else n_layers
    return dict(embed=_normal(w, "embed", -1, (w.vocab, w.d_model), 0.02, device),
                lm_head=_normal(w, "lm_head", -1, (w.vocab, w.d_model), 0.02, device),
                final_norm=torch.ones(w.d_model, dtype=w.torch_dtype, device=device),
                layers=[layer_weights(w, l, device) for l in range(n)])


def make_lengths(w: Workload) -> dict:
    """Per-sequence lengths: ctx_len uniform in [ctx_min, ctx_max]; Lb, W, L_remain fixed."""
    g = _gen(w, "ctx_len")
    ctx = torch.randint(w.ctx_min, w.ctx_max + 1, (w.batch,), generator=g, dtype=torch.int32)
    return dict(ctx_len=ctx,
                last_len=torch.full((w.batch,), w.last_len, dtype=torch.int32),
                win_len=torch.full((w.batch,), w.win_len, dtype=torch.int32),
                remain_len=torch.full((w.batch,), w.gen_len, dtype=torch.int32))


def make_tokens(w: Workload, n_decoded_in_window: int = 0) -> dict:
    """Prompt, last decoded block (uniform ids without the mask id) and the window.

    The window is all [MASK] unless n_decoded_in_window > 0, in which case that many seeded
    positions per sequence already hold clean ids (a step in the middle of a block).
    """
    hi = w.vocab - 1                                   # mask id = vocab - 1 is excluded
    prompt = torch.randint(0, hi, (w.batch, w.ctx_max), generator=_gen(w, "prompt"),
                           dtype=torch.int32)
    last = torch.randint(0, hi, (w.batch, w.last_len), generator=_gen(w, "last"),
                         dtype=torch.int32)
    win = torch.full((w.batch, w.win_len), w.mask_id, dtype=torch.int32)
    if n_decoded_in_window:
        g = _gen(w, "decoded")
        for b in range(w.batch):
            idx = torch.randperm(w.win_len, generator=g)[:n_decoded_in_window]
            win[b, idx] = torch.randint(0, hi, (n_decoded_in_window,), generator=g,
                                        dtype=torch.int32)
    return dict(prompt=prompt, last_ids=last, win_ids=win)


def make_ctx_kv(w: Workload, device="cpu", n_layers: int | None = None):
    """Seeded N(0,1) context cache, logical layout [layers, batch, n_kv, ctx_max, head_dim].

    K is treated as already rotated.  Stands in for a real prefill of the prompt.
    """
    n = w.n_layers if n_layers is None else n_layers
    shape = (n, w.batch, w.n_kv_heads, w.ctx_max, w.head_dim)
    k = _normal(w, "k_ctx", -1, shape, 1.0, device)
    v = _normal(w, "v_ctx", -1, shape, 1.0, device)
    return k, v


def make_steering(w: Workload, lm_head: torch.Tensor, profile: str = "decay",
                  device="cpu") -> torch.Tensor:
    """LM-head input [batch, 2, win_len, d] (curr, prev) that shapes the distributions.

    Row k of the curr variant is a_k * u(t_k) (+ rho * a_k * u(t_partner)) + noise, with
    u(t) = lm_head[t] / |lm_head[t]|^2, so the logit of the target t_k is about a_k and every
    other logit stays near zero: the top probability is about sigmoid(a_k - log(V - 2)).
    The prev variant scales a_k by (1 - 0.6 exp(-k/16)): the last block's influence decays
    with the distance from the frontier.
      profile "decay"  : a_k uniform in [log V - 4, log V + 6], shrinking with k
      profile "bimodal": each position peaked (a_k = log V + 2.8, p_top > 0.9) or flat (a_k = 0)
    A quarter of the peaked positions get a partner within distance 4 whose target they also
    support (rho = 0.75, a conflicting pair); 5% copy a neighbour's target.
    """
    B, W, d, V = w.batch, w.win_len, w.d_model, w.vocab
    g = _gen(w, "steer/" + profile)
    logV = math.log(V)
    tgt = torch.randint(0, V - 1, (B, W), generator=g)
    k_idx = torch.arange(W, dtype=torch.float32)
    if profile == "bimodal":
        peaked = torch.rand((B, W), generator=g) < 0.5
        a = torch.where(peaked, torch.tensor(logV + 2.8), torch.tensor(0.0))
    else:
        a = (logV - 4.0) + 10.0 * torch.rand((B, W), generator=g) * torch.exp(-k_idx / 48.0)
        peaked = a > logV + 2.0
    dup = (torch.rand((B, W), generator=g) < 0.05)
    dup[:, 0] = False
    tgt = torch.where(dup, torch.roll(tgt, 1, dims=1), tgt)
    paired = (torch.rand((B, W), generator=g) < 0.25) & peaked
    offs = torch.randint(1, 5, (B, W), generator=g)
    partner = torch.clamp(torch.arange(W)[None, :] + offs, max=W - 1)
    out = torch.zeros((B, 2, W, d), dtype=torch.float32)
    for b in range(B):
        u = lm_head[tgt[b].to(lm_head.device)].detach().to("cpu", torch.float32)
        u = u / (u * u).sum(dim=1, keepdim=True)                       # [W, d]
        base = a[b][:, None] * u
        extra = torch.where(paired[b][:, None], 0.75 * a[b][:, None] * u[partner[b]],
                            torch.zeros_like(u))
        noise = 1e-3 * torch.randn((W, d), generator=g)
        curr = base + extra + noise
        damp = (1.0 - 0.6 * torch.exp(-k_idx / 16.0))[:, None]
        prev = damp * (base + extra) + noise
        out[b, 0], out[b, 1] = curr, prev
    return out.to(w.torch_dtype).to(device)
