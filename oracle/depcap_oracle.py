"""CPU oracle for one DepCap block-step.  TEST INFRASTRUCTURE ONLY.

Plain, slow, deliberately unoptimised numpy: fp64 for every floating-point reduction, a
library matmul as the only primitive, no blocking, no fusion.  It shares no code with the
CUDA path and must never be imported by it; only tests, the smoke check and the CPU-baseline
leg of the benchmark may call it.

What it follows (paper: "DepCap: Adaptive Block-Wise Parallel Decoding for Efficient
Diffusion LM Inference"):

  * block-wise masked-diffusion step, Eq. (1)-(2): predictions for the masked positions of
    the active block given a clean decoded context;
  * last-block influence I_k = KL(p_curr || p_prev), Eq. (3), where p_curr conditions on
    the last decoded block and p_prev does not (Section 4.4: p(Z_k | c, b) vs p(Z_k | c));
  * entropy H_k, dependency score S_k = I~_k - lambda H~_k, Eq. (4), first-negative scan and
    clipping to [L_min, L_window] (Section 4.2);
  * cumulative form of the same criterion (Section 4.4 / appendix "Detailed Derivation");
  * candidate pool Eq. (5), conflict score D_ij Eq. (6), CAP-Decoding Algorithm 1.

The backbone is a black box in the paper; here it is the pre-norm transformer the workload
configurations name (RMSNorm, rotate-half RoPE, bidirectional attention, grouped KV heads,
SwiGLU MLP, untied LM head; no biases, or biases on the q / k / v projections only).

Parity status of each function (what pins it is in tests/test_oracle_*.py):
  forward / attention / rope / rmsnorm / swiglu : pinned (library routines, closed forms)
  signals (argmax, confidence, entropy, KL)     : pinned (closed forms, brute force)
  cap_select                                    : pinned (hand cases, exhaustive invariants)
  boundary                                      : the scan, clip and cumulative rule are
      pinned; the smoothing kernel and the normalisation are this build's reading of
      "smoothed and normalized" (the paper does not define them): parity unpinned.
  end-to-end numbers against the authors' code or tables: parity unpinned (needs trained
      weights and datasets that are not available).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# reading selectors -----------------------------------------------------------------------
NORM_MAX, NORM_MINMAX, NORM_NONE = 0, 1, 2
BOUNDARY_FIRST_NEG, BOUNDARY_CUMULATIVE = 0, 1
CAP_LITERAL, CAP_STRICT = 0, 1
FX_SHIFT = 40  # fixed-point scale 2**40 of the cumulative sums


@dataclass
class OracleConfig:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    mask_id: int
    bf16: bool = False            # round every GEMM input to bf16 (weights are given as-is)
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    # DepCap hyper-parameters, defaults of the "Hyperparameter settings" paragraph
    lam: float = 1.2
    L_min: int = 8
    L_max: int = 128
    tau_low: float = 0.8
    tau_high: float = 0.95
    gamma: float = -16.0
    # readings of points the paper leaves open
    smooth_radius: int = 1
    norm_mode: int = NORM_MAX
    boundary_mode: int = BOUNDARY_FIRST_NEG
    cap_mode: int = CAP_LITERAL
    forbid_mask_pred: bool = True


@dataclass
class OracleWeights:
    """All arrays float32/float64 numpy, row-major [out, in] like the GPU library."""
    embed: np.ndarray                    # [V, d]
    wq: list = field(default_factory=list)      # per layer [n_q*hd, d]
    wk: list = field(default_factory=list)      # [n_kv*hd, d]
    wv: list = field(default_factory=list)      # [n_kv*hd, d]
    wo: list = field(default_factory=list)      # [d, n_q*hd]
    w_gate: list = field(default_factory=list)  # [F, d]
    w_up: list = field(default_factory=list)    # [F, d]
    w_down: list = field(default_factory=list)  # [d, F]
    norm1: list = field(default_factory=list)   # [d]
    norm2: list = field(default_factory=list)   # [d]
    # optional biases of the q / k / v projections (the Dream backbone's attention layers carry
    # them; LLaDA's do not): per layer [n_q*hd], [n_kv*hd], [n_kv*hd], added before the rotation
    bq: list = field(default_factory=list)
    bk: list = field(default_factory=list)
    bv: list = field(default_factory=list)
    final_norm: np.ndarray | None = None        # [d]
    lm_head: np.ndarray | None = None           # [V, d]


# ------------------------------------------------------------------------------------------
# precision helper
# ------------------------------------------------------------------------------------------
def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as float64.

    bfloat16 keeps the top 16 bits of an IEEE binary32; rounding adds half of the dropped
    part, plus the parity of the kept part for ties.  NaN/Inf are passed through.
    """
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    keep_lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + keep_lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32).astype(np.float64)
    finite = np.isfinite(f)
    return np.where(finite, out, f.astype(np.float64))


def _gemm_in(x: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    return bf16_round(x) if cfg.bf16 else np.asarray(x, dtype=np.float64)


# ------------------------------------------------------------------------------------------
# backbone pieces (the paper's black-box DLM; shape named by the workload configurations)
# ------------------------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y = x * rsqrt(mean(x^2) + eps) * g, row-wise."""
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(g, dtype=np.float64)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate-half rotary embedding.  x: [rows, heads, hd]; pos: [rows] absolute positions.

    Pair (i, i + hd/2) is rotated by the angle pos * theta**(-2i/hd).
    """
    x = np.asarray(x, dtype=np.float64)
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / hd)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]   # [rows, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, n_q_heads: int,
              n_kv_heads: int) -> np.ndarray:
    """Bidirectional (unmasked) softmax attention of every query over every key.

    q: [Rq, n_q, hd]; k, v: [Rk, n_kv, hd].  Query head h reads KV head h // (n_q/n_kv).
    Returns [Rq, n_q, hd].
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    hd = q.shape[-1]
    group = n_q_heads // n_kv_heads
    out = np.empty_like(q)
    for h in range(n_q_heads):
        g = h // group
        s = q[:, h, :] @ k[:, g, :].T / math.sqrt(hd)            # [Rq, Rk]
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, h, :] = p @ v[:, g, :]
    return out


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def forward(cfg: OracleConfig, w: OracleWeights, tok: np.ndarray, pos0: int,
            k_ctx: np.ndarray | None, v_ctx: np.ndarray | None,
            return_kv: bool = False, n_layers: int | None = None):
    """Hidden states (before the final norm) of the active rows of one variant.

    tok: [R] token ids of the active rows; their absolute positions are pos0 + r.
    k_ctx, v_ctx: cached context [n_layers, n_kv, P, hd] (K already rotated) or None (P=0).
    Every active row attends all P context rows and all R active rows (bidirectional).
    """
    R = len(tok)
    pos = pos0 + np.arange(R)
    nq, nkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    x = np.asarray(w.embed, dtype=np.float64)[np.asarray(tok, dtype=np.int64)]
    kv_out = []
    L = cfg.n_layers if n_layers is None else n_layers
    for l in range(L):
        a = _gemm_in(rmsnorm(x, w.norm1[l], cfg.rms_eps), cfg)
        q = a @ np.asarray(w.wq[l], dtype=np.float64).T
        k = a @ np.asarray(w.wk[l], dtype=np.float64).T
        v = a @ np.asarray(w.wv[l], dtype=np.float64).T
        if w.bq:
            q = q + np.asarray(w.bq[l], dtype=np.float64)
            k = k + np.asarray(w.bk[l], dtype=np.float64)
            v = v + np.asarray(w.bv[l], dtype=np.float64)
        q, k, v = q.reshape(R, nq, hd), k.reshape(R, nkv, hd), v.reshape(R, nkv, hd)
        q = _gemm_in(rope(q, pos, cfg.rope_theta), cfg)
        k = _gemm_in(rope(k, pos, cfg.rope_theta), cfg)
        v = _gemm_in(v, cfg)
        if return_kv:
            kv_out.append((k.copy(), v.copy()))
        if k_ctx is not None and k_ctx.shape[2] > 0:
            kc = np.transpose(np.asarray(k_ctx[l], dtype=np.float64), (1, 0, 2))  # [P,nkv,hd]
            vc = np.transpose(np.asarray(v_ctx[l], dtype=np.float64), (1, 0, 2))
            k_all = np.concatenate([kc, k], axis=0)
            v_all = np.concatenate([vc, v], axis=0)
        else:
            k_all, v_all = k, v
        o = _gemm_in(attention(q, k_all, v_all, nq, nkv).reshape(R, nq * hd), cfg)
        x = x + o @ np.asarray(w.wo[l], dtype=np.float64).T
        a2 = _gemm_in(rmsnorm(x, w.norm2[l], cfg.rms_eps), cfg)
        gate = a2 @ np.asarray(w.w_gate[l], dtype=np.float64).T
        up = a2 @ np.asarray(w.w_up[l], dtype=np.float64).T
        act = _gemm_in(silu(gate) * up, cfg)
        x = x + act @ np.asarray(w.w_down[l], dtype=np.float64).T
    if return_kv:
        return x, kv_out
    return x


def prefill(cfg: OracleConfig, w: OracleWeights, ids: np.ndarray, k_ctx=None, v_ctx=None,
            ctx_len: int = 0, n_layers: int | None = None, pos0: int | None = None):
    """K / V of a run of clean tokens (a prompt), as one bidirectional pass over them makes
    them: the tokens sit at positions ctx_len + r, attend one another and the ctx_len cached
    keys (Section 3: the model attends the whole known sequence, no causal mask).
    pos0: position of ids[0] when the tokens do not follow the cached ones in the sequence (the
    still masked suffix behind the window that a dual cache keeps, Section 5.2): attention is
    bidirectional and K carries its rotation, so a cached row's position matters only here.
    Returns (k, v), each [n_layers, n_kv_heads, len(ids), head_dim], K rotated.
    """
    if k_ctx is not None:
        k_ctx, v_ctx = k_ctx[:, :, :ctx_len, :], v_ctx[:, :, :ctx_len, :]
    _, kv = forward(cfg, w, np.asarray(ids), int(ctx_len if pos0 is None else pos0), k_ctx, v_ctx,
                    return_kv=True, n_layers=n_layers)
    k = np.stack([np.transpose(k_, (1, 0, 2)) for k_, _ in kv])
    v = np.stack([np.transpose(v_, (1, 0, 2)) for _, v_ in kv])
    return k, v


def final_hidden(cfg: OracleConfig, w: OracleWeights, x_rows: np.ndarray) -> np.ndarray:
    """LM-head input: final RMSNorm of the given rows (rounded when the path is bf16)."""
    return _gemm_in(rmsnorm(x_rows, w.final_norm, cfg.rms_eps), cfg)


# ------------------------------------------------------------------------------------------
# predictive signals (Section 4.2 and 4.3)
# ------------------------------------------------------------------------------------------
def logits_of(h: np.ndarray, lm_head: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    z = np.asarray(h, dtype=np.float64) @ np.asarray(lm_head, dtype=np.float64).T
    if cfg.forbid_mask_pred:
        z = z.copy()
        z[:, cfg.mask_id] = -np.inf     # the final sequence holds no [MASK] (Section 3)
    return z


def log_softmax(z: np.ndarray):
    m = z.max(axis=-1, keepdims=True)
    lse = m + np.log(np.exp(z - m).sum(axis=-1, keepdims=True))
    return z - lse, lse[..., 0]


def signals_from_logits(z_curr: np.ndarray, z_prev: np.ndarray | None):
    """Top-1 id, confidence c = max_v p(v), entropy H(p_curr), influence KL(p_curr||p_prev).

    Argmax ties resolve to the lowest token id.  Terms with p_curr(v) = 0 add nothing to
    the entropy or the KL sum.  Without a prev variant the influence is reported as 0.
    """
    logp, lse = log_softmax(z_curr)
    p = np.exp(logp)
    pred = np.argmax(z_curr, axis=-1).astype(np.int32)          # first maximum = lowest id
    conf = p[np.arange(len(pred)), pred]
    safe_logp = np.where(p > 0, logp, 0.0)
    ent = -(p * safe_logp).sum(axis=-1)
    if z_prev is None:
        infl = np.zeros_like(ent)
        lse_prev = np.zeros_like(lse)
    else:
        logq, lse_prev = log_softmax(z_prev)
        safe_logq = np.where(p > 0, logq, 0.0)
        infl = np.maximum((p * (safe_logp - safe_logq)).sum(axis=-1), 0.0)
    return pred, conf, ent, infl, lse, lse_prev


def cross_logprob(z_curr: np.ndarray, pred: np.ndarray, lse: np.ndarray) -> np.ndarray:
    """xlogp[i, j] = log p_i(yhat_j): the two halves of Eq. (6)."""
    return z_curr[:, pred] - lse[:, None]


# ------------------------------------------------------------------------------------------
# DepGA-Block boundary (Section 4.2; cumulative form from Section 4.4)
# ------------------------------------------------------------------------------------------
_F = np.float32


def _smooth(x: np.ndarray, radius: int) -> np.ndarray:
    """Centered moving average over the in-range taps, fp32, left-to-right adds, one divide."""
    n = len(x)
    out = np.empty(n, dtype=_F)
    for k in range(n):
        lo, hi = max(0, k - radius), min(n - 1, k + radius)
        acc = _F(x[lo])
        for j in range(lo + 1, hi + 1):
            acc = _F(acc + _F(x[j]))
        out[k] = _F(acc / _F(hi - lo + 1))
    return out


def _normalise(x: np.ndarray, mode: int) -> np.ndarray:
    if mode == NORM_NONE or len(x) == 0:
        return x.astype(_F)
    hi = _F(np.max(x))
    if mode == NORM_MAX:
        den = _F(max(hi, _F(1e-8)))
        return (x / den).astype(_F)
    lo = _F(np.min(x))
    den = _F(max(_F(hi - lo), _F(1e-8)))
    return ((x - lo).astype(_F) / den).astype(_F)


def _fx(s) -> int:
    """Fixed point llrint(s * 2**40) of an fp32 value (round half to even), as a Python int."""
    return int(np.rint(np.float64(_F(s)) * float(1 << FX_SHIFT)))


def boundary(infl: np.ndarray, ent: np.ndarray, win_len: int, remain_len: int,
             have_prev: bool, cfg: OracleConfig):
    """Next block length L and the per-position score arrays.

    L_window = min(L_max, L_remain) bounded by the positions actually supplied.  Without a
    last decoded block (the initial step) L = L_min, the conservative cold start.
    Otherwise: smooth, normalise, S_k = I~_k - lambda*H~_k (two fp32 roundings: product,
    then difference), k* = first k with S_k < 0 (or with the running fixed-point sum of S
    below zero in the cumulative mode), the block ends just before k*, L is clipped to
    [L_min, L_window] and never exceeds L_window.
    Returns (L, score[f32], cum_influence[f32], cum_score[f32]) over k < L_window.
    """
    Lw = max(0, min(cfg.L_max, int(remain_len), int(win_len)))
    I = np.asarray(infl[:Lw], dtype=_F)
    H = np.asarray(ent[:Lw], dtype=_F)
    if not have_prev:
        z = np.zeros(Lw, dtype=_F)
        return min(cfg.L_min, Lw), z, z.copy(), z.copy()
    Is = _normalise(_smooth(I, cfg.smooth_radius), cfg.norm_mode)
    Hs = _normalise(_smooth(H, cfg.smooth_radius), cfg.norm_mode)
    lam = _F(cfg.lam)
    score = np.empty(Lw, dtype=_F)
    for k in range(Lw):
        score[k] = _F(Is[k] - _F(lam * Hs[k]))
    cum_i = np.empty(Lw, dtype=_F)
    cum_s = np.empty(Lw, dtype=_F)
    acc_i = acc_s = 0
    kstar = Lw
    for k in range(Lw):
        acc_i += _fx(I[k])
        acc_s += _fx(score[k])
        cum_i[k] = _F(np.float64(acc_i) * 2.0 ** -FX_SHIFT)
        cum_s[k] = _F(np.float64(acc_s) * 2.0 ** -FX_SHIFT)
        neg = (acc_s < 0) if cfg.boundary_mode == BOUNDARY_CUMULATIVE else (score[k] < 0)
        if neg and kstar == Lw:
            kstar = k
    L = min(max(kstar, cfg.L_min), Lw)
    return L, score, cum_i, cum_s


# ------------------------------------------------------------------------------------------
# CAP-Decoding (Section 4.3, Algorithm 1)
# ------------------------------------------------------------------------------------------
def cap_select(conf: np.ndarray, masked: np.ndarray, xlogp: np.ndarray, block_len: int,
               tau_low: float, tau_high: float, gamma: float, mode: int = CAP_LITERAL):
    """Safe subset S of the masked positions of the block [0, block_len).

    conf, xlogp are used as fp32 (the precision the decision is taken in); D_ij is the
    fp32 sum xlogp[i, j] + xlogp[j, i]; i and j conflict iff D_ij > gamma.
    Returns the selected positions in ascending order.
    """
    c = np.asarray(conf, dtype=_F)
    x = np.asarray(xlogp, dtype=_F)
    tl, th, gm = _F(tau_low), _F(tau_high), _F(gamma)
    block = [i for i in range(int(block_len)) if masked[i]]           # M^t ∩ B^t
    if not block:
        return []

    def conflict(i, j):
        return bool(_F(x[i, j] + x[j, i]) > gm)

    pool = [i for i in block if c[i] >= tl]                            # Eq. (5)
    order = lambda items: sorted(items, key=lambda i: (-float(c[i]), i))
    S: list[int] = []
    if mode == CAP_LITERAL:
        S = [i for i in pool if c[i] >= th]                            # phase 1
        pool = [i for i in pool if i not in S and not any(conflict(i, s) for s in S)]
    else:
        for i in order([i for i in pool if c[i] >= th]):               # phase 1, checked
            if not any(conflict(i, s) for s in S):
                S.append(i)
        pool = [i for i in pool if i not in S and not any(conflict(i, s) for s in S)]
    remaining = order(pool)                                            # phase 2
    while remaining:
        i = remaining.pop(0)
        S.append(i)
        remaining = [j for j in remaining if not conflict(i, j)]
    if not S:                                                          # fallback
        S = [order(block)[0]]
    return sorted(S)


# ------------------------------------------------------------------------------------------
# one whole block-step for one sequence
# ------------------------------------------------------------------------------------------
def step(cfg: OracleConfig, w: OracleWeights, k_ctx, v_ctx, ctx_len: int,
         last_ids: np.ndarray, win_ids: np.ndarray, remain_len: int,
         influence: bool = True, h_final=None, n_layers: int | None = None,
         return_kv: bool = False, carried=None, pos0: int | None = None) -> dict:
    """All per-step outputs for one sequence.

    curr variant rows = last decoded block followed by the window; prev variant = the same
    rows with the last block's ids replaced by [MASK] (everything else fixed), so that
    p_prev = p(Z_k | c) and p_curr = p(Z_k | c, b).  h_final, if given, is
    (h_curr [W,d], h_prev [W,d] or None) and replaces the transformer stack's output.
    pos0: position of the first active row; default ctx_len (the rows follow the cached keys).
    With a dual cache the context also holds suffix rows, and the frontier's position is given.
    """
    pos0 = int(ctx_len if pos0 is None else pos0)
    Lb, W = len(last_ids), len(win_ids)
    have_prev = bool(influence and Lb > 0)
    if carried is not None:
        # p_prev carried from an earlier pass ("logits immediately before and after decoding B",
        # Implementation Approximation): carried = (rows [>= prev_len, d], prev_len); row k is the
        # LM-head input whose distribution is p_prev of window position k.  Positions without a
        # carried row get p_prev = p_curr, hence I_k = 0.  No second pass runs.
        influence = False
        have_prev = False
    if k_ctx is not None:
        k_ctx, v_ctx = k_ctx[:, :, :ctx_len, :], v_ctx[:, :, :ctx_len, :]
    if h_final is None:
        tok_curr = np.concatenate([last_ids, win_ids]).astype(np.int64)
        x = forward(cfg, w, tok_curr, pos0, k_ctx, v_ctx, n_layers=n_layers,
                    return_kv=return_kv)
        kv_last = None
        if return_kv:  # K / V of the last decoded block's rows, as this (curr) forward made them
            x, kv = x
            kv_last = [(k[:Lb], v[:Lb]) for k, v in kv]
        h_curr = final_hidden(cfg, w, x[Lb:])
        h_prev = None
        if have_prev:
            tok_prev = tok_curr.copy()
            tok_prev[:Lb] = cfg.mask_id
            xp = forward(cfg, w, tok_prev, pos0, k_ctx, v_ctx, n_layers=n_layers)
            h_prev = final_hidden(cfg, w, xp[Lb:])
    else:
        kv_last = None
        h_curr = _gemm_in(h_final[0], cfg)
        h_prev = _gemm_in(h_final[1], cfg) if have_prev else None
    if carried is not None:
        rows, n_prev = carried
        n_prev = int(n_prev)
        h_prev = np.array(h_curr, dtype=np.float64, copy=True)
        h_prev[:n_prev] = _gemm_in(np.asarray(rows, dtype=np.float64)[:n_prev], cfg)
        have_prev = n_prev > 0
    z = logits_of(h_curr, w.lm_head, cfg)
    zp = logits_of(h_prev, w.lm_head, cfg) if have_prev else None
    pred, conf, ent, infl, lse, lse_prev = signals_from_logits(z, zp)
    xl = cross_logprob(z, pred, lse)
    L, score, cum_i, cum_s = boundary(infl, ent, W, remain_len, have_prev, cfg)
    masked = np.asarray(win_ids) == cfg.mask_id
    sel = cap_select(conf, masked, xl, L, cfg.tau_low, cfg.tau_high, cfg.gamma, cfg.cap_mode)
    return dict(pred=pred, conf=conf, entropy=ent, influence=infl, lse=lse, lse_prev=lse_prev,
                xlogp=xl, block_len=L, score=score, cum_influence=cum_i, cum_score=cum_s,
                selected=sel, logits=z, logits_prev=zp, h_curr=h_curr, h_prev=h_prev,
                kv_last=kv_last)


# ------------------------------------------------------------------------------------------
# the decoding loop around the step (Section 3, Eq. 1-2; Section 4.2; Algorithm 1 per step)
# ------------------------------------------------------------------------------------------
def generate(cfg: OracleConfig, w: OracleWeights, k_ctx, v_ctx, ctx_len: int, gen_len: int,
             max_window: int, max_steps: int | None = None, carried: bool = False) -> dict:
    """Decode gen_len tokens after a cached context, one sequence.

    Every stage (Section 4.2): from the frontier, one forward over the last decoded block
    followed by L_window = min(L_max, remaining, max_window) masked positions gives I_k and
    H_k, hence the next block length L (L_min when nothing has been decoded yet).  The last
    block's K / V from that forward join the cache (block-wise cache reuse, Section 4.1).  The
    same forward's predictions already serve the new block: Algorithm 1 picks the subset of
    [0, L) to commit (Eq. 2).  Then the block's L positions are denoised alone - forward,
    Algorithm 1, Eq. 2 - until no [MASK] is left; the block becomes the last decoded block.
    carried: the boundary step takes p_prev from the LM-head rows the boundary step before it
    left for the same positions (rows L.. of its window) instead of a second pass.
    Returns tokens [gen_len], block_lens (list), nfe (forwards of the curr variant = steps) and
    a per-step trace (kind, pred, conf, selected, block_len, score, ids after the commit).
    """
    P0 = int(ctx_len)
    n_l = cfg.n_layers
    nkv, hd = cfg.n_kv_heads, cfg.head_dim
    kc = np.zeros((n_l, nkv, P0 + gen_len, hd))
    vc = np.zeros((n_l, nkv, P0 + gen_len, hd))
    if P0 > 0:
        kc[:, :, :P0] = np.asarray(k_ctx, dtype=np.float64)[:, :, :P0]
        vc[:, :, :P0] = np.asarray(v_ctx, dtype=np.float64)[:, :, :P0]
    cache = P0
    last = np.zeros(0, dtype=np.int64)
    tokens: list[int] = []
    block_lens: list[int] = []
    trace: list[dict] = []
    nfe = 0
    carry_rows = np.zeros((0, cfg.d_model))
    limit = 4 * gen_len if not max_steps or max_steps <= 0 else max_steps
    while len(tokens) < gen_len:
        remaining = gen_len - len(tokens)
        # ---- boundary step
        if nfe >= limit:
            raise RuntimeError("max_steps reached")
        W = min(cfg.L_max, max_window, remaining)
        win = np.full(W, cfg.mask_id, dtype=np.int64)
        if carried:
            r = step(cfg, w, kc, vc, cache, last, win, remaining, return_kv=True,
                     carried=(carry_rows, min(len(carry_rows), W)))
        else:
            r = step(cfg, w, kc, vc, cache, last, win, remaining, influence=True, return_kv=True)
        nfe += 1
        for l in range(n_l):        # the last block moves into the cache
            k_l, v_l = r["kv_last"][l]
            for j in range(len(last)):
                kc[l, :, cache + j] = k_l[j]
                vc[l, :, cache + j] = v_l[j]
        cache += len(last)
        last = np.zeros(0, dtype=np.int64)
        L = int(r["block_len"])
        carry_rows = r["h_curr"][L:]
        block_lens.append(L)
        for i in r["selected"]:
            win[i] = r["pred"][i]
        trace.append(dict(kind="boundary", pred=r["pred"], conf=r["conf"], selected=r["selected"],
                          block_len=L, score=r["score"], ids=win[:L].copy(),
                          influence=r["influence"], entropy=r["entropy"]))
        blk = win[:L].copy()
        # ---- denoising steps inside the block
        while np.any(blk == cfg.mask_id):
            if nfe >= limit:
                raise RuntimeError("max_steps reached")
            r = step(cfg, w, kc, vc, cache, last, blk, remaining, influence=False)
            nfe += 1
            # the block length is fixed now: Algorithm 1 runs over the whole block
            masked = blk == cfg.mask_id
            sel = cap_select(r["conf"], masked, r["xlogp"], L, cfg.tau_low, cfg.tau_high,
                             cfg.gamma, cfg.cap_mode)
            for i in sel:
                blk[i] = r["pred"][i]
            trace.append(dict(kind="denoise", pred=r["pred"], conf=r["conf"], selected=sel,
                              block_len=L, ids=blk.copy()))
        tokens.extend(int(t) for t in blk)
        last = blk.astype(np.int64)
    return dict(tokens=np.asarray(tokens, dtype=np.int64), block_lens=block_lens, nfe=nfe,
                trace=trace)
