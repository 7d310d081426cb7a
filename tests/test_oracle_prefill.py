"""Pins of the oracle's prefill (K / V of a prompt from one bidirectional pass)."""
import numpy as np

from oracle import adapters
from oracle import depcap_oracle as O
from paper_2604_15750_b200 import Hyper, inputs

from parity import Case

TINY = inputs.WORKLOADS["tiny_f32"]


def _setup():
    case = Case(TINY, ctx_from_oracle=False)
    ids = case.prompt[0, :24].numpy().astype(np.int64)
    return case.ocfg, case.ow, ids


def test_first_layer_is_the_rotated_projection_of_the_normed_embedding():
    """Layer 0 has no attention before its K / V: K = RoPE(Wk . rmsnorm(E[id])), V = Wv . rmsnorm(E[id]),
    written out here with numpy alone."""
    cfg, w, ids = _setup()
    k, v = O.prefill(cfg, w, ids, ctx_len=0)
    E = np.asarray(w.embed, dtype=np.float64)[ids]
    a = E / np.sqrt((E * E).mean(axis=1, keepdims=True) + cfg.rms_eps) * np.asarray(w.norm1[0], dtype=np.float64)
    kk = (a @ np.asarray(w.wk[0], dtype=np.float64).T).reshape(len(ids), cfg.n_kv_heads, cfg.head_dim)
    vv = (a @ np.asarray(w.wv[0], dtype=np.float64).T).reshape(len(ids), cfg.n_kv_heads, cfg.head_dim)
    half = cfg.head_dim // 2
    pos = np.arange(len(ids))[:, None, None]
    ang = pos * cfg.rope_theta ** (-2.0 * np.arange(half) / cfg.head_dim)[None, None, :]
    x1, x2 = kk[..., :half], kk[..., half:]
    kr = np.concatenate([x1 * np.cos(ang) - x2 * np.sin(ang), x2 * np.cos(ang) + x1 * np.sin(ang)], axis=-1)
    assert np.abs(np.transpose(kr, (1, 0, 2)) - k[0]).max() < 1e-9
    assert np.abs(np.transpose(vv, (1, 0, 2)) - v[0]).max() < 1e-9


def test_the_pass_is_bidirectional_and_layer_zero_is_token_local():
    """Changing the LAST token leaves layer-0 K / V of the first token alone and changes its
    layer-1 K / V: every token attends the whole prompt, later tokens included."""
    cfg, w, ids = _setup()
    k, v = O.prefill(cfg, w, ids)
    ids2 = ids.copy()
    ids2[-1] = (ids2[-1] + 7) % (TINY.vocab - 1)
    k2, v2 = O.prefill(cfg, w, ids2)
    assert np.array_equal(k[0][:, 0], k2[0][:, 0]) and np.array_equal(v[0][:, 0], v2[0][:, 0])
    assert np.abs(k[1][:, 0] - k2[1][:, 0]).max() > 1e-6


def test_positions_start_after_the_cached_context():
    """With ctx_len cached keys the tokens sit at positions ctx_len + r: layer-0 K of a run
    prefilled behind a context equals layer-0 K of the same tokens placed there in a longer run."""
    cfg, w, ids = _setup()
    k_all, v_all = O.prefill(cfg, w, ids)
    k_tail, _ = O.prefill(cfg, w, ids[16:], k_all, v_all, ctx_len=16)
    assert np.abs(k_tail[0] - k_all[0][:, 16:]).max() < 1e-9


def test_suffix_rows_of_a_dual_cache_prefix_block_suffix_equals_one_whole_pass():
    """Dual cache (Section 5.2, cache compatibility): the cache holds the prefix AND the still masked
    suffix behind the window.  With suffix rows prefilled at their own positions (pos0 beyond the
    window), a step over the window alone sees exactly what one bidirectional pass over
    [prefix ; window ; suffix] sees: the window's layer-0 K / V and, through attention over both
    cached parts, its hidden states agree with the whole pass."""
    cfg, w, ids = _setup()
    P, Wn, S = 8, 6, 10                       # prefix, window, suffix lengths
    whole = ids[:P + Wn + S].copy()
    whole[P:] = cfg.mask_id                   # window and suffix are still masked
    x_whole, kv_whole = O.forward(cfg, w, whole, 0, None, None, return_kv=True)
    # caches: prefix rows and suffix rows taken from the whole pass (what a refresh would store)
    k_all = np.stack([np.transpose(k_, (1, 0, 2)) for k_, _ in kv_whole])     # [L, nkv, rows, hd]
    v_all = np.stack([np.transpose(v_, (1, 0, 2)) for _, v_ in kv_whole])
    keep = np.r_[0:P, P + Wn:P + Wn + S]
    x_win = O.forward(cfg, w, whole[P:P + Wn], P, k_all[:, :, keep], v_all[:, :, keep])
    assert np.abs(x_win - x_whole[P:P + Wn]).max() < 1e-9
    # and the position argument of prefill: suffix tokens prefilled at pos0 = P + Wn get the layer-0
    # K of the whole pass at those rows, whereas the default (positions = cache slots) does not
    k_suf, _ = O.prefill(cfg, w, whole[P + Wn:], k_all[:, :, :P], v_all[:, :, :P], ctx_len=P, pos0=P + Wn)
    assert np.abs(k_suf[0] - k_all[0][:, P + Wn:]).max() < 1e-9
    k_bad, _ = O.prefill(cfg, w, whole[P + Wn:], k_all[:, :, :P], v_all[:, :, :P], ctx_len=P)
    assert np.abs(k_bad[0] - k_all[0][:, P + Wn:]).max() > 1e-3
