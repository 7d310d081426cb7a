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
