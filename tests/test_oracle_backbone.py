"""Pins for the oracle's backbone pieces: library routines, closed forms, invariances."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import depcap_oracle as O


def _rng(seed=0):
    return np.random.default_rng(seed)


def test_bf16_round_matches_torch_conversion():
    r = _rng(1)
    x = np.concatenate([r.standard_normal(20000) * 10.0 ** r.integers(-6, 6, 20000),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38])])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    got = O.bf16_round(x)
    assert np.array_equal(got, want)
    # ties go to even: 1 + 2^-8 is exactly between 1 and 1 + 2^-7
    assert O.bf16_round(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert O.bf16_round(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_rmsnorm_matches_torch_and_unit_rms():
    r = _rng(2)
    x, g = r.standard_normal((7, 48)), r.standard_normal(48)
    want = F.rms_norm(torch.from_numpy(x), (48,), torch.from_numpy(g), eps=1e-5).numpy()
    assert np.allclose(O.rmsnorm(x, g, 1e-5), want, rtol=1e-12, atol=1e-12)
    y = O.rmsnorm(x, np.ones(48), 0.0)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0, atol=1e-12)


def test_rope_identity_norm_and_relative_property():
    r = _rng(3)
    x = r.standard_normal((5, 3, 16))
    assert np.allclose(O.rope(x, np.zeros(5), 10000.0), x)           # position 0 = identity
    y = O.rope(x, np.arange(5) + 11, 10000.0)
    assert np.allclose((y * y).sum(-1), (x * x).sum(-1))             # a rotation keeps norms
    # <rope(q,m), rope(k,n)> depends on m - n only
    q, k = r.standard_normal((1, 1, 16)), r.standard_normal((1, 1, 16))
    d1 = (O.rope(q, [7], 1e4) * O.rope(k, [3], 1e4)).sum()
    d2 = (O.rope(q, [107], 1e4) * O.rope(k, [103], 1e4)).sum()
    assert abs(d1 - d2) < 1e-9


def test_rope_matches_transformers_rotate_half():
    from transformers import LlamaConfig
    from transformers.models.llama.modeling_llama import (LlamaRotaryEmbedding,
                                                          apply_rotary_pos_emb)
    cfg = LlamaConfig(hidden_size=64, num_attention_heads=4, head_dim=16, rope_theta=10000.0,
                      max_position_embeddings=512)
    rot = LlamaRotaryEmbedding(cfg)
    r = _rng(4)
    x = r.standard_normal((6, 4, 16))
    pos = np.array([0, 1, 5, 17, 100, 301])
    xt = torch.from_numpy(x).permute(1, 0, 2)[None]                   # [1, heads, rows, hd]
    cos, sin = rot(xt, torch.from_numpy(pos)[None])
    want, _ = apply_rotary_pos_emb(xt, xt, cos.double(), sin.double())
    want = want[0].permute(1, 0, 2).numpy()
    # the library evaluates cos/sin in fp32: agreement to ~1e-5, far below any mis-pairing
    assert np.allclose(O.rope(x, pos, 10000.0), want, rtol=1e-4, atol=1e-4)


def test_attention_matches_sdpa_with_grouped_heads():
    r = _rng(5)
    q, k, v = r.standard_normal((9, 6, 8)), r.standard_normal((13, 2, 8)), \
        r.standard_normal((13, 2, 8))
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2)[None]
    want = F.scaled_dot_product_attention(tq, tk, tv, enable_gqa=True)[0].permute(1, 0, 2)
    got = O.attention(q, k, v, 6, 2)
    assert np.allclose(got, want.numpy(), rtol=1e-10, atol=1e-12)
    # grouped heads == the same KV heads repeated for plain multi-head attention
    got_mha = O.attention(q, np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1), 6, 6)
    assert np.allclose(got, got_mha)


def test_attention_single_key_and_key_permutation():
    r = _rng(6)
    q = r.standard_normal((4, 2, 8))
    k1, v1 = r.standard_normal((1, 2, 8)), r.standard_normal((1, 2, 8))
    out = O.attention(q, k1, v1, 2, 2)
    assert np.allclose(out, np.broadcast_to(v1, out.shape))          # one key: output = v
    k, v = r.standard_normal((11, 2, 8)), r.standard_normal((11, 2, 8))
    perm = r.permutation(11)
    assert np.allclose(O.attention(q, k, v, 2, 2), O.attention(q, k[perm], v[perm], 2, 2))


def _hf_model(n_q=4, n_kv=2, hd=8, d=32, ff=48, layers=2, vocab=97):
    from transformers import LlamaConfig, LlamaModel
    cfg = LlamaConfig(vocab_size=vocab, hidden_size=d, intermediate_size=ff,
                      num_hidden_layers=layers, num_attention_heads=n_q,
                      num_key_value_heads=n_kv, head_dim=hd, rms_norm_eps=1e-5,
                      rope_theta=10000.0, attention_bias=False, mlp_bias=False,
                      max_position_embeddings=256)
    cfg._attn_implementation = "eager"
    torch.manual_seed(0)
    m = LlamaModel(cfg).double().eval()
    with torch.no_grad():
        for n, p in m.named_parameters():
            if "norm" in n:
                p.copy_(1.0 + 0.1 * torch.randn_like(p))
    return cfg, m


def _oracle_weights_from_hf(m):
    sd = {k: v.detach().numpy() for k, v in m.state_dict().items()}
    w = O.OracleWeights(embed=sd["embed_tokens.weight"], final_norm=sd["norm.weight"],
                        lm_head=None)
    for l in range(len(m.layers)):
        p = f"layers.{l}."
        w.wq.append(sd[p + "self_attn.q_proj.weight"])
        w.wk.append(sd[p + "self_attn.k_proj.weight"])
        w.wv.append(sd[p + "self_attn.v_proj.weight"])
        w.wo.append(sd[p + "self_attn.o_proj.weight"])
        w.w_gate.append(sd[p + "mlp.gate_proj.weight"])
        w.w_up.append(sd[p + "mlp.up_proj.weight"])
        w.w_down.append(sd[p + "mlp.down_proj.weight"])
        w.norm1.append(sd[p + "input_layernorm.weight"])
        w.norm2.append(sd[p + "post_attention_layernorm.weight"])
    return w


def test_forward_matches_transformers_llama_bidirectional():
    """Whole stack (norms, rotate-half RoPE, grouped heads, SwiGLU, residuals, final norm)."""
    cfg, m = _hf_model()
    w = _oracle_weights_from_hf(m)
    ocfg = O.OracleConfig(n_layers=2, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8,
                          d_ff=48, vocab=97, mask_id=96)
    R, pos0 = 10, 5
    ids = torch.randint(0, 97, (1, R))
    with torch.no_grad():
        want = m(input_ids=ids, attention_mask=torch.zeros(1, 1, R, R, dtype=torch.float64),
                 position_ids=torch.arange(pos0, pos0 + R)[None]).last_hidden_state[0].numpy()
    x = O.forward(ocfg, w, ids[0].numpy(), pos0, None, None)
    got = O.rmsnorm(x, w.final_norm, 1e-5)
    assert np.allclose(got, want, rtol=1e-5, atol=1e-6)   # library RoPE tables are fp32


def test_forward_with_context_cache_matches_transformers_cache():
    """Active rows over an arbitrary cached context == the library model given that cache."""
    from transformers import DynamicCache
    cfg, m = _hf_model()
    w = _oracle_weights_from_hf(m)
    ocfg = O.OracleConfig(n_layers=2, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8,
                          d_ff=48, vocab=97, mask_id=96)
    R, P = 7, 12
    r = _rng(8)
    kc, vc = r.standard_normal((2, 2, P, 8)), r.standard_normal((2, 2, P, 8))
    cache = DynamicCache(config=cfg)
    for l in range(2):
        cache.update(torch.from_numpy(kc[l])[None], torch.from_numpy(vc[l])[None], l)
    ids = torch.randint(0, 97, (1, R))
    with torch.no_grad():
        want = m(input_ids=ids, past_key_values=cache,
                 attention_mask=torch.zeros(1, 1, R, P + R, dtype=torch.float64),
                 position_ids=torch.arange(P, P + R)[None]).last_hidden_state[0].numpy()
    x = O.forward(ocfg, w, ids[0].numpy(), P, kc, vc)
    got = O.rmsnorm(x, w.final_norm, 1e-5)
    assert np.allclose(got, want, rtol=1e-5, atol=1e-6)   # library RoPE tables are fp32


def test_forward_bf16_mode_rounds_only_gemm_inputs():
    """bf16 mode stays close to the exact stack and differs from it (rounding is applied)."""
    cfg, m = _hf_model()
    w = _oracle_weights_from_hf(m)
    kw = dict(n_layers=2, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48,
              vocab=97, mask_id=96)
    ids = np.arange(9) * 5 % 97
    x0 = O.forward(O.OracleConfig(**kw), w, ids, 3, None, None)
    x1 = O.forward(O.OracleConfig(bf16=True, **kw), w, ids, 3, None, None)
    err = np.abs(x1 - x0).max()
    assert 0 < err < 2e-2 * np.abs(x0).max()


def test_swiglu_matches_torch_silu():
    x = np.linspace(-8, 8, 101)
    assert np.allclose(O.silu(x), F.silu(torch.from_numpy(x)).numpy(), rtol=1e-12, atol=1e-15)


def test_forward_with_qkv_biases_matches_transformers_qwen2():
    """Biases on the q / k / v projections (none on the output projection), added before the
    rotation: the attention layers of the Qwen2 family, which the Dream backbone comes from."""
    from transformers import Qwen2Config, Qwen2Model
    cfg = Qwen2Config(vocab_size=97, hidden_size=32, intermediate_size=48, num_hidden_layers=2,
                      num_attention_heads=4, num_key_value_heads=2, rms_norm_eps=1e-5,
                      rope_theta=10000.0, max_position_embeddings=256, use_sliding_window=False)
    cfg._attn_implementation = "eager"
    torch.manual_seed(1)
    m = Qwen2Model(cfg).double().eval()
    with torch.no_grad():
        for n, p in m.named_parameters():
            if "norm" in n:
                p.copy_(1.0 + 0.1 * torch.randn_like(p))
            if n.endswith("proj.bias"):
                p.copy_(0.5 * torch.randn_like(p))
    w = _oracle_weights_from_hf(m)
    sd = {k: v.detach().numpy() for k, v in m.state_dict().items()}
    for l in range(2):
        w.bq.append(sd[f"layers.{l}.self_attn.q_proj.bias"])
        w.bk.append(sd[f"layers.{l}.self_attn.k_proj.bias"])
        w.bv.append(sd[f"layers.{l}.self_attn.v_proj.bias"])
    assert f"layers.0.self_attn.o_proj.bias" not in sd
    ocfg = O.OracleConfig(n_layers=2, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8,
                          d_ff=48, vocab=97, mask_id=96)
    R, pos0 = 10, 5
    ids = torch.randint(0, 97, (1, R))
    with torch.no_grad():
        want = m(input_ids=ids, attention_mask=torch.zeros(1, 1, R, R, dtype=torch.float64),
                 position_ids=torch.arange(pos0, pos0 + R)[None]).last_hidden_state[0].numpy()
    x = O.forward(ocfg, w, ids[0].numpy(), pos0, None, None)
    got = O.rmsnorm(x, w.final_norm, 1e-5)
    assert np.allclose(got, want, rtol=1e-5, atol=1e-6)
    # and the biases matter: without them the result is far off
    w.bq, w.bk, w.bv = [], [], []
    x0 = O.forward(ocfg, w, ids[0].numpy(), pos0, None, None)
    assert np.abs(O.rmsnorm(x0, w.final_norm, 1e-5) - want).max() > 1e-2
