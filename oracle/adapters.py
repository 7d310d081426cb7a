"""Marshalling between seeded torch inputs and the numpy oracle.  TEST INFRASTRUCTURE ONLY.

No arithmetic: bf16/fp32 torch tensors become float32 numpy arrays (exact), workload
descriptions become OracleConfig.
"""
from __future__ import annotations

import numpy as np
import torch

from .depcap_oracle import OracleConfig, OracleWeights


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def weights_from_torch(wd: dict) -> OracleWeights:
    w = OracleWeights(embed=to_np(wd["embed"]), final_norm=to_np(wd["final_norm"]),
                      lm_head=to_np(wd["lm_head"]))
    for lw in wd["layers"]:
        for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2"):
            getattr(w, name).append(to_np(lw[name]))
        if "bq" in lw:
            for name in ("bq", "bk", "bv"):
                getattr(w, name).append(to_np(lw[name]))
    return w


def config_from_workload(wl, **overrides) -> OracleConfig:
    cfg = OracleConfig(n_layers=wl.n_layers, d_model=wl.d_model, n_q_heads=wl.n_q_heads,
                       n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim, d_ff=wl.d_ff,
                       vocab=wl.vocab, mask_id=wl.mask_id, bf16=(wl.dtype == "bf16"),
                       rms_eps=wl.rms_eps, rope_theta=wl.rope_theta)
    for k, v in overrides.items():
        setattr(cfg, k, v)
    return cfg
