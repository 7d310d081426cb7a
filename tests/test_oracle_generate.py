"""Pins of the oracle's decoding loop (Section 3 Eq. 1-2, Section 4.2, Algorithm 1 per step)
against what the definitions fix: counts in the two limiting threshold settings, structural
invariants, and a brute-force sequential decoder written here without the loop's bookkeeping."""
import numpy as np
import pytest

from oracle import adapters
from oracle import depcap_oracle as O
from paper_2604_15750_b200 import Hyper, inputs

from parity import Case

TINY = inputs.WORKLOADS["tiny_f32"]
GEN = 24


def _case(hyper, scale=25.0):
    case = Case(TINY, ctx_from_oracle=True, hyper=hyper)
    case.weights["lm_head"] = case.weights["lm_head"] * scale     # peaked predictions
    case.ow = adapters.weights_from_torch(case.weights)
    kc, vc = adapters.to_np(case.k_log[:, 0]), adapters.to_np(case.v_log[:, 0])
    return case, kc, vc


def test_one_commit_per_step_costs_one_forward_per_token():
    """tau_low above every confidence: the pool (Eq. 5) is empty, the fallback commits exactly one
    position per step, so NFE == tokens, whatever the block lengths."""
    case, kc, vc = _case(Hyper(tau_low=2.0, tau_high=2.0, L_min=4, L_max=16))
    r = O.generate(case.ocfg, case.ow, kc, vc, 64, GEN, 32)
    assert r["nfe"] == GEN
    assert all(len(t["selected"]) == 1 for t in r["trace"])


def test_commit_everything_costs_one_forward_per_block():
    """tau_high = 0 with the literal phase 1: every masked position of the block commits in the
    boundary step itself, so NFE == number of blocks and the tokens are that step's argmax."""
    case, kc, vc = _case(Hyper(tau_low=0.0, tau_high=0.0, L_min=4, L_max=16))
    r = O.generate(case.ocfg, case.ow, kc, vc, 64, GEN, 32)
    assert r["nfe"] == len(r["block_lens"])
    assert all(t["kind"] == "boundary" for t in r["trace"])
    got = np.concatenate([t["pred"][:t["block_len"]] for t in r["trace"]])
    assert np.array_equal(got, r["tokens"])


@pytest.mark.parametrize("lam,norm", [(0.8, 2), (1.2, 0), (0.3, 1)])
def test_structure_of_a_generation(lam, norm):
    hy = Hyper(tau_low=0.3, tau_high=0.6, lam=lam, norm_mode=norm, L_min=4, L_max=16)
    case, kc, vc = _case(hy)
    r = O.generate(case.ocfg, case.ow, kc, vc, 64, 48, 32)
    assert len(r["tokens"]) == 48 and sum(r["block_lens"]) == 48
    assert not np.any(r["tokens"] == TINY.mask_id)
    done = 0
    for L in r["block_lens"]:
        Lw = min(hy.L_max, 48 - done, 32)
        assert min(hy.L_min, Lw) <= L <= Lw                 # clip of Section 4.2
        done += L
    assert r["block_lens"][0] == hy.L_min                   # cold start
    assert len(r["block_lens"]) <= r["nfe"] <= 48
    # Eq. (2): a committed id never changes afterwards, and every step commits something
    ids_prev, n_boundary = None, 0
    for t in r["trace"]:
        assert len(t["selected"]) >= 1
        if t["kind"] == "boundary":
            n_boundary += 1
            ids_prev = None
        if ids_prev is not None:
            keep = ids_prev != TINY.mask_id
            assert np.array_equal(t["ids"][keep], ids_prev[keep])
        ids_prev = t["ids"]
    assert n_boundary == len(r["block_lens"])


def test_against_a_brute_force_sequential_decoder():
    """Fixed block length (L_min = L_max) and one commit per step: the loop must reproduce a
    decoder that keeps every block's K / V in a list, rebuilds the cache by concatenation each
    step and decodes the most confident masked position of the block, nothing else."""
    Lb = 4
    case, kc, vc = _case(Hyper(tau_low=2.0, tau_high=2.0, L_min=Lb, L_max=Lb))
    cfg, w = case.ocfg, case.ow
    r = O.generate(cfg, w, kc, vc, 64, 12, 32)
    assert r["block_lens"] == [Lb] * 3

    def probs(x_rows):
        z = O.logits_of(O.final_hidden(cfg, w, x_rows), w.lm_head, cfg)
        z = z - z.max(axis=1, keepdims=True)
        p = np.exp(z)
        return p / p.sum(axis=1, keepdims=True)

    kv_blocks = [(np.asarray(kc, dtype=np.float64)[:, :, :64], np.asarray(vc, dtype=np.float64)[:, :, :64])]
    last = np.zeros(0, dtype=np.int64)
    out = []
    for _ in range(3):
        k_all = np.concatenate([k for k, _ in kv_blocks], axis=2)
        v_all = np.concatenate([v for _, v in kv_blocks], axis=2)
        P = k_all.shape[2]
        blk = np.full(Lb, cfg.mask_id, dtype=np.int64)
        # first forward of the stage sees the last block as active rows
        x, kv = O.forward(cfg, w, np.concatenate([last, blk]), P, k_all, v_all, return_kv=True)
        p = probs(x[len(last):])
        if len(last):
            kv_blocks.append((np.stack([np.transpose(k[:len(last)], (1, 0, 2)) for k, _ in kv]),
                              np.stack([np.transpose(v[:len(last)], (1, 0, 2)) for _, v in kv])))
            k_all = np.concatenate([k for k, _ in kv_blocks], axis=2)
            v_all = np.concatenate([v for _, v in kv_blocks], axis=2)
        while True:
            conf = p.max(axis=1)
            conf[blk != cfg.mask_id] = -1.0
            i = int(np.argmax(conf))
            blk[i] = int(np.argmax(p[i]))
            if not np.any(blk == cfg.mask_id):
                break
            p = probs(O.forward(cfg, w, blk, k_all.shape[2], k_all, v_all))
        out.extend(blk.tolist())
        last = blk.copy()
    assert out == r["tokens"].tolist()


def test_carried_prev_generation_keeps_the_structure_and_the_cold_start():
    """With p_prev carried between boundary steps the loop has the same structure; the first block
    is the cold start, and a later block never reaches beyond the positions that had a carried
    row (window of the boundary step before it, minus its block)."""
    hy = Hyper(tau_low=0.3, tau_high=0.6, lam=0.8, norm_mode=2, L_min=4, L_max=16)
    case, kc, vc = _case(hy)
    r = O.generate(case.ocfg, case.ow, kc, vc, 64, 48, 32, carried=True)
    assert sum(r["block_lens"]) == 48 and not np.any(r["tokens"] == TINY.mask_id)
    assert r["block_lens"][0] == hy.L_min
    done, prev_w = 0, None
    for i, L in enumerate(r["block_lens"]):
        W = min(hy.L_max, 48 - done, 32)
        if i > 0:
            carried_rows = prev_w - r["block_lens"][i - 1]
            assert L <= max(min(carried_rows, W), min(hy.L_min, W))
        prev_w, done = W, done + L
