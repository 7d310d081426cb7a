"""Pins for the oracle's boundary rule (Section 4.2 / 4.4) and CAP-Decoding (Algorithm 1)."""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import depcap_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _cfg(**kw):
    base = dict(n_layers=0, d_model=1, n_q_heads=1, n_kv_heads=1, head_dim=1, d_ff=1, vocab=2,
                mask_id=1)
    base.update(kw)
    return O.OracleConfig(**base)


# ---------------------------------------------------------------- boundary -----------------
with open(os.path.join(GOLD, "boundary_cases.json")) as f:
    BOUNDARY_CASES = json.load(f)["cases"]


@pytest.mark.parametrize("case", BOUNDARY_CASES, ids=[c["name"] for c in BOUNDARY_CASES])
def test_boundary_hand_cases(case):
    cfg = _cfg(lam=case["lambda"], L_min=case["L_min"], L_max=case["L_max"],
               smooth_radius=case["smooth_radius"], norm_mode=case["norm_mode"],
               boundary_mode=case["mode"])
    I, H = np.array(case["influence"]), np.array(case["entropy"])
    L, score, cum_i, cum_s = O.boundary(I, H, len(I), case["remain"], case["have_prev"], cfg)
    assert L == case["block_len"]
    if "score" in case:
        assert np.array_equal(score, np.array(case["score"], dtype=np.float32))


def _random_signals(r, n):
    I = np.abs(r.standard_normal(n)) * np.exp(-np.arange(n) / 6.0)
    H = r.random(n) * 5 + 0.1
    return I.astype(np.float32), H.astype(np.float32)


def test_boundary_invariants_and_lambda_limits():
    r = np.random.default_rng(0)
    for trial in range(300):
        n = int(r.integers(1, 130))
        I, H = _random_signals(r, n)
        remain = int(r.integers(1, 300))
        for mode in (O.BOUNDARY_FIRST_NEG, O.BOUNDARY_CUMULATIVE):
            for norm in (O.NORM_MAX, O.NORM_MINMAX, O.NORM_NONE):
                cfg = _cfg(boundary_mode=mode, norm_mode=norm, smooth_radius=int(r.integers(0, 3)))
                Lw = min(cfg.L_max, remain, n)
                L, score, ci, cs = O.boundary(I, H, n, remain, True, cfg)
                assert min(cfg.L_min, Lw) <= L <= Lw and len(score) == Lw
                cfg0 = _cfg(boundary_mode=mode, norm_mode=norm, lam=0.0)
                if norm != O.NORM_MINMAX:        # I~ >= 0: no penalty -> whole window
                    assert O.boundary(I, H, n, remain, True, cfg0)[0] == Lw
                cfg_inf = _cfg(boundary_mode=mode, norm_mode=O.NORM_MAX, lam=1e9)
                assert O.boundary(I, H, n, remain, True, cfg_inf)[0] == min(cfg.L_min, Lw)


def test_boundary_is_monotone_in_lambda():
    r = np.random.default_rng(1)
    for trial in range(200):
        n = int(r.integers(8, 129))
        I, H = _random_signals(r, n)
        prev = None
        for lam in (0.2, 0.6, 0.8, 1.0, 1.2, 1.4, 1.6, 3.0):      # includes the swept range
            L = O.boundary(I, H, n, 256, True, _cfg(lam=lam))[0]
            if prev is not None:
                assert L <= prev
            prev = L


def test_cumulative_sums_are_prefix_sums_and_order_free():
    r = np.random.default_rng(2)
    I, H = _random_signals(r, 64)
    cfg = _cfg(norm_mode=O.NORM_NONE, smooth_radius=0, boundary_mode=O.BOUNDARY_CUMULATIVE)
    L, score, ci, cs = O.boundary(I, H, 64, 64, True, cfg)
    assert np.allclose(ci, np.cumsum(I.astype(np.float64)), rtol=1e-6, atol=1e-9)
    assert np.allclose(cs, np.cumsum(score.astype(np.float64)), rtol=1e-5, atol=1e-7)
    # fixed point: summing the same terms in any order gives the same total bit for bit
    fx = [O._fx(s) for s in score]
    assert sum(fx) == sum(reversed(fx)) == sum(sorted(fx))
    first_neg_cum = next((k for k in range(64) if sum(fx[:k + 1]) < 0), 64)
    assert L == min(max(first_neg_cum, cfg.L_min), 64)


def test_fx_rounding_is_half_to_even_of_the_scaled_value():
    assert O._fx(1.0) == 1 << 40 and O._fx(-0.5) == -(1 << 39)
    assert O._fx(np.float32(2.0 ** -41)) == 0 and O._fx(np.float32(3 * 2.0 ** -41)) == 2


# ---------------------------------------------------------------- CAP-Decoding -------------
with open(os.path.join(GOLD, "cap_cases.json")) as f:
    CAP_CASES = json.load(f)["cases"]


def _xlogp_from_conflicts(n, conflicts):
    x = np.full((n, n), -20.0, dtype=np.float32)
    for i, j in conflicts:
        x[i, j] = x[j, i] = -5.0
    return x


@pytest.mark.parametrize("case", CAP_CASES, ids=[c["name"] for c in CAP_CASES])
def test_cap_hand_cases(case):
    n = len(case["conf"])
    x = _xlogp_from_conflicts(n, case["conflicts"])
    args = (np.array(case["conf"]), np.array(case["masked"], dtype=bool), x, case["block_len"],
            case["tau_low"], case["tau_high"], case["gamma"])
    assert O.cap_select(*args, mode=O.CAP_LITERAL) == case["selected_literal"]
    assert O.cap_select(*args, mode=O.CAP_STRICT) == case["selected_strict"]


def _brute_force_greedy(order, conflict):
    """The greedy pass over `order` returns the lexicographically first maximal independent
    set (w.r.t. that order); found here by enumerating every subset."""
    n = len(order)
    best = None
    for bits in itertools.product([1, 0], repeat=n):          # 1 first: lexicographic order
        T = [order[t] for t in range(n) if bits[t]]
        if any(conflict(a, b) for a, b in itertools.combinations(T, 2)):
            continue
        if any(all(not conflict(o, t) for t in T) for o in order if o not in T):
            continue                                           # not maximal
        best = T
        break
    return best


def test_cap_exhaustive_invariants_small_blocks():
    r = np.random.default_rng(5)
    for trial in range(400):
        n = int(r.integers(1, 9))
        conf = np.round(r.random(n) * 0.4 + 0.6, 2).astype(np.float32)   # ties on purpose
        masked = r.random(n) < 0.85
        block_len = int(r.integers(1, n + 1))
        x = np.where(r.random((n, n)) < 0.3, -5.0, -20.0).astype(np.float32)
        gamma, tl, th = -16.0, 0.8, 0.95
        conflict = lambda i, j: bool(np.float32(x[i, j] + x[j, i]) > np.float32(gamma))
        block = [i for i in range(block_len) if masked[i]]
        for mode in (O.CAP_LITERAL, O.CAP_STRICT):
            S = O.cap_select(conf, masked, x, block_len, tl, th, gamma, mode)
            if not block:
                assert S == []
                continue
            assert S and set(S) <= set(block) and S == sorted(S)
            top = sorted(block, key=lambda i: (-float(conf[i]), i))[0]
            assert top in S                                    # "always decodes the top token"
            pool = [i for i in block if conf[i] >= np.float32(tl)]
            if not pool:
                assert S == [top]
                continue
            for i in pool:                                     # maximal within the pool
                assert i in S or any(conflict(i, s) for s in S)
            for a, b in itertools.combinations(S, 2):
                if conflict(a, b):
                    assert mode == O.CAP_LITERAL
                    assert conf[a] >= np.float32(th) and conf[b] >= np.float32(th)
            if mode == O.CAP_LITERAL:                          # independent re-derivation
                p1 = [i for i in pool if conf[i] >= np.float32(th)]
                rest = [i for i in pool if i not in p1 and not any(conflict(i, s) for s in p1)]
                rest = sorted(rest, key=lambda i: (-float(conf[i]), i))
                assert S == sorted(p1 + _brute_force_greedy(rest, conflict))


def test_cap_degenerate_settings_reduce_to_the_baselines():
    r = np.random.default_rng(6)
    for trial in range(100):
        n = int(r.integers(2, 40))
        conf = r.random(n).astype(np.float32)
        masked = np.ones(n, dtype=bool)
        x = (r.standard_normal((n, n)) * 10 - 15).astype(np.float32)
        # tau_low above 1: empty pool, exactly the single most confident token ("Vanilla")
        S = O.cap_select(conf, masked, x, n, 1.5, 2.0, -16.0)
        assert S == [int(np.argmax(conf))]
        # gamma = +inf: no conflicts, plain confidence-threshold decoding
        S = O.cap_select(conf, masked, x, n, 0.9, 0.95, np.inf)
        want = [i for i in range(n) if conf[i] >= np.float32(0.9)] or [int(np.argmax(conf))]
        assert S == want


def test_same_top1_token_at_two_confident_positions_conflicts_at_default_gamma():
    """If yhat_i = yhat_j then D_ij = log c_i + log c_j, far above gamma = -16."""
    z = np.zeros((2, 50)); z[0, 7] = 9.0; z[1, 7] = 8.0
    pred, conf, _, _, lse, _ = O.signals_from_logits(z, None)
    x = O.cross_logprob(z, pred, lse)
    assert np.isclose(x[0, 1] + x[1, 0], np.log(conf[0]) + np.log(conf[1]))
    S = O.cap_select(conf, np.array([True, True]), x, 2, 0.8, 0.999, -16.0)
    assert S == [0]
