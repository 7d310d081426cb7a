"""Pins for confidence / argmax / entropy / last-block influence (Eq. 3) and Eq. 6 halves."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import depcap_oracle as O


def _cfg(V, mask_id, forbid=True):
    return O.OracleConfig(n_layers=0, d_model=V, n_q_heads=1, n_kv_heads=1, head_dim=V, d_ff=1,
                          vocab=V, mask_id=mask_id, forbid_mask_pred=forbid)


def test_uniform_logits_closed_form():
    V = 50
    z = np.full((3, V), 0.37)
    pred, conf, ent, infl, lse, _ = O.signals_from_logits(z, z.copy())
    assert list(pred) == [0, 0, 0]                       # ties -> lowest id
    assert np.allclose(conf, 1.0 / V)
    assert np.allclose(ent, math.log(V))
    assert np.allclose(infl, 0.0, atol=1e-15)
    assert np.allclose(lse, 0.37 + math.log(V))


def test_forbidden_mask_id_leaves_the_softmax():
    V = 8
    cfg = _cfg(V, mask_id=3)
    h = np.eye(V)[[3, 5]] * 20.0                         # V = d, lm_head = I: logits = h
    z = O.logits_of(h, np.eye(V), cfg)
    pred, conf, ent, *_ = O.signals_from_logits(z, None)
    assert pred[0] != 3 and pred[0] == 0                 # mask logit removed, rest tie -> id 0
    assert np.isclose(conf[0], 1.0 / (V - 1)) and np.isclose(ent[0], math.log(V - 1))
    assert pred[1] == 5 and conf[1] > 0.99
    cfg2 = _cfg(V, mask_id=3, forbid=False)
    assert O.signals_from_logits(O.logits_of(h, np.eye(V), cfg2), None)[0][0] == 3


def test_spike_plus_uniform_binary_kl_closed_form():
    """p = (a, (1-a)/(V-1), ...), q = (b, (1-b)/(V-1), ...): KL reduces to the binary KL."""
    V, a, b = 40, 0.9, 0.3
    def logits(t):
        p = np.full(V, (1 - t) / (V - 1)); p[7] = t
        return np.log(p)[None, :] + 2.5                   # any shift must not matter
    pred, conf, ent, infl, lse, lse_p = O.signals_from_logits(logits(a), logits(b) - 4.0)
    want_kl = a * math.log(a / b) + (1 - a) * math.log((1 - a) / (1 - b))
    want_h = -a * math.log(a) - (1 - a) * math.log((1 - a) / (V - 1))
    assert pred[0] == 7 and np.isclose(conf[0], a)
    assert np.isclose(infl[0], want_kl, rtol=1e-12)
    assert np.isclose(ent[0], want_h, rtol=1e-12)
    assert np.isclose(lse[0], 2.5) and np.isclose(lse_p[0], -1.5)


def test_against_scipy_on_random_logits():
    r = np.random.default_rng(0)
    z, zp = r.standard_normal((6, 300)) * 3, r.standard_normal((6, 300)) * 3
    pred, conf, ent, infl, lse, _ = O.signals_from_logits(z, zp)
    p, q = scipy.special.softmax(z, axis=1), scipy.special.softmax(zp, axis=1)
    assert np.allclose(ent, scipy.stats.entropy(p, axis=1), rtol=1e-12)
    assert np.allclose(infl, scipy.special.rel_entr(p, q).sum(axis=1), rtol=1e-10)
    assert np.allclose(lse, scipy.special.logsumexp(z, axis=1), rtol=1e-13)
    assert np.array_equal(pred, p.argmax(axis=1))
    assert np.allclose(conf, p.max(axis=1), rtol=1e-13)
    assert np.allclose(conf, np.exp(z.max(axis=1) - lse))            # c = exp(m - lse)
    assert (ent >= 0).all() and (ent <= math.log(300) + 1e-12).all() and (infl >= 0).all()


def test_shift_invariance_and_kl_not_symmetric():
    r = np.random.default_rng(1)
    z, zp = r.standard_normal((4, 64)), r.standard_normal((4, 64))
    a = O.signals_from_logits(z, zp)
    b = O.signals_from_logits(z + 13.0, zp - 7.0)
    for x, y in zip(a[:4], b[:4]):
        assert np.allclose(x, y, rtol=1e-11, atol=1e-13)
    rev = O.signals_from_logits(zp, z)[3]
    assert not np.allclose(a[3], rev)                    # KL(curr||prev), not the reverse


def test_dominant_logit_limits():
    z = np.zeros((1, 100)); z[0, 42] = 60.0
    pred, conf, ent, infl, *_ = O.signals_from_logits(z, np.zeros((1, 100)))
    assert pred[0] == 42 and conf[0] > 1 - 1e-20 or np.isclose(conf[0], 1.0)
    assert ent[0] < 1e-20
    assert np.isclose(infl[0], math.log(100), rtol=1e-12)   # KL(delta || uniform) = log V


def test_identical_variants_give_zero_influence():
    r = np.random.default_rng(2)
    z = r.standard_normal((5, 128)) * 4
    assert np.all(O.signals_from_logits(z, z.copy())[3] == 0.0)


def test_cross_logprob_definition_and_diagonal():
    r = np.random.default_rng(3)
    z = r.standard_normal((5, 30)) * 2
    pred, conf, _, _, lse, _ = O.signals_from_logits(z, None)
    x = O.cross_logprob(z, pred, lse)
    logp = scipy.special.log_softmax(z, axis=1)
    for i in range(5):
        for j in range(5):
            assert np.isclose(x[i, j], logp[i, pred[j]], rtol=1e-12)   # log p_i(yhat_j)
    assert np.allclose(np.diag(x), np.log(conf))
    D = x + x.T                                                       # Eq. (6) is symmetric
    assert np.allclose(D, D.T)


def test_step_prev_variant_is_the_last_block_masked():
    """With V = d and an identity-like stack disabled (h_final hook) the step glue is checked:
    influence is zero iff both variants feed the same rows."""
    V = 16
    cfg = _cfg(V, mask_id=V - 1)
    w = O.OracleWeights(embed=np.eye(V), lm_head=np.eye(V), final_norm=np.ones(V))
    r = np.random.default_rng(4)
    h = r.standard_normal((6, V)) * 3
    win = np.full(6, V - 1)
    out = O.step(cfg, w, None, None, 0, np.array([1, 2]), win, 6, h_final=(h, h.copy()))
    assert np.all(out["influence"] == 0)
    out2 = O.step(cfg, w, None, None, 0, np.array([1, 2]), win, 6, h_final=(h, h * 0.5))
    assert np.all(out2["influence"] > 0)
    out3 = O.step(cfg, w, None, None, 0, np.array([], dtype=np.int64), win, 6,
                  h_final=(h, h * 0.5))
    assert np.all(out3["influence"] == 0) and out3["block_len"] == min(cfg.L_min, 6)
