"""Brute-force check of the identities behind the cumulative-influence criterion
(Section 4.4; appendix 'Detailed Derivation')."""
import numpy as np

from oracle import depcap_oracle as O
from oracle import infotheory as T


def _random_joint(shape, seed):
    r = np.random.default_rng(seed)
    j = r.random(shape) ** 3
    return j / j.sum()


def test_expected_sample_influence_is_conditional_mutual_information():
    j = _random_joint((4, 3, 3, 3), 0)
    for k in (1, 2, 3):
        assert abs(T.expected_influence(j, k) - T.mutual_information(j, (k,), (0,))) < 1e-12


def test_sample_influence_equals_the_oracle_kl_on_the_same_distributions():
    """The KL the oracle computes from logits is the KL of the analysis."""
    j = _random_joint((4, 5, 3), 1)
    pbz = j.sum(axis=2)                                  # [B, Z_1]
    p_prev = pbz.sum(axis=0)
    for b in range(4):
        p_curr = pbz[b] / pbz[b].sum()
        infl = O.signals_from_logits(np.log(p_curr)[None], np.log(p_prev)[None] + 1.7)[3][0]
        assert abs(infl - T.sample_influence(j, 1, b)) < 1e-12


def test_chain_rule_and_additivity_with_overlap_correction():
    j = _random_joint((4, 3, 3, 3), 2)
    for L in (1, 2, 3):
        chain = sum(T.mutual_information(j, (k,), (0,), tuple(range(1, k)))
                    for k in range(1, L + 1))
        total = T.cumulative_influence(j, L)
        assert abs(total - chain) < 1e-12
        additive = sum(T.expected_influence(j, k) for k in range(1, L + 1))
        assert abs(total - (additive - T.overlap_correction(j, L))) < 1e-12


def test_no_overlap_when_block_parts_act_on_separate_positions():
    r = np.random.default_rng(3)
    parts = [np.array([0.3, 0.7]), np.array([0.6, 0.4]), np.array([0.5, 0.5])]
    chans = []
    for _ in range(3):
        c = r.random((2, 3)); chans.append(c / c.sum(axis=1, keepdims=True))
    j = T.independent_channels_joint(parts, chans)
    assert abs(j.sum() - 1) < 1e-12
    for L in (1, 2, 3):
        assert abs(T.overlap_correction(j, L)) < 1e-12
        additive = sum(T.expected_influence(j, k) for k in range(1, L + 1))
        assert abs(T.cumulative_influence(j, L) - additive) < 1e-12


def test_overlap_is_positive_when_positions_share_the_same_information():
    # Z_1 = Z_2 = B: the block tells both positions the same thing, the sum double counts
    j = np.zeros((3, 3, 3))
    for b in range(3):
        j[b, b, b] = 1 / 3
    assert T.overlap_correction(j, 2) > 0.5
    assert abs(T.cumulative_influence(j, 2) - np.log(3)) < 1e-12
