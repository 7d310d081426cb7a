"""Brute-force information quantities on a small explicit joint distribution.

TEST INFRASTRUCTURE ONLY (see depcap_oracle.py).  Used to check, by enumeration, the
identities the paper's analysis of the dependency score rests on (Section 4.4 and the
appendix "Detailed Derivation"):

  * E_B[ KL(p(Z_k|c,B) || p(Z_k|c)) ] = I(Z_k; B | c)          (expected vs sample influence)
  * I(Z_{1:L}; B | c) = sum_k I(Z_k; B | c, Z_{<k})            (chain rule)
  * I(Z_{1:L}; B | c) = sum_k I(Z_k; B | c) - eps(L)            (additivity with correction)

The context c is fixed, so the joint is a table p[b, z_1, ..., z_L].
"""
from __future__ import annotations

import itertools

import numpy as np


def _entropy(p: np.ndarray) -> float:
    p = np.asarray(p, dtype=np.float64).ravel()
    nz = p[p > 0]
    return float(-(nz * np.log(nz)).sum())


def mutual_information(joint: np.ndarray, a_axes, b_axes, cond_axes=()) -> float:
    """I(A; B | C) from entropies: H(A,C) + H(B,C) - H(A,B,C) - H(C)."""
    n = joint.ndim

    def marg(keep):
        drop = tuple(i for i in range(n) if i not in keep)
        return joint.sum(axis=drop) if drop else joint

    a, b, c = tuple(a_axes), tuple(b_axes), tuple(cond_axes)
    h_c = _entropy(marg(c)) if c else 0.0
    return _entropy(marg(a + c)) + _entropy(marg(b + c)) - _entropy(marg(a + b + c)) - h_c


def sample_influence(joint: np.ndarray, k: int, b: int) -> float:
    """KL(p(Z_k | B=b) || p(Z_k)) by direct enumeration; axis 0 is B, axis k (1-based) Z_k."""
    n = joint.ndim
    drop = tuple(i for i in range(1, n) if i != k)
    pbz = joint.sum(axis=drop)                       # [B, Z_k]
    pz = pbz.sum(axis=0)
    pz_b = pbz[b] / pbz[b].sum()
    nz = pz_b > 0
    return float((pz_b[nz] * (np.log(pz_b[nz]) - np.log(pz[nz]))).sum())


def expected_influence(joint: np.ndarray, k: int) -> float:
    pb = joint.sum(axis=tuple(range(1, joint.ndim)))
    return float(sum(pb[b] * sample_influence(joint, k, b) for b in range(joint.shape[0])
                     if pb[b] > 0))


def cumulative_influence(joint: np.ndarray, L: int) -> float:
    """I(Z_{1:L}; B | c)."""
    return mutual_information(joint, tuple(range(1, L + 1)), (0,))


def overlap_correction(joint: np.ndarray, L: int) -> float:
    """eps(L) = sum_k [ I(Z_k;B|c) - I(Z_k;B|c,Z_{<k}) ]."""
    eps = 0.0
    for k in range(1, L + 1):
        eps += mutual_information(joint, (k,), (0,)) - \
            mutual_information(joint, (k,), (0,), tuple(range(1, k)))
    return eps


def independent_channels_joint(pb_parts, channels) -> np.ndarray:
    """Joint where B = (B_1..B_L) has independent parts and Z_k depends on B_k only.

    pb_parts[k]: distribution of B_k; channels[k][b_k, z]: p(Z_k = z | B_k = b_k).
    Axis 0 enumerates the tuples (b_1..b_L) in row-major order.  For this family eps(L) = 0.
    """
    L = len(pb_parts)
    sizes_b = [len(p) for p in pb_parts]
    sizes_z = [ch.shape[1] for ch in channels]
    joint = np.zeros([int(np.prod(sizes_b))] + sizes_z)
    for flat, bs in enumerate(itertools.product(*[range(s) for s in sizes_b])):
        pb = float(np.prod([pb_parts[k][bs[k]] for k in range(L)]))
        for zs in itertools.product(*[range(s) for s in sizes_z]):
            pz = float(np.prod([channels[k][bs[k], zs[k]] for k in range(L)]))
            joint[(flat,) + zs] = pb * pz
    return joint
