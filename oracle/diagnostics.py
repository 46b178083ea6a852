"""Diagnostics from the paper's Ideal Merging section -- TEST INFRASTRUCTURE (numpy, fp64), not a product path.

ideal_merged_value: the value that replaces two adjacent values v1, v2 when k1 is dropped and k2 kept so that the
attention output of query q does not change (the closed form printed in the Ideal Merging section).
instant_convex_merge: the section's two-term approximation, a convex combination of v1 and v2 weighted by the
instantaneous exponentials of q.k1 and q.k2 (Algorithm 1 replaces those weights by historical average scores).
"""
import numpy as np


def attention_output(q, K, V, scale):
    s = scale * (K @ q)
    e = np.exp(s - s.max())
    return (e / e.sum()) @ V


def ideal_merged_value(q, K, V, scale):
    """K, V [t, d] with the pair to compress at rows 0 and 1; returns v~ [d]."""
    s = scale * (K @ q)
    e = np.exp(s - s.max())
    S = e.sum()
    ratio = np.exp(s[0] - s[1])                       # e^{q.(k1 - k2)/sqrt(d)}
    return (1.0 - e[0] / S) * (ratio * V[0] + V[1]) - (ratio / S) * (e[2:] @ V[2:])


def instant_convex_merge(q, K, V, scale):
    s = scale * (K[:2] @ q)
    w = np.exp(s - s.max())
    w = w / w.sum()
    return w[0] * V[0] + w[1] * V[1], w
