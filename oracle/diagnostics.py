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


def compression_output_error(Q, K, V, budget, window, sink=0, merge=1, scale=None):
    """Mean relative error of the outputs of a budget-limited cache against full attention on one stream
    (the quantity behind the paper's merge-versus-eviction ablation, on whatever inputs the caller supplies).

    Q [T, n, G, d], K, V [T, n, d] for n independent lanes.  Runs Algorithm 1 (fp64 mode) twice: once with the given
    budget and once with a budget of T (nothing is ever compressed, i.e. full attention); returns the mean over steps
    t >= budget and lanes of |o_budget - o_full| / |o_full| and the number of compressions.
    """
    import oracle
    T, n, G, d = Q.shape
    kw = dict(window=window, sink=sink, group=G, dtype=oracle.F32, mode=oracle.MODE_DOUBLE)
    if scale is not None:
        kw["scale"] = scale
    small = oracle.Oracle(n, d, budget, merge=merge, **kw)
    full = oracle.Oracle(n, d, T, merge=1, **kw)
    errs, n_comp = [], 0
    for t in range(T):
        o_s, ev, _ = small.step(Q[t], K[t], V[t])
        o_f, _, _ = full.step(Q[t], K[t], V[t])
        n_comp += int((ev >= 0).sum())
        if t >= budget:
            num = np.linalg.norm((o_s - o_f).reshape(n, -1), axis=1)
            errs.append(num / np.linalg.norm(o_f.reshape(n, -1), axis=1))
    small.close()
    full.close()
    return float(np.mean(errs)), n_comp
