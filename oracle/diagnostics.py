"""Diagnostics from the paper's Ideal Merging section -- TEST INFRASTRUCTURE (numpy, fp64), not a product path.

ideal_merged_value: the value that replaces two adjacent values v1, v2 when k1 is dropped and k2 kept so that the
attention output of query q does not change (the closed form printed in the Ideal Merging section).
instant_convex_merge: the section's two-term approximation, a convex combination of v1 and v2 weighted by the
instantaneous exponentials of q.k1 and q.k2 (Algorithm 1 replaces those weights by historical average scores).
merge_perturbation: how far each way of compressing the pair that Algorithm 1 picks moves the attention output away
from the ideal merge's (which leaves it unchanged): Algorithm 1's weights, the instantaneous convex cut, plain eviction.
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


def merge_perturbation(Q, K, V, budget, window, sink=0, scale=None):
    """For every compressing step of Algorithm 1 (fp64 mode) on one stream, the distance between the attention output
    with the ideal merged value -- by the Ideal Merging section's identity, the output of the uncompressed cache -- and
    the output after compressing the picked pair (j, its right neighbour) in three ways:
      "algorithm1": the convex combination with Algorithm 1's historical average scores as weights (what the step does),
      "instant"   : the convex combination with the instantaneous exponentials of q_t.k_j and q_t.k_r as weights,
      "evict"     : the value of j dropped with its key (the paper's ablation).
    Each is measured for the step's own query q_t (the query the ideal value is built for) and for the next query
    q_{t+1} (which the ideal value of step t knows nothing about), relative to the norm of the uncompressed output.

    Q [T, n, 1, d], K, V [T, n, d] (single query head).  Returns {"now": {...}, "next": {...}, "ideal_residual": r,
    "steps": count} with the means over steps and lanes; ideal_residual is the same distance for the ideal value itself
    (zero up to rounding: the identity)."""
    import oracle
    T, n, G, d = Q.shape
    assert G == 1
    sc = scale if scale is not None else 1.0 / np.sqrt(d)
    ref = oracle.Oracle(n, d, budget, window=window, sink=sink, group=1, dtype=oracle.F32, mode=oracle.MODE_DOUBLE,
                        scale=0.0 if scale is None else scale)
    acc = {"now": {k: [] for k in ("algorithm1", "instant", "evict")}, "next": {k: [] for k in ("algorithm1", "instant", "evict")}}
    resid = []
    Qd, Kd, Vd = (np.asarray(x, np.float32).astype(np.float64) for x in (Q, K, V))
    for t in range(T):
        before = [ref.export(lane) for lane in range(n)] if ref.length(0) >= budget else None
        ref.step(Q[t], K[t], V[t])
        if before is None:
            continue
        for lane in range(n):
            j, wj, wr, _ = ref.last_step(lane)
            if j < 0:
                continue
            Kt = np.vstack([before[lane]["K"].astype(np.float64), Kd[t, lane][None]])      # the cache the step attends
            Vt = np.vstack([before[lane]["V"].astype(np.float64), Vd[t, lane][None]])
            r = j + 1
            keep = [i for i in range(len(Kt)) if i != j]
            order = [j, r] + [i for i in range(len(Kt)) if i not in (j, r)]
            q_now = Qd[t, lane, 0]
            v_ideal = ideal_merged_value(q_now, Kt[order], Vt[order], sc)
            v_inst, _ = instant_convex_merge(q_now, Kt[order], Vt[order], sc)
            variants = {"algorithm1": wj * Vt[j] + wr * Vt[r], "instant": v_inst, "evict": Vt[r].copy()}
            queries = {"now": q_now}
            if t + 1 < T:
                queries["next"] = Qd[t + 1, lane, 0]
            for when, q in queries.items():
                full = attention_output(q, Kt, Vt, sc)
                for name, vr in variants.items():
                    Vc = Vt.copy()
                    Vc[r] = vr
                    acc[when][name].append(np.linalg.norm(attention_output(q, Kt[keep], Vc[keep], sc) - full) / np.linalg.norm(full))
            Vc = Vt.copy()
            Vc[r] = v_ideal
            full = attention_output(q_now, Kt, Vt, sc)
            resid.append(np.linalg.norm(attention_output(q_now, Kt[keep], Vc[keep], sc) - full) / np.linalg.norm(full))
    ref.close()
    out = {when: {k: float(np.mean(v)) for k, v in d_.items()} for when, d_ in acc.items()}
    out["ideal_residual"] = float(np.max(resid))
    out["steps"] = len(resid)
    return out
