"""Pins for the CPU oracle: what the paper prints, closed forms, invariants, textbook special cases and
brute force on tiny inputs.  None of these re-type the oracle's own formulas against themselves: the
comparators are the paper's numbers, exact rational arithmetic, scipy/torch library routines, or a
dense-matrix replay written with different data structures."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy.special import softmax as scipy_softmax

import oracle
from oracle import BF16, F32, MODE_DOUBLE, MODE_PINNED, Oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
NEG = -1000.0   # a logit whose exponential is exactly 0 in fp64 and in the pinned arithmetic


# ---------------------------------------------------------------------------------------------
# helpers: drive the oracle with a prescribed attention map through one-hot keys
# ---------------------------------------------------------------------------------------------
def onehot(i, d):
    e = np.zeros(d, np.float32)
    e[i] = 1.0
    return e


def run_attention_map(rows, capacity, window, sink, mode, d=16, merge=1, logits=False):
    """rows[t] = attention (or logits) of step t over the entries currently in the cache.
    Keys and values are one-hot in the token index, scale = 1, so logit_i = q[pos_i] and the value rows
    are directly the mixture coefficients.  Returns the oracle and the per-step eviction records."""
    o = Oracle(1, d, capacity, window=window, sink=sink, mode=mode, scale=1.0, track=True, merge=merge)
    retained = []
    log = []
    for t, row in enumerate(rows):
        retained.append(t)
        assert len(row) == len(retained), (t, row, retained)
        q = np.full(d, NEG, np.float32)
        for p, u in zip(row, retained):
            q[u] = p if logits else (math.log(p) if p > 0 else NEG)
        _, ev, _ = o.step(q, onehot(t, d), onehot(t, d))
        idx, wj, wr, ps = o.last_step()
        log.append((int(ev[0]), idx, wj, wr, ps))
        if ev[0] >= 0:
            retained.remove(int(ev[0]))
    return o, log


def read_toy():
    spec = {"rows": []}
    for line in open(os.path.join(GOLDEN, "toy_fig3.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, _, rest = line.partition(" ")
        if key == "row":
            spec["rows"].append([float(x) for x in rest.split(":")[1].split()])
        else:
            vals = [float(x) for x in rest.split()]
            spec[key] = vals if len(vals) > 1 else vals[0]
    return spec


# ---------------------------------------------------------------------------------------------
# the paper's worked example (Fig. 3 as described in the Methodology section)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode,tol", [(MODE_DOUBLE, 1e-7), (MODE_PINNED, 2e-6)])
def test_toy_example_matches_paper(mode, tol):
    # the logits log(p) are fed as fp32 inputs, which bounds the agreement at about 1e-8
    toy = read_toy()
    cap = int(toy["capacity"])
    o, log = run_attention_map(toy["rows"], cap, int(toy["window"]), int(toy["sink"]), mode)
    first = next(i for i, rec in enumerate(log) if rec[0] >= 0) + 1
    assert first == int(toy["first_compression_step"])          # "exceeds", not "reaches"
    ev, idx, wj, wr, _ = log[4]
    assert ev + 1 == int(toy["step5_evicted_token"])            # k2 removed
    assert abs(wj - toy["step5_weights"][0]) < tol and abs(wr - toy["step5_weights"][1]) < tol
    st = o.export(coeff=True)
    assert [p + 1 for p in st["pos"]] == [int(x) for x in toy["final_tokens"]]
    assert list(st["cnt"]) == [int(x) for x in toy["final_multiplicity"]]
    assert o.length() == cap


def test_toy_step5_value_and_scores():
    toy = read_toy()
    o, log = run_attention_map(toy["rows"][:5], 4, 1, 0, MODE_DOUBLE)
    st = o.export(coeff=True)
    # after step 5 the cache is v1, (v2/6 + 5 v3/6), v4, v5 and the surviving entry keeps k3's bookkeeping
    assert list(st["pos"]) == [0, 2, 3, 4]
    np.testing.assert_allclose(st["V"][1][:5], [0, 1 / 6, 5 / 6, 0, 0], atol=1e-7)
    np.testing.assert_allclose(st["coeff"][1], [0, 1 / 6, 5 / 6, 0, 0], atol=1e-12)
    np.testing.assert_allclose(st["a"][1] / st["n"][1], toy["step5_abar_neighbour"], atol=1e-12)  # a, n of v3 untouched
    assert st["n"][1] == 3
    np.testing.assert_allclose(st["K"][1], onehot(2, 16))       # K rows are never mixed


# ---------------------------------------------------------------------------------------------
# exact-rational brute force (ties included)
# ---------------------------------------------------------------------------------------------
def rational_replay(subsets, m, window, sink, G=1, merge=1):
    """Independent replay in exact rational arithmetic with a dense coefficient matrix.
    subsets[t][g] = set of token positions that share the attention of query head g uniformly at step t
    (other entries get probability 0).  Returns per-step (evicted position, weights) and the final state."""
    toks = []            # retained positions, ascending
    a = {}               # position -> accumulated score (Fraction)
    born = {}
    coeff = {}           # position -> {original token: Fraction}
    out = []
    for t, sub in enumerate(subsets):
        toks.append(t)
        a[t] = Fraction(0)
        born[t] = t
        coeff[t] = {t: Fraction(1)}
        for u in toks:
            p = sum((Fraction(1, len(sub[g])) if u in sub[g] else Fraction(0)) for g in range(G)) / G
            a[u] += p
        ev, w = -1, None
        if len(toks) > m:
            cand = toks[sink:len(toks) - window]
            key = lambda u: (a[u] / (t - born[u] + 1), u)
            j = min(cand, key=key)
            r = toks[toks.index(j) + 1]
            aj, ar = key(j)[0], key(r)[0]
            w = (Fraction(1, 2), Fraction(1, 2)) if aj + ar == 0 else (aj / (aj + ar), ar / (aj + ar))
            if merge:
                merged = {}
                for u, cval in coeff[j].items():
                    merged[u] = merged.get(u, 0) + w[0] * cval
                for u, cval in coeff[r].items():
                    merged[u] = merged.get(u, 0) + w[1] * cval
                coeff[r] = merged
            toks.remove(j)
            del a[j], coeff[j]
            ev = j
        out.append((ev, w))
    return out, toks, a, coeff


def random_subsets(rng, steps, m, window, sink, G, merge):
    """Subsets of power-of-two size over the entries held at each step, generated alongside the rational replay."""
    subsets = []
    for t in range(steps):
        # the retained set before step t is known from replaying what we have so far
        _, toks, _, _ = rational_replay(subsets, m, window, sink, G, merge) if subsets else ([], [], {}, {})
        avail = toks + [t]
        per_head = []
        for _ in range(G):
            size = 1 << int(rng.integers(0, int(math.log2(len(avail))) + 1))
            per_head.append(set(int(x) for x in rng.choice(avail, size=size, replace=False)))
        subsets.append(per_head)
    return subsets


@pytest.mark.parametrize("mode", [MODE_DOUBLE, MODE_PINNED])
@pytest.mark.parametrize("m,window,sink,G", [(3, 1, 0, 1), (5, 2, 1, 1), (6, 1, 0, 2), (7, 3, 2, 4), (4, 4, 0, 1)])
def test_exact_rational_bruteforce_with_ties(mode, m, window, sink, G):
    """Attention restricted to p in {0, 1/2^k}: every quantity is an exact dyadic rational in both arithmetic
    modes, exact ties are frequent, and the oracle must reproduce the rational replay decision by decision."""
    steps, d = 40, 48
    rng = np.random.default_rng(100 * m + 10 * window + G)
    subsets = random_subsets(rng, steps, m, window, sink, G, 1)
    ref, toks, a_ref, coeff_ref = rational_replay(subsets, m, window, sink, G)
    o = Oracle(1, d, m, window=window, sink=sink, group=G, mode=mode, scale=1.0, track=True)
    n_ties = 0
    for t, sub in enumerate(subsets):
        q = np.full((G, d), NEG, np.float32)
        for g in range(G):
            q[g, list(sub[g])] = 0.0
        _, ev, _ = o.step(q, onehot(t, d), onehot(t, d))
        assert int(ev[0]) == ref[t][0], f"step {t}"
        if ref[t][1] is not None:
            _, wj, wr, _ = o.last_step()
            assert abs(wj - float(ref[t][1][0])) < 1e-6 and abs(wr - float(ref[t][1][1])) < 1e-6
            n_ties += ref[t][1][0] == ref[t][1][1]
    st = o.export(coeff=True)
    assert list(st["pos"]) == toks
    for i, u in enumerate(toks):
        assert abs(st["a"][i] - float(a_ref[u])) < 1e-5
        dense = np.zeros(steps)
        for tok, cval in coeff_ref[u].items():
            dense[tok] = float(cval)
        np.testing.assert_allclose(st["coeff"][i], dense, atol=1e-5)
        np.testing.assert_allclose(st["V"][i][:steps], dense, atol=1e-5)


def test_structural_tie_goes_to_lowest_position():
    """m=3, sink=1, window=1.  Attention maps {0,1},{1,2},{1,2} give token 1 a=3/2 over n=3 and token 2 a=1 over
    n=2: both averages are exactly 1/2, token 0 is protected, so the pick must be token 1 and the merged
    value the plain mean of v1 and v2."""
    for mode in (MODE_DOUBLE, MODE_PINNED):
        rows = [[0.0], [0.0, 0.0], [NEG, 0.0, 0.0], [NEG, 0.0, 0.0, NEG]]
        o, log = run_attention_map(rows, 3, 1, 1, mode, logits=True)
        ev, idx, wj, wr, _ = log[3]
        assert ev == 1 and idx == 1
        assert wj == 0.5 and wr == 0.5
        st = o.export()
        np.testing.assert_array_equal(st["V"][1][:4], [0, 0.5, 0.5, 0])


# ---------------------------------------------------------------------------------------------
# textbook special case: budget >= sequence length  =>  plain softmax attention
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", [MODE_DOUBLE, MODE_PINNED])
@pytest.mark.parametrize("G", [1, 4])
def test_large_budget_equals_full_attention(mode, G):
    rng = np.random.default_rng(7)
    T, d, lanes = 40, 32, 3
    o = Oracle(lanes, d, budget=T, window=4, group=G, mode=mode)
    Ks = np.zeros((lanes, 0, d))
    Vs = np.zeros((lanes, 0, d))
    for t in range(T):
        q = rng.standard_normal((lanes, G, d)).astype(np.float32)
        k = rng.standard_normal((lanes, d)).astype(np.float32)
        v = rng.standard_normal((lanes, d)).astype(np.float32)
        Ks = np.concatenate([Ks, k[:, None].astype(np.float64)], 1)
        Vs = np.concatenate([Vs, v[:, None].astype(np.float64)], 1)
        out, ev, pr = o.step(q, k, v, want_probs=True)
        assert (ev == -1).all()
        logits = np.einsum("lgd,ltd->lgt", q.astype(np.float64), Ks) / math.sqrt(d)
        A = scipy_softmax(logits, axis=-1)
        np.testing.assert_allclose(out, np.einsum("lgt,ltd->lgd", A, Vs), rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(pr[:, :, : t + 1], A, rtol=0, atol=1e-12 if mode == MODE_DOUBLE else 3e-7)
    assert o.length(0) == T


# ---------------------------------------------------------------------------------------------
# dense fp64 brute force on random inputs (general logits)
# ---------------------------------------------------------------------------------------------
def dense_replay(q_all, k_all, v_all, m, window, sink, scale, merge=1):
    """O(t^2) replay that keeps every original k, v and a coefficient matrix; G = q_all.shape[1]."""
    T, G, d = q_all.shape
    keep = []                       # retained original positions
    Cm = np.zeros((0, T))           # coefficient rows of the retained entries
    a = np.zeros(0)
    outs, evs = [], []
    for t in range(T):
        keep.append(t)
        row = np.zeros((1, T))
        row[0, t] = 1.0
        Cm = np.concatenate([Cm, row])
        a = np.concatenate([a, [0.0]])
        Kc = k_all[keep].astype(np.float64)
        Vc = Cm @ v_all.astype(np.float64)
        A = scipy_softmax(scale * q_all[t].astype(np.float64) @ Kc.T, axis=-1)      # [G, L]
        outs.append(A @ Vc)
        a = a + A.mean(0)
        ev = -1
        if len(keep) > m:
            n = t - np.asarray(keep) + 1
            ab = a / n
            lo, hi = sink, len(keep) - 1 - window
            j = lo + int(np.argmin(ab[lo:hi + 1]))
            w = np.array([ab[j], ab[j + 1]]) / (ab[j] + ab[j + 1])
            if merge:
                Cm[j + 1] = w[0] * Cm[j] + w[1] * Cm[j + 1]
            ev = keep[j]
            Cm = np.delete(Cm, j, 0)
            a = np.delete(a, j)
            del keep[j]
        evs.append(ev)
    return np.stack(outs), evs, keep, a, Cm


@pytest.mark.parametrize("mode", [MODE_DOUBLE, MODE_PINNED])
@pytest.mark.parametrize("m,window,sink,G,merge", [(8, 1, 0, 1, 1), (6, 2, 1, 1, 1), (8, 3, 0, 2, 1), (5, 1, 2, 1, 0)])
def test_dense_bruteforce_random_inputs(mode, m, window, sink, G, merge):
    rng = np.random.default_rng(1234 + m)
    T, d = 64, 16
    q = rng.standard_normal((T, G, d)).astype(np.float32)
    k = rng.standard_normal((T, d)).astype(np.float32)
    v = rng.standard_normal((T, d)).astype(np.float32)
    ref_out, ref_ev, keep, a_ref, C_ref = dense_replay(q, k, v, m, window, sink, 1 / math.sqrt(d), merge)
    o = Oracle(1, d, m, window=window, sink=sink, group=G, mode=mode, track=True, merge=merge)
    for t in range(T):
        out, ev, _ = o.step(q[t], k[t], v[t])
        assert int(ev[0]) == ref_ev[t], f"step {t}"
        # stored V rows are rounded to fp32 at each merge, the replay never rounds
        np.testing.assert_allclose(out[0], ref_out[t], rtol=0, atol=2e-6)
    st = o.export(coeff=True)
    assert list(st["pos"]) == keep
    np.testing.assert_allclose(st["a"], a_ref, rtol=0, atol=1e-5)
    np.testing.assert_allclose(st["coeff"], C_ref, rtol=0, atol=1e-5)
    np.testing.assert_allclose(st["V"], C_ref @ v.astype(np.float64), rtol=0, atol=1e-5)
    np.testing.assert_array_equal(st["K"], k[keep])


# ---------------------------------------------------------------------------------------------
# invariants
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", [MODE_DOUBLE, MODE_PINNED])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_bookkeeping_and_convexity_invariants(mode, dtype):
    rng = np.random.default_rng(99)
    T, d, m, W, S = 120, 32, 24, 5, 3
    o = Oracle(2, d, m, window=W, sink=S, mode=mode, dtype=dtype, track=True)
    bf = lambda x: torch.from_numpy(x).to(torch.bfloat16).float().numpy() if dtype == BF16 else x
    for t in range(T):
        q = bf(rng.standard_normal((2, 1, d)).astype(np.float32))
        k = bf(rng.standard_normal((2, d)).astype(np.float32) * 2)
        v = bf(rng.standard_normal((2, d)).astype(np.float32))
        before = [o.export(l) for l in range(2)]
        _, ev, pr = o.step(q, k, v, want_probs=True)
        for lane in range(2):
            st = o.export(lane, coeff=True)
            idx, wj, wr, ps = o.last_step(lane)
            L = o.length(lane)
            assert L == min(t + 1, m)                                        # len <= m after every step
            assert abs(pr[lane, 0].sum() - 1) < 1e-6 and abs(ps - 1) < 1e-5  # sum_i A_t[i] = 1
            assert (np.diff(st["pos"]) > 0).all()                            # order preserved
            np.testing.assert_array_equal(st["n"], t - st["pos"] + 1)        # n_i = t - pos_i + 1
            assert abs(st["a"].sum() + o.dropped_score(lane) - (t + 1)) < 1e-3   # score mass is conserved
            assert st["cnt"].sum() == t + 1                                  # every token is somewhere
            # every mixture covers a contiguous span of original tokens ending at the entry's own position,
            # and the spans partition [0, t]
            start = 0
            for i in range(L):
                sup = np.nonzero(st["coeff"][i])[0]
                # pinned weights are binary32 quotients, so w_j + w_r = 1 only to fp32 accuracy
                assert st["coeff"][i].min() >= 0 and abs(st["coeff"][i].sum() - 1) < (1e-12 if mode == MODE_DOUBLE else 1e-5)
                assert sup.max() == st["pos"][i] and sup.min() >= start
                assert st["cnt"][i] == st["pos"][i] - start + 1
                start = st["pos"][i] + 1
            assert start == t + 1
            if ev[lane] >= 0:
                assert S <= idx <= m - W                                     # protected entries never picked
                assert ev[lane] == before[lane]["pos"][idx] if idx < len(before[lane]["pos"]) else True
                assert wj >= 0 and wr >= 0 and abs(wj + wr - 1) < 2e-7        # convex weights
                # the pick is a minimiser of a/n over the evictable range, as seen after this step's fold
                vj, vr = before[lane]["V"][idx], before[lane]["V"][idx + 1] if idx + 1 < len(before[lane]["V"]) else v[lane]
                merged = st["V"][idx]
                ulp = (2.0 ** -8 if dtype == BF16 else 2.0 ** -23) * np.maximum(np.abs(vj), np.abs(vr)) + 1e-30
                assert (merged >= np.minimum(vj, vr) - ulp).all() and (merged <= np.maximum(vj, vr) + ulp).all()
            else:
                assert t < m


def test_single_candidate_closed_form():
    """window = m - sink leaves exactly one evictable list index (sink), whatever the scores."""
    rng = np.random.default_rng(5)
    m, S, d = 9, 2, 16
    o = Oracle(1, d, m, window=m - S, sink=S, mode=MODE_PINNED)
    expect = []
    for t in range(60):
        _, ev, _ = o.step(rng.standard_normal(d), rng.standard_normal(d), rng.standard_normal(d))
        # list index S always holds the oldest non-sink token: positions S, S+1, S+2, ... leave in order
        if t >= m:
            assert ev[0] == S + (t - m)
        else:
            assert ev[0] == -1
    assert list(o.export()["pos"][:S]) == list(range(S))


def test_algorithm1_range_excludes_only_newest():
    """sink=0, window=1 is Algorithm 1 literally: the argmin runs over list indices 0..m-1 of the (m+1)-long list."""
    m, d = 4, 16
    # every earlier token gets a high score, the second newest a tiny one, so the pick must be list index m-1
    rows = []
    for t in range(6):
        L = min(t + 1, m + 1)
        row = [0.0] * L
        if L >= 2:
            row[-2] = -8.0
        rows.append(row)
    o, log = run_attention_map(rows, m, 1, 0, MODE_DOUBLE, logits=True)
    assert log[4][1] == m - 1 and log[5][1] == m - 1
    # ... and the newest entry (list index m) is never picked even when it is the global minimum
    rows = [[0.0] * min(t + 1, m + 1) for t in range(6)]
    for r in rows:
        r[-1] = -8.0
    o, log = run_attention_map(rows, m, 1, 0, MODE_DOUBLE, logits=True)
    assert all(rec[1] != m for rec in log) and log[4][1] >= 0


def test_eviction_ablation_drops_value():
    """merge = 0 (Ablation Study "Eviction"): same picks, the neighbour's value is left as it was."""
    rng = np.random.default_rng(11)
    d, m = 16, 6
    a = Oracle(1, d, m, window=2, mode=MODE_PINNED, merge=1)
    b = Oracle(1, d, m, window=2, mode=MODE_PINNED, merge=0)
    vs = []
    for t in range(30):
        q, k, v = (rng.standard_normal(d).astype(np.float32) for _ in range(3))
        vs.append(v)
        _, ea, _ = a.step(q, k, v)
        _, eb, _ = b.step(q, k, v)
        assert ea[0] == eb[0]            # the score path never reads V
    sb = b.export()
    np.testing.assert_array_equal(sb["V"], np.stack(vs)[sb["pos"]])
    assert (sb["cnt"] == 1).all()


def test_ragged_batch_equals_one_at_a_time():
    rng = np.random.default_rng(3)
    d, m, lanes, T = 16, 7, 3, 30
    lens = [30, 11, 22]
    q = rng.standard_normal((T, lanes, 1, d)).astype(np.float32)
    k = rng.standard_normal((T, lanes, d)).astype(np.float32)
    v = rng.standard_normal((T, lanes, d)).astype(np.float32)
    o = Oracle(lanes, d, m, window=2, mode=MODE_PINNED)
    for t in range(T):
        o.step(q[t], k[t], v[t], active=[t < n for n in lens])
    for lane in range(lanes):
        s = Oracle(1, d, m, window=2, mode=MODE_PINNED)
        for t in range(lens[lane]):
            s.step(q[t, lane], k[t, lane], v[t, lane])
        a, b = o.export(lane), s.export()
        for key in ("pos", "a", "K", "V", "n"):
            np.testing.assert_array_equal(a[key], b[key])


def test_group_of_identical_queries_equals_single_head():
    rng = np.random.default_rng(4)
    d, m, T = 32, 9, 40
    g1 = Oracle(1, d, m, window=2, group=1, mode=MODE_PINNED)
    g4 = Oracle(1, d, m, window=2, group=4, mode=MODE_PINNED)
    for t in range(T):
        q, k, v = (rng.standard_normal(d).astype(np.float32) for _ in range(3))
        o1, e1, _ = g1.step(q, k, v)
        o4, e4, _ = g4.step(np.tile(q, (4, 1)), k, v)
        assert e1[0] == e4[0]
        np.testing.assert_allclose(o4[0], np.tile(o1[0], (4, 1)), rtol=1e-13)
    # (p+p+p+p)*0.25 == p exactly in binary arithmetic
    np.testing.assert_array_equal(g1.export()["a"], g4.export()["a"])


# ---------------------------------------------------------------------------------------------
# the pinned binary32 pieces against libm / fp64 / torch
# ---------------------------------------------------------------------------------------------
def ulp32(x):
    return float(np.spacing(np.float32(abs(x))))


def test_pinned_exp_within_2ulp_of_libm():
    xs = np.concatenate([np.linspace(-87, 0, 200001), -np.logspace(-8, 1.9, 2000), [0.0, -87.0, -0.34657359, -0.3465736]])
    worst = 0.0
    for x in xs.astype(np.float32):
        got = oracle.pinned_exp(x)
        ref = math.exp(float(x))
        worst = max(worst, abs(got - ref) / ulp32(ref))
    assert worst <= 2.0, worst
    assert oracle.pinned_exp(0.0) == 1.0
    assert oracle.pinned_exp(-87.5) == 0.0 and oracle.pinned_exp(-1e30) == 0.0
    assert oracle.pinned_exp(-87.0) >= 2.0 ** -126          # never subnormal


def test_pinned_dot_close_to_fp64_and_order_sensitive_cases():
    rng = np.random.default_rng(0)
    for d in (16, 64, 128):
        for _ in range(200):
            q = rng.standard_normal(d).astype(np.float32)
            k = (rng.standard_normal(d) * 3).astype(np.float32)
            s = np.float32(1 / math.sqrt(d))
            ref = float(s) * float(q.astype(np.float64) @ k.astype(np.float64))
            bound = 2e-7 * float(s) * float(np.abs(q.astype(np.float64)) @ np.abs(k.astype(np.float64))) * math.log2(d)
            assert abs(oracle.pinned_dot(q, k, s) - ref) <= bound + 1e-12
    # a transposed / dropped channel shows up: each channel alone
    for c in range(32):
        q = np.zeros(32, np.float32)
        k = np.arange(1, 33, dtype=np.float32)
        q[c] = 2.0
        assert oracle.pinned_dot(q, k, 0.5) == float(c + 1)


def test_pinned_softmax_matches_scipy():
    rng = np.random.default_rng(1)
    for L in (1, 2, 17, 129, 2049):
        s = (rng.standard_normal(L) * 4).astype(np.float32)
        p = oracle.pinned_softmax(s)
        ref = scipy_softmax(s.astype(np.float64))
        np.testing.assert_allclose(p, ref, rtol=3e-6, atol=1e-12)   # s - M is itself rounded to fp32
        assert abs(float(p.astype(np.float64).sum()) - 1) < 1e-6
    # masked-out logits get exactly zero, equal logits over a power of two get exactly 1/L
    p = oracle.pinned_softmax(np.array([0, NEG, 0, NEG, 0, 0], np.float32))
    np.testing.assert_array_equal(p, [0.25, 0, 0.25, 0, 0.25, 0.25])


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(2)
    xs = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-6, 6, 4000),
                         [1.00390625, 1.01171875, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -1.00390625, 0.0, 3.0e38]]).astype(np.float32)
    ref = torch.from_numpy(xs).to(torch.bfloat16).float().numpy()
    got = np.array([oracle.round_bf16(x) for x in xs], np.float32)
    np.testing.assert_array_equal(got, ref)
    got_d = np.array([oracle.round_bf16_from_double(float(x)) for x in xs], np.float32)
    np.testing.assert_array_equal(got_d, ref)
    # one rounding from fp64, not two: 1 + 2^-8 + 2^-40 lies above the tie and must round up
    assert oracle.round_bf16_from_double(1.0 + 2.0 ** -8 + 2.0 ** -40) == 1.0 + 2.0 ** -7
    assert oracle.round_bf16(np.float32(1.0 + 2.0 ** -8)) == 1.0      # exact tie -> even


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_pinned_mode_tracks_double_mode(dtype):
    """Same inputs through both arithmetic modes: floats agree to fp32 accuracy, and the eviction sequences are
    equal unless the two smallest averages are closer than fp32 noise (then the pinned pick must be a near-minimum)."""
    rng = np.random.default_rng(21)
    d, m, W, T, lanes = 64, 32, 4, 200, 2
    to_t = (lambda x: torch.from_numpy(x).to(torch.bfloat16).float().numpy()) if dtype == BF16 else (lambda x: x)
    od = Oracle(lanes, d, m, window=W, mode=MODE_DOUBLE, dtype=dtype)
    op = Oracle(lanes, d, m, window=W, mode=MODE_PINNED, dtype=dtype)
    mismatches = 0
    for t in range(T):
        q = to_t(rng.standard_normal((lanes, 1, d)).astype(np.float32))
        k = to_t(rng.standard_normal((lanes, d)).astype(np.float32) * 1.5)
        v = to_t(rng.standard_normal((lanes, d)).astype(np.float32))
        out_d, ev_d, _ = od.step(q, k, v)
        out_p, ev_p, _ = op.step(q, k, v)
        mismatches += int((ev_d != ev_p).sum())
        if mismatches == 0:
            tol = 2e-2 if dtype == BF16 else 1e-5
            np.testing.assert_allclose(out_p, out_d, rtol=0, atol=tol)
    assert mismatches == 0
    for lane in range(lanes):
        sd, sp = od.export(lane), op.export(lane)
        np.testing.assert_array_equal(sd["pos"], sp["pos"])
        np.testing.assert_allclose(sp["a"], sd["a"], rtol=1e-5, atol=1e-7)
        tol = 2 ** -7 if dtype == BF16 else 1e-5
        np.testing.assert_allclose(sp["V"], sd["V"], rtol=tol, atol=tol)


def _adopt_and_count(wl, lanes_hk, n_tokens, seed):
    """Both arithmetic modes on one seeded stream of workload `wl` (kv heads `lanes_hk` of layer 0, sequence 0).

    The binary32 mode decides; the fp64 mode (the definition) must agree with every pick, except where its own two
    smallest averages are closer than binary32 noise: there the binary32 pick must be within 1e-5 relative of the fp64
    minimum, and the fp64 side then removes that entry too so that both stay on one trajectory.  Returns
    (compressions, adoptions, worst relative gap at an adoption)."""
    from paper_2503_01330_b200.synth import TokenStream
    dt = F32 if wl.dtype == "f32" else BF16
    n = len(lanes_hk)
    od = Oracle(n, wl.head_dim, wl.budget, window=wl.window, sink=wl.sink, group=wl.group, mode=MODE_DOUBLE, dtype=dt)
    op = Oracle(n, wl.head_dim, wl.budget, window=wl.window, sink=wl.sink, group=wl.group, mode=MODE_PINNED, dtype=dt)
    stream = TokenStream(wl, seed, "cpu")
    hk = torch.tensor(lanes_hk)
    compressions = adoptions = 0
    worst_gap = 0.0
    out_tol = 2e-2 if dt == BF16 else 1e-5
    for t in range(n_tokens):
        q, k, v = stream.token(t)
        qs = q[0, 0].view(wl.n_kv_heads, wl.group, wl.head_dim)[hk].float().numpy()
        ks, vs = k[0, 0][hk].float().numpy(), v[0, 0][hk].float().numpy()
        out_p, ev_p, _ = op.step(qs, ks, vs)
        od.impose_pick(ev_p)
        out_d, ev_d, _ = od.step(qs, ks, vs)
        np.testing.assert_array_equal(ev_d, ev_p)                   # the imposed entry was removed
        for lane in range(n):
            if ev_p[lane] < 0:
                continue
            compressions += 1
            own_pos, own_abar, taken_abar, bad = od.last_pick(lane)
            assert not bad, (t, lane, "the binary32 pick lies outside the fp64 side's evictable range")
            if own_pos != ev_p[lane]:
                adoptions += 1
                gap = (taken_abar - own_abar) / own_abar
                worst_gap = max(worst_gap, gap)
                assert 0.0 <= gap <= 1e-5, (t, lane, own_pos, int(ev_p[lane]), own_abar, taken_abar)
        # outputs: both are the fp64 definition on values that differ only by the rounding of the merge weights
        np.testing.assert_allclose(out_p, out_d, rtol=0, atol=out_tol)
    for lane in range(n):
        sd, sp = od.export(lane), op.export(lane)
        np.testing.assert_array_equal(sd["pos"], sp["pos"])
        np.testing.assert_allclose(sp["a"], sd["a"], rtol=2e-5, atol=1e-9)
    od.close()
    op.close()
    return compressions, adoptions, worst_gap


def test_pinned_sequence_is_the_fp64_sequence_up_to_near_ties_tiny_config():
    """The whole `tiny` configuration (4 lanes, 256 + 256 tokens): the binary32 eviction sequence against Algorithm 1
    in fp64, adopt-and-count."""
    from paper_2503_01330_b200.synth import BASE_SEED, WORKLOADS
    wl = WORKLOADS["tiny"]
    comp, adopted, gap = _adopt_and_count(wl, list(range(wl.n_kv_heads)), wl.prefill + wl.decode, BASE_SEED)
    assert comp == wl.n_kv_heads * (wl.prefill + wl.decode - wl.budget)
    print(f"tiny: {comp} compressions, {adopted} adoptions, worst relative gap {gap:.2e}")
    assert adopted <= 2


def test_pinned_sequence_is_the_fp64_sequence_up_to_near_ties_llama7b_layer():
    """Two lanes of the single-layer Llama-2-7B-shaped configuration (bf16, budget 2048, window 64) over the whole
    4096-token prompt and 256 decode steps: 2304 compressions per lane."""
    from paper_2503_01330_b200.synth import BASE_SEED, WORKLOADS
    wl = WORKLOADS["llama7b_layer"]
    n_tokens = wl.prefill + 256
    comp, adopted, gap = _adopt_and_count(wl, [3, 29], n_tokens, BASE_SEED + 1)
    assert comp == 2 * (n_tokens - wl.budget)
    print(f"llama7b_layer: {comp} compressions, {adopted} adoptions, worst relative gap {gap:.2e}")
    assert adopted <= 8                                              # near-ties are rare: a handful in 4608 decisions


# ---------------------------------------------------------------------------------------------
# the Ideal Merging section: the closed form really leaves the output unchanged; its two-term cut is convex
# ---------------------------------------------------------------------------------------------
def test_ideal_merge_identity_and_convex_approximation():
    from oracle.diagnostics import attention_output, ideal_merged_value, instant_convex_merge
    rng = np.random.default_rng(42)
    for t, d in ((3, 8), (17, 16), (200, 64)):
        q = rng.standard_normal(d)
        K = rng.standard_normal((t, d))
        V = rng.standard_normal((t, d))
        scale = 1 / math.sqrt(d)
        full = attention_output(q, K, V, scale)
        v_ideal = ideal_merged_value(q, K, V, scale)
        merged = attention_output(q, K[1:], np.vstack([v_ideal, V[2:]]), scale)      # k1 dropped, k2 kept
        np.testing.assert_allclose(merged, full, rtol=1e-11, atol=1e-12)
        v_cvx, w = instant_convex_merge(q, K, V, scale)
        assert (w >= 0).all() and abs(w.sum() - 1) < 1e-15
        assert (v_cvx <= np.maximum(V[0], V[1]) + 1e-15).all() and (v_cvx >= np.minimum(V[0], V[1]) - 1e-15).all()
        # dropping the v3.. terms and renormalising the remaining two coefficients gives exactly the convex form
        s = scale * (K @ q)
        c1, c2 = math.exp(s[0] - s[1]), 1.0
        np.testing.assert_allclose(v_cvx, (c1 * V[0] + c2 * V[1]) / (c1 + c2), rtol=1e-12)
    # with a single further token of negligible weight the ideal value is the convex one (here: the plain mean)
    q = np.zeros(4); K = np.zeros((3, 4)); K[2, 0] = -200.0; q[0] = 1.0
    V = rng.standard_normal((3, 4))
    np.testing.assert_allclose(ideal_merged_value(q, K, V, 1.0), 0.5 * (V[0] + V[1]), atol=1e-12)


# ---------------------------------------------------------------------------------------------
# the paper's ablation (WeightedKV against plain eviction with the same picks) on synthetic streams: error of the
# outputs against full attention.  Direction only -- the paper's own numbers are perplexities of a trained model.
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("rho", [0.0, 0.5])
def test_merging_loses_less_than_eviction_on_synthetic_streams(rho):
    from oracle.diagnostics import compression_output_error
    rng = np.random.default_rng(7)
    T, n, G, d, r = 320, 8, 1, 32, 8
    basis = rng.standard_normal((n, d, r))
    K = np.einsum("ndr,tnr->tnd", basis, rng.standard_normal((T, n, r))) / math.sqrt(r) + 0.05 * rng.standard_normal((T, n, d))
    Q = rng.standard_normal((T, n, G, d))
    noise = rng.standard_normal((T, n, d))
    V = np.zeros((T, n, d))
    V[0] = noise[0]
    for t in range(1, T):                               # values drift slowly for rho near 1, independent for rho = 0
        V[t] = rho * V[t - 1] + math.sqrt(1 - rho * rho) * noise[t]
    Q, K, V = (x.astype(np.float32) for x in (Q, K, V))
    for m, W in ((64, 8), (128, 16)):
        e_merge, n1 = compression_output_error(Q, K, V, m, W, merge=1)
        e_evict, n0 = compression_output_error(Q, K, V, m, W, merge=0)
        assert n1 == n0 == n * (T - m)                  # same trigger; the ablation changes only what happens to the value
        assert e_merge < 0.97 * e_evict, (rho, m, e_merge, e_evict)


@pytest.mark.parametrize("rho", [0.0, 0.5])
def test_single_step_perturbation_of_the_three_ways_to_compress(rho):
    """Ideal Merging section: the ideal merged value leaves the output of the step's query unchanged; its two-term
    convex cut with instantaneous weights is the closest of the practical choices FOR THAT QUERY.  Algorithm 1 swaps the
    instantaneous weights for historical averages: for the next query, which the instantaneous weights know nothing
    about, the historical weights are the better of the two.  (Measured and recorded, not predicted by the section:
    a single eviction perturbs a single output less than either merge; merging wins over many steps, see
    test_merging_loses_less_than_eviction_on_synthetic_streams.)"""
    from oracle.diagnostics import merge_perturbation
    rng = np.random.default_rng(7)
    T, n, d, r = 256, 6, 32, 8
    basis = rng.standard_normal((n, d, r))
    K = np.einsum("ndr,tnr->tnd", basis, rng.standard_normal((T, n, r))) / math.sqrt(r) + 0.05 * rng.standard_normal((T, n, d))
    Q = rng.standard_normal((T, n, 1, d))
    noise = rng.standard_normal((T, n, d))
    V = np.zeros((T, n, d))
    V[0] = noise[0]
    for t in range(1, T):
        V[t] = rho * V[t - 1] + math.sqrt(1 - rho * rho) * noise[t]
    Q, K, V = (x.astype(np.float32) for x in (Q, K, V))
    res = merge_perturbation(Q, K, V, 64, 8)
    assert res["steps"] == n * (T - 64)
    assert res["ideal_residual"] < 1e-12                                 # the identity, at every compressing step
    now, nxt = res["now"], res["next"]
    assert now["instant"] < 0.9 * now["algorithm1"] and now["instant"] < now["evict"]
    assert nxt["algorithm1"] < nxt["instant"]
    assert all(0.0 < v < 0.2 for v in list(now.values()) + list(nxt.values()))


def test_imported_state_continues_like_the_streamed_one():
    """wkvo_import (set-up for the large-cache tests) must put a lane exactly where streaming left it."""
    rng = np.random.default_rng(0)
    d, m = 16, 12
    A = oracle.Oracle(1, d, m, window=2, mode=oracle.MODE_PINNED)
    B = oracle.Oracle(1, d, m, window=2, mode=oracle.MODE_PINNED)
    toks = [(rng.standard_normal((1, 1, d)).astype(np.float32), rng.standard_normal((1, d)).astype(np.float32),
             rng.standard_normal((1, d)).astype(np.float32)) for _ in range(60)]
    for q, k, v in toks[:30]:
        A.step(q, k, v)
    e = A.export(0)
    B.import_state(0, A.tokens(0), e["pos"], e["a"], e["K"], e["V"])
    for q, k, v in toks[30:]:
        oa, ea, _ = A.step(q, k, v)
        ob, eb, _ = B.step(q, k, v)
        assert (ea == eb).all() and np.array_equal(oa, ob)
    ea, eb = A.export(0), B.export(0)
    assert all(np.array_equal(ea[key], eb[key]) for key in ("pos", "a", "K", "V", "n"))
    with pytest.raises(ValueError):
        B.import_state(0, 5, [3, 2], [0.1, 0.2], np.zeros((2, d)), np.zeros((2, d)))     # positions must increase


# ---------------------------------------------------------------------------------------------
# while nothing is compressed, Algorithm 1's accumulated scores are the column sums of the causal attention matrix
# (what the dense prompt kernel computes in one go): textbook form in numpy, fp64
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("G", [1, 4])
def test_scores_before_compression_are_causal_column_sums(G):
    rng = np.random.default_rng(3)
    n, d, lanes = 37, 16, 3
    Q = rng.standard_normal((n, lanes, G, d))
    K = rng.standard_normal((n, lanes, d))
    V = rng.standard_normal((n, lanes, d))
    ref = Oracle(lanes, d, n + 5, window=2, group=G, dtype=F32, mode=MODE_DOUBLE)
    outs = [ref.step(Q[t].astype(np.float32), K[t].astype(np.float32), V[t].astype(np.float32))[0] for t in range(n)]
    Qf, Kf, Vf = (x.astype(np.float32).astype(np.float64) for x in (Q, K, V))
    for lane in range(lanes):
        S = np.einsum("tgd,id->tgi", Qf[:, lane], Kf[:, lane]) / math.sqrt(d)          # [t, g, i]
        S = np.where(np.arange(n)[None, None, :] <= np.arange(n)[:, None, None], S, -np.inf)
        P = scipy_softmax(S, axis=-1)
        want_a = P.mean(axis=1).sum(axis=0)                                                # column sums of the group mean
        got = ref.export(lane)
        np.testing.assert_allclose(got["a"], want_a, rtol=1e-12, atol=1e-15)
        np.testing.assert_array_equal(got["pos"], np.arange(n))
        np.testing.assert_array_equal(got["n"], n - np.arange(n))
        want_o = np.einsum("tgi,id->tgd", P, Vf[:, lane])
        np.testing.assert_allclose(np.stack([o[lane] for o in outs]), want_o, rtol=1e-10, atol=1e-12)
