"""CUDA library vs CPU oracle on the same seeded inputs, through the C ABI.  Eviction positions, retained
positions and accumulated scores are compared bit for bit; attention outputs and merged values within the
tolerances stated in parity_util."""
import numpy as np
import pytest
import torch

from paper_2503_01330_b200 import binding
from paper_2503_01330_b200.synth import WORKLOADS, Workload

from parity_util import Parity, assert_close

pytestmark = pytest.mark.gpu


def small(name="s", layers=1, batch=2, hq=4, hkv=4, d=64, dtype="f32", m=40, W=4, S=0, rank=0):
    return Workload(name, layers, batch, hq, hkv, d, dtype, m, W, S, 0, 0, 0, rank, 0.05, rank == 0)


def test_tiny_config_every_step():
    """1 layer, batch 1, 4 heads x 64, fp32, budget 128, window 16: 256 prefill tokens, 256 decode steps."""
    wl = WORKLOADS["tiny"]
    p = Parity(wl)
    p.prefill(wl.prefill, chunk=64)
    p.compare_state()
    p.decode(wl.decode)
    p.compare_state()
    assert p.n_evictions == wl.lanes * (wl.prefill + wl.decode - wl.budget)
    p.close()


@pytest.mark.parametrize("dtype,d,hq,hkv,m,W,S,splits,steps", [
    ("f32", 64, 4, 4, 40, 4, 0, 0, 120),       # several tiles, ragged tail (41 = 32 + 9)
    ("f32", 128, 2, 2, 70, 1, 0, 3, 150),      # Algorithm 1's own range (window 1), 3 tiles over 3 CTAs
    ("bf16", 128, 4, 4, 100, 8, 4, 2, 220),    # sinks
    ("bf16", 64, 4, 4, 33, 5, 2, 5, 100),      # more splits than tiles
    ("bf16", 128, 8, 4, 64, 16, 0, 2, 160),    # group of 2
    ("bf16", 128, 8, 2, 95, 16, 1, 0, 200),    # group of 4
    ("bf16", 64, 8, 2, 70, 4, 0, 3, 170),      # group of 4 on 128-byte rows (one swizzled half per value tile), ragged tail
    ("bf16", 128, 16, 4, 45, 6, 2, 5, 130),    # group of 4: the last tile's box reaches past the lane and, for the last lane, past the cache
    ("f32", 128, 8, 2, 60, 4, 1, 2, 140),      # group of 4 on fp32 rows (plain value tiles, 384-thread lane epilogue)
    ("f32", 64, 8, 1, 31, 3, 0, 1, 90),        # group of 8, exactly one tile
    ("f32", 64, 2, 2, 1, 1, 0, 0, 20),         # smallest possible cache
    ("bf16", 128, 2, 2, 8, 8, 0, 0, 40),       # window == budget: a single candidate
    ("bf16", 128, 2, 2, 200, 32, 0, 64, 260),  # maximum split count
])
@pytest.mark.parametrize("schedule", [binding.WKV_SCHEDULE_SPLIT, binding.WKV_SCHEDULE_CLUSTER, binding.WKV_SCHEDULE_FLAT])
def test_shapes_every_step(dtype, d, hq, hkv, m, W, S, splits, steps, schedule):
    if schedule == binding.WKV_SCHEDULE_CLUSTER and splits not in (0, 1, 2, 4, 8, 16):
        pytest.skip("a cluster needs a power-of-two split count")
    wl = small(batch=3, hq=hq, hkv=hkv, d=d, dtype=dtype, m=m, W=W, S=S, rank=16 if dtype == "bf16" else 0)
    p = Parity(wl, seed=17 + m, n_splits=splits, schedule=schedule)
    p.decode(steps)
    p.compare_state()
    assert p.n_evictions == wl.lanes * max(0, steps - m)
    p.close()


@pytest.mark.parametrize("dtype,hq,hkv,m,splits", [("bf16", 32, 32, 70, 0), ("bf16", 32, 8, 100, 0), ("f32", 16, 16, 40, 0),
                                                    ("bf16", 8, 8, 300, 3)])
def test_flat_deal_runs_of_tiles_across_lanes(dtype, hq, hkv, m, splits):
    """The flat deal with runs that do not line up with the lanes: with splits = 0 the scan takes one wave of CTAs, so
    with far more lanes than CTAs a CTA holds a piece of several lanes (the end of one, whole lanes, the start of the
    next), and with few lanes a lane is cut into pieces of unequal size; ragged prompts leave some lanes shorter than
    their tile count.  Compared with the oracle every step, and with the even deal at the end."""
    batch = 40 if splits == 0 else 3
    wl = small(batch=batch, hq=hq, hkv=hkv, d=128 if dtype == "bf16" else 64, dtype=dtype, m=m, W=6, S=1,
               rank=16 if dtype == "bf16" else 0)
    lens = [m + 30 - (7 * b) % 50 for b in range(batch)]
    p = Parity(wl, seed=23, sample=24, n_splits=splits, schedule=binding.WKV_SCHEDULE_FLAT, ragged=lens)
    q = Parity(wl, seed=23, sample=24, schedule=binding.WKV_SCHEDULE_SPLIT, ragged=lens)
    p.prefill(m + 30, chunk=40)
    q.prefill(m + 30, chunk=40, compare=False)
    p.decode(12)
    p.decode(4, layers_entry=True)
    q.decode(16)
    p.compare_state()
    for ln in p.lanes:
        s0, s1 = p.ctx.wkv_export_state(*ln), q.ctx.wkv_export_state(*ln)
        assert torch.equal(s0["pos"], s1["pos"]) and torch.equal(s0["a"], s1["a"]) and torch.equal(s0["V"], s1["V"])
    p.close()
    q.close()


def test_split_count_does_not_change_results():
    """The same stream under 1, 2, 5 and 16 CTAs per lane: identical eviction sequences and bit-identical a."""
    wl = small(batch=2, d=128, dtype="bf16", m=150, W=8, rank=16)
    states = []
    for splits, schedule in ((1, 1), (2, 2), (5, 1), (16, 2), (8, 1), (4, 0), (3, 3), (0, 3)):
        p = Parity(wl, seed=5, n_splits=splits, schedule=schedule)
        assert schedule == 3 or p.ctx.wkv_splits() == splits
        p.decode(230)
        states.append([p.ctx.wkv_export_state(*ln) for ln in p.lanes])
        p.close()
    for other in states[1:]:
        for s0, s1 in zip(states[0], other):
            assert torch.equal(s0["pos"], s1["pos"]) and torch.equal(s0["a"], s1["a"]) and torch.equal(s0["V"], s1["V"])


@pytest.mark.parametrize("schedule", [binding.WKV_SCHEDULE_SPLIT, binding.WKV_SCHEDULE_CLUSTER])
def test_ragged_prefill_then_decode(schedule):
    """Per-sequence prompt lengths, one shorter than the budget so that lane is still growing during decode."""
    wl = small(layers=2, batch=4, d=128, dtype="bf16", m=96, W=8, rank=16)
    p = Parity(wl, seed=9, ragged=[150, 40, 97, 96], schedule=schedule)
    p.prefill(150, chunk=50)
    p.compare_state()
    p.decode(80)
    p.compare_state()
    p.close()


@pytest.mark.parametrize("schedule,splits", [(binding.WKV_SCHEDULE_SPLIT, 3), (binding.WKV_SCHEDULE_CLUSTER, 2)])
def test_probabilities_output(schedule, splits):
    wl = small(batch=1, hq=4, hkv=2, d=64, dtype="f32", m=70, W=2)
    p = Parity(wl, seed=3, check_probs=True, schedule=schedule, n_splits=splits)
    p.decode(95)
    p.close()


def test_eviction_ablation():
    wl = small(batch=2, d=64, dtype="f32", m=30, W=4)
    p = Parity(wl, seed=4, merge=0)
    p.decode(100)
    p.compare_state()
    p.close()


def test_host_buffer_entry_point():
    wl = small(layers=2, batch=2, d=128, dtype="bf16", m=50, W=4, rank=16)
    p = Parity(wl, seed=6)
    p.decode(30)
    p.decode(60, host_entry=True)
    p.decode(20, host_entry=True, layers_entry=True)
    p.compare_state()
    p.close()


@pytest.mark.parametrize("schedule", [binding.WKV_SCHEDULE_SPLIT, binding.WKV_SCHEDULE_CLUSTER])
def test_all_layers_entry_point(schedule):
    """wkv_decode_step_layers lets consecutive layers overlap on the GPU; results must not change."""
    wl = small(layers=6, batch=3, d=128, dtype="bf16", m=120, W=8, rank=16)
    p = Parity(wl, seed=12, schedule=schedule, n_splits=2)
    p.decode(100, layers_entry=True)
    p.decode(20)
    p.decode(60, layers_entry=True)
    p.compare_state()
    p.close()


def test_export_import_roundtrip_and_continue():
    wl = small(batch=1, hq=2, hkv=2, d=64, dtype="f32", m=24, W=3)
    p = Parity(wl, seed=8)
    p.decode(60)
    snap = [p.ctx.wkv_export_state(*ln) for ln in p.lanes]
    p.ctx.wkv_reset()
    for ln in p.lanes:
        assert p.ctx.wkv_export_state(*ln)["len"] == 0
    for ln, s in zip(p.lanes, snap):
        p.ctx.wkv_import_state(*ln, tokens=s["tokens"], pos=s["pos"], a=s["a"], K=s["K"], V=s["V"])
    p.compare_state()
    p.decode(40)           # the imported (compacted) layout must keep matching the oracle
    p.compare_state()
    p.close()


def test_large_budget_is_full_attention():
    """budget >= tokens: nothing is ever removed and the output is plain softmax attention (torch, fp64)."""
    wl = small(batch=2, hq=4, hkv=4, d=64, dtype="f32", m=300, W=4)
    p = Parity(wl, seed=10)
    ks, vs = [], []
    from paper_2503_01330_b200.synth import TokenStream
    st = TokenStream(wl, 10, "cuda:0")
    for t in range(70):
        q, k, v = st.token(t)
        ks.append(k[0].double())
        vs.append(v[0].double())
        p.decode(1)
        K, V = torch.stack(ks, 2), torch.stack(vs, 2)           # [B, H, t, d]
        att = torch.softmax(torch.einsum("bhd,bhtd->bht", q[0].double(), K) / 8.0, -1)
        want = torch.einsum("bht,bhtd->bhd", att, V)
        assert_close(p.out[0].cpu().numpy(), want.cpu().numpy(), "f32", f"full attention step {t}")
        assert (p.ev == -1).all()
    p.close()


@pytest.mark.parametrize("schedule", [binding.WKV_SCHEDULE_AUTO, binding.WKV_SCHEDULE_SPLIT])
def test_bounded_wait_reports_timeout_and_context_survives(schedule):
    """A wait that nothing completes runs out of polls: the status word says so, once, and decoding goes on (with the
    two-kernel schedule the status call also clears the lanes' arrival counters, which must leave the next step intact)."""
    wl = small(batch=1, hq=2, hkv=2, d=64, dtype="f32", m=12, W=2)
    p = Parity(wl, seed=2, schedule=schedule, n_splits=2 if schedule else 0)
    p.decode(20)
    p.ctx.wkv_selftest_wait_timeout()
    assert p.ctx.wkv_status() == binding.WKV_ERR_TIMEOUT
    assert p.ctx.wkv_status() == binding.WKV_OK          # reading clears it
    p.decode(20)                                         # same context, still in step with the oracle
    p.compare_state()
    p.close()


def test_argument_errors_leave_context_usable():
    ctx = binding.Context(1, 1, 2, 2, 64, 16, 2, dtype=binding.WKV_F32)
    q = torch.zeros(1, 2, 64, device="cuda")
    with pytest.raises(binding.WkvError) as e:
        ctx.wkv_decode_step(3, q, q, q, q)
    assert e.value.code == binding.WKV_ERR_INVALID
    with pytest.raises(binding.WkvError):
        ctx.wkv_decode_step(0, None, q, q, q)
    with pytest.raises(binding.WkvError):
        ctx.wkv_export_state(0, 5, 0)
    ctx.wkv_decode_step(0, q, q, q, torch.empty_like(q))
    assert ctx.wkv_status() == 0 and ctx.wkv_export_state(0, 0, 1)["len"] == 1
    assert ctx.wkv_launch_count() == 2      # the reset at creation and one step
    ctx.close()


@pytest.mark.parametrize("schedule", [binding.WKV_SCHEDULE_AUTO, binding.WKV_SCHEDULE_CLUSTER])
def test_llama7b_layer_config_all_lanes(schedule):
    """One Llama-2-7B-shaped layer at its full size (32 heads x 128, bf16, budget 2048, window 64): prefill 4096,
    1024 decode steps, every lane, every step -- 3072 compressions per lane, about 10^5 bit-exact picks in all."""
    wl = WORKLOADS["llama7b_layer"]
    p = Parity(wl, schedule=schedule)
    p.prefill(wl.prefill, chunk=128)
    p.compare_state()
    p.decode(wl.decode)
    p.compare_state()
    assert p.n_evictions == wl.lanes * (wl.prefill + wl.decode - wl.budget)
    p.close()


def test_two_contexts_interleaved_on_one_stream():
    """Calls of two contexts alternate on the same stream; each must stay in step with its own oracle (the library
    may overlap consecutive launches of ONE context, never across contexts)."""
    wa = small(layers=3, batch=2, d=128, dtype="bf16", m=60, W=4, rank=16)
    wb = small(layers=2, batch=3, hq=4, hkv=2, d=64, dtype="f32", m=45, W=3)
    pa = Parity(wa, seed=31, schedule=binding.WKV_SCHEDULE_SPLIT, n_splits=2)
    pb = Parity(wb, seed=32, schedule=binding.WKV_SCHEDULE_SPLIT, n_splits=3)
    for _ in range(12):
        pa.decode(5, layers_entry=True)
        pb.decode(4)
        pa.decode(3)
        pb.decode(4, layers_entry=True)
    pa.compare_state()
    pb.compare_state()
    pa.close()
    pb.close()


@pytest.mark.parametrize("schedule", [binding.WKV_SCHEDULE_SPLIT, binding.WKV_SCHEDULE_CLUSTER])
def test_decode_steps_replayed_from_a_cuda_graph(schedule):
    """wkv_decode_step neither allocates nor synchronises, so a step (all layers) can be captured once and replayed:
    the replayed steps must leave the same outputs and state as the same steps issued call by call."""
    wl = small(layers=4, batch=2, hq=4, hkv=2, d=128, dtype="bf16", m=80, W=8, rank=16)
    dev = torch.device("cuda:0")
    from paper_2503_01330_b200.synth import TokenStream
    res = {}
    for mode in ("calls", "graph"):
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            ctx = binding.Context(4, 2, 4, 2, 128, 80, 8, dtype=binding.WKV_BF16, schedule=schedule, n_splits=2)
            st = TokenStream(wl, 3, dev)
            q = torch.empty(4, 2, 4, 128, dtype=torch.bfloat16, device=dev)
            k = torch.empty(4, 2, 2, 128, dtype=torch.bfloat16, device=dev)
            v = torch.empty_like(k)
            out = torch.empty_like(q)
            ev = torch.empty(4, 2, 2, dtype=torch.int32, device=dev)

            def step():
                for layer in range(4):
                    ctx.wkv_decode_step(layer, q[layer], k[layer], v[layer], out[layer], ev[layer])

            graph, outs, evs = None, [], []
            for t in range(130):
                a, b, c = st.token(t)
                q.copy_(a); k.copy_(b); v.copy_(c)
                if mode == "graph" and t == 2:
                    s.synchronize()
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=s):
                        step()
                if graph is not None:
                    graph.replay()
                else:
                    step()
                outs.append(out.float().clone())
                evs.append(ev.clone())
            s.synchronize()
            assert ctx.wkv_status() == 0
            res[mode] = (torch.stack(outs), torch.stack(evs),
                         [ctx.wkv_export_state(l, b, h) for l in range(4) for b in range(2) for h in range(2)])
            ctx.close()
    assert torch.equal(res["calls"][0], res["graph"][0]) and torch.equal(res["calls"][1], res["graph"][1])
    assert int((res["graph"][1] >= 0).sum()) == 16 * (130 - 80)
    for x, y in zip(res["calls"][2], res["graph"][2]):
        for key in ("pos", "a", "K", "V"):
            assert torch.equal(x[key], y[key]), key


def test_maximum_budget_at_the_capacity_limit():
    """budget = 2^20 - 1, the largest the configuration accepts: a step attends 2^20 entries, the capacity the integer
    normaliser is specified for (2^20 terms of at most 2^40).  Full caches are imported on both sides; a few steps and
    the whole exported state must agree."""
    m = (1 << 20) - 1
    wl = small(batch=1, hq=2, hkv=2, d=64, dtype="f32", m=m, W=16)
    p = Parity(wl, seed=77)
    assert p.ctx.wkv_splits() == 64
    rng = np.random.default_rng(1)
    tokens = m + 7
    pos = np.sort(rng.choice(tokens, size=m, replace=False)).astype(np.int32)
    for i, ln in enumerate(p.lanes):
        a = (rng.random(m) * (tokens - pos) * 1e-6 + 1e-9).astype(np.float32)
        K = (rng.standard_normal((m, 64)) * 0.5).astype(np.float32)
        V = rng.standard_normal((m, 64)).astype(np.float32)
        p.ctx.wkv_import_state(*ln, tokens=tokens, pos=torch.from_numpy(pos), a=torch.from_numpy(a),
                               K=torch.from_numpy(K), V=torch.from_numpy(V))
        p.ref.import_state(i, tokens, pos, a.astype(np.float64), K, V)
    p.t = tokens
    p.decode(3)
    p.compare_state()
    assert p.n_evictions == 3 * len(p.lanes)
    p.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("dtype,d,hq,hkv,m,schedule", [("bf16", 128, 8, 2, 50001, binding.WKV_SCHEDULE_SPLIT),
                                                      ("f32", 64, 8, 1, 30011, binding.WKV_SCHEDULE_SPLIT),
                                                      ("bf16", 128, 4, 2, 20003, binding.WKV_SCHEDULE_CLUSTER)])
def test_large_imported_caches_grouped_heads(dtype, d, hq, hkv, m, schedule):
    """Tens of thousands of entries per lane with 4, 8 and 2 query heads per key (odd budgets: ragged last tile and
    uneven units), caches imported on both sides, sinks kept: picks, scores and state after a few compressing steps."""
    wl = small(batch=2, hq=hq, hkv=hkv, d=d, dtype=dtype, m=m, W=24, S=3, rank=16 if dtype == "bf16" else 0)
    p = Parity(wl, seed=m, schedule=schedule)
    rng = np.random.default_rng(m)
    tokens = m + 1000
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    for i, ln in enumerate(p.lanes):
        pos = np.sort(np.concatenate([np.arange(3), 3 + rng.choice(tokens - 3, size=m - 3, replace=False)])).astype(np.int32)
        a = (rng.random(m) * (tokens - pos) * 1e-5 + 1e-8).astype(np.float32)
        K = torch.from_numpy((rng.standard_normal((m, d)) * 0.3).astype(np.float32)).to(tdt)
        V = torch.from_numpy(rng.standard_normal((m, d)).astype(np.float32)).to(tdt)
        p.ctx.wkv_import_state(*ln, tokens=tokens, pos=torch.from_numpy(pos), a=torch.from_numpy(a), K=K, V=V)
        p.ref.import_state(i, tokens, pos, a.astype(np.float64), K.float().numpy(), V.float().numpy())
    p.t = tokens
    p.decode(5)
    p.decode(2, layers_entry=True)
    p.compare_state()
    assert p.n_evictions == 7 * len(p.lanes)
    for ln in p.lanes:
        assert p.ctx.wkv_export_state(*ln)["pos"][:3].tolist() == [0, 1, 2]
    p.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("hq,hkv,batch,m", [
    (20, 20, 16, 4351),     # 320 lanes x 4352 entries: exactly what 256 threads x 17 slots hold (the register epilogue's limit)
    (20, 20, 16, 4352),     # one entry more: the loop version of the epilogue, and a streamed prompt tail
    (4, 4, 4, 4607),        # 16 lanes x 4608 entries: the limit of the 512-thread epilogue (9 slots per thread)
    (4, 4, 4, 4608),        # ... and one more
    (8, 2, 8, 3455),        # four heads per key, 16 lanes x 3456 entries: the limit of the 384-thread epilogue
    (8, 2, 8, 3456),
])
def test_lane_lengths_at_the_register_epilogue_limits(hq, hkv, batch, m):
    """Lanes exactly as long as the register version of the lane epilogue takes, and one entry longer (the loop version
    through global scratch): imported full caches, a prompt chunk through wkv_prefill_bulk (blocked tail on one side of
    the limit, streamed on the other), decode steps through both entry points; sampled lanes against the oracle."""
    wl = small(batch=batch, hq=hq, hkv=hkv, d=128, dtype="bf16", m=m, W=40, S=2, rank=16)
    p = Parity(wl, seed=m, sample=8, ragged=[m + 500] * batch)
    rng = np.random.default_rng(m)
    tokens = m + 300
    lane_set = {ln: i for i, ln in enumerate(p.lanes)}
    K1 = torch.from_numpy((rng.standard_normal((m, 128)) * 0.3).astype(np.float32)).to(torch.bfloat16)
    V1 = torch.from_numpy(rng.standard_normal((m, 128)).astype(np.float32)).to(torch.bfloat16)
    for b in range(batch):
        for h in range(hkv):
            pos = np.sort(np.concatenate([np.arange(2), 2 + rng.choice(tokens - 2, size=m - 2, replace=False)])).astype(np.int32)
            pos[-40:] = np.arange(tokens - 40, tokens)                       # the recent window is always whole
            pos = np.unique(pos)
            while len(pos) < m:                                              # (the window may have swallowed a drawn position)
                pos = np.unique(np.concatenate([pos, 2 + rng.choice(tokens - 42, size=m - len(pos))])).astype(np.int32)
            a = (rng.random(m) * (tokens - pos) * 1e-4 + 1e-8).astype(np.float32)
            p.ctx.wkv_import_state(0, b, h, tokens=tokens, pos=torch.from_numpy(pos), a=torch.from_numpy(a), K=K1, V=V1)
            if (0, b, h) in lane_set:
                p.ref.import_state(lane_set[(0, b, h)], tokens, pos, a.astype(np.float64), K1.float().numpy(), V1.float().numpy())
    p.t = tokens
    p.lens = torch.full((batch,), tokens + 100, dtype=torch.int32)
    p.prefill(19, chunk=19, bulk=True)       # two blocks of 8 and a block of 3 where the tail is blocked
    p.decode(4)
    p.decode(2, layers_entry=True)
    p.compare_state()
    assert p.n_evictions == 25 * len(p.lanes)
    p.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("dtype,schedule", [("f32", binding.WKV_SCHEDULE_SPLIT), ("bf16", binding.WKV_SCHEDULE_CLUSTER)])
def test_structural_ties_and_saturated_softmax(dtype, schedule):
    """Degenerate score distributions.  (1) zero queries: every probability is exactly 1/(m+1) (m+1 a power of two), so
    whole runs of entries tie bit for bit and the pick must be the lowest evictable position.  (2) queries scaled by
    25: logit gaps far beyond the exponential's cut-off, most probabilities exactly zero, scores stop growing and tie
    at equal values.  Both against the oracle, every step."""
    wl = small(batch=2, hq=4, hkv=2, d=64, dtype=dtype, m=63, W=4, rank=16 if dtype == "bf16" else 0)
    for kind in ("zero_q", "huge_q"):
        p = Parity(wl, seed=91, schedule=schedule, n_splits=2)
        draw = p.stream.token

        def token(t, draw=draw, kind=kind):
            q, k, v = draw(t)
            return (torch.zeros_like(q) if kind == "zero_q" else (q.float() * 25.0).to(q.dtype)), k, v

        p.stream.token = token
        p.decode(160)
        p.compare_state()
        assert p.n_evictions == wl.lanes * (160 - 63)
        if kind == "zero_q":
            # uniform attention: the oldest evictable entry always has the smallest average once all have tied or aged
            g = p.ctx.wkv_export_state(*p.lanes[0])
            assert g["len"] == 63
        p.close()


@pytest.mark.parametrize("scale", [0.03125, 0.3])
def test_softmax_scale_override(scale):
    """A caller-chosen softmax scale (a power of two and one that is not) in place of 1/sqrt(head_dim): the one
    multiplication after the dot, same on both sides; dense prompt phase, streamed tail and decode."""
    wl = small(batch=2, hq=4, hkv=2, d=64, dtype="f32", m=50, W=4)
    p = Parity(wl, seed=8, scale=scale, ragged=[90, 90])
    p.prefill(90, chunk=90, bulk=True)
    p.decode(40)
    p.compare_state()
    p.close()
