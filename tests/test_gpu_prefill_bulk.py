"""wkv_prefill_bulk against the CPU oracle (which streams, as Algorithm 1 does) and against wkv_prefill: the dense
start of the prompt must leave exactly the state that token-by-token processing leaves."""
import numpy as np
import pytest
import torch

from paper_2503_01330_b200 import binding
from paper_2503_01330_b200.synth import WORKLOADS, TokenStream, Workload

from parity_util import Parity

pytestmark = pytest.mark.gpu


def small(layers=1, batch=2, hq=4, hkv=4, d=64, dtype="f32", m=40, W=4, S=0, rank=0):
    return Workload("s", layers, batch, hq, hkv, d, dtype, m, W, S, 0, 0, 0, rank, 0.05, rank == 0)


@pytest.mark.parametrize("dtype,d,hq,hkv,m,W,S,T", [
    ("f32", 64, 4, 4, 40, 4, 0, 100),        # budget not a multiple of the row block; streamed tail of 60 tokens
    ("f32", 128, 2, 2, 300, 8, 0, 300),      # prompt == budget: three key tiles, nothing streamed
    ("f32", 64, 2, 2, 200, 4, 0, 131),       # prompt shorter than the budget, ragged last tile and last row block
    ("bf16", 128, 4, 4, 150, 8, 4, 260),     # sinks, bf16
    ("bf16", 128, 8, 4, 129, 16, 0, 200),    # group of 2, one key past a tile boundary
    ("bf16", 128, 8, 2, 95, 16, 1, 170),     # group of 4
    ("f32", 64, 8, 1, 70, 3, 0, 120),        # group of 8: a token's heads span two warps
    ("bf16", 64, 4, 2, 1, 1, 0, 20),         # smallest cache: one token in bulk, the rest streamed
    ("f32", 64, 2, 2, 16, 2, 0, 1),          # a single token
])
def test_bulk_prefill_matches_oracle_every_token(dtype, d, hq, hkv, m, W, S, T):
    wl = small(batch=3, hq=hq, hkv=hkv, d=d, dtype=dtype, m=m, W=W, S=S, rank=16 if dtype == "bf16" else 0)
    p = Parity(wl, seed=40 + m, ragged=[T, T, T])
    p.prefill(T, chunk=T, bulk=True)
    p.compare_state()
    p.decode(m // 2 + 5)
    p.compare_state()
    assert p.n_evictions == wl.lanes * max(0, T + m // 2 + 5 - m)
    p.close()


def test_bulk_prefill_ragged_lengths():
    """Per-sequence lengths: empty, shorter than the budget, exactly the budget, longer."""
    wl = small(layers=2, batch=4, d=128, dtype="bf16", m=96, W=8, rank=16)
    p = Parity(wl, seed=9, ragged=[150, 0, 96, 41])
    p.prefill(150, chunk=150, bulk=True)
    p.compare_state()
    p.decode(70)
    p.compare_state()
    p.close()


@pytest.mark.parametrize("schedule", [binding.WKV_SCHEDULE_SPLIT, binding.WKV_SCHEDULE_CLUSTER])
def test_bulk_and_streamed_prefill_leave_identical_state(schedule):
    wl = small(layers=2, batch=2, hq=8, hkv=2, d=128, dtype="bf16", m=200, W=8, rank=16)
    st = TokenStream(wl, 21, "cuda:0")
    Q, K, V = st.tokens(0, 330)
    lens = torch.tensor([330, 177], dtype=torch.int32, device="cuda:0")
    states, outs = [], []
    for bulk in (False, True):
        ctx = binding.Context(wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.budget, wl.window,
                              dtype=binding.WKV_BF16, schedule=schedule)
        out = torch.zeros(wl.n_layers, wl.batch, 330, wl.n_q_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda:0")
        ev = torch.full((wl.n_layers, wl.batch, 330, wl.n_kv_heads), -7, dtype=torch.int32, device="cuda:0")
        for layer in range(wl.n_layers):
            (ctx.wkv_prefill_bulk if bulk else ctx.wkv_prefill)(layer, Q[layer], K[layer], V[layer], lens, out[layer], ev[layer])
        assert ctx.wkv_status() == 0
        states.append([ctx.wkv_export_state(l, b, h) for l in range(2) for b in range(2) for h in range(2)])
        outs.append((out.float().cpu(), ev.cpu()))
        ctx.close()
    for s0, s1 in zip(*states):
        assert s0["len"] == s1["len"] and s0["tokens"] == s1["tokens"]
        for key in ("pos", "a", "K", "V"):
            assert torch.equal(s0[key], s1[key]), key
    assert torch.equal(outs[0][1], outs[1][1])                       # removed positions, -1 where nothing was removed
    torch.testing.assert_close(outs[1][0], outs[0][0], rtol=2e-2, atol=1e-3)


def test_bulk_prefill_continues_uncompressed_layers_and_streams_the_rest():
    """A prompt that arrives in pieces: while no lane of the layer can have reached the budget, each piece goes through
    the dense kernel on top of what the lanes hold; afterwards the pieces are streamed.  Decode steps in between count
    as tokens too.  The result is Algorithm 1's throughout."""
    wl = small(batch=2, d=64, dtype="f32", m=50, W=4)
    p = Parity(wl, seed=5, ragged=[140, 140])
    p.prefill(30, chunk=30, bulk=True)      # empty layer: dense
    n1 = p.ctx.wkv_launch_count()
    p.prefill(12, chunk=12, bulk=True)      # 30 tokens held, 42 after: still dense (one launch)
    assert p.ctx.wkv_launch_count() == n1 + 1
    p.decode(3)                             # 45
    p.prefill(45, chunk=45, bulk=True)      # 5 more fit densely, 40 streamed
    p.decode(10)
    p.prefill(40, chunk=40, bulk=True)      # full: streamed
    p.compare_state()
    launches = p.ctx.wkv_launch_count()
    p.ctx.wkv_reset()
    assert p.ctx.wkv_launch_count() == launches + 1
    p.close()


@pytest.mark.parametrize("dtype,d,hq,hkv,m,chunk,all_layers", [("bf16", 128, 8, 2, 300, 37, False), ("f32", 64, 4, 4, 190, 64, False),
                                                               ("bf16", 128, 4, 4, 260, 50, True), ("bf16", 64, 8, 1, 150, 16, True)])
def test_chunked_prompts_through_the_dense_kernel(dtype, d, hq, hkv, m, chunk, all_layers):
    """Prompts fed in chunks (chunked prefill): every chunk that still fits under the budget is a dense launch that
    reads the earlier tokens' keys and values from the cache; ragged sequence ends fall inside and between chunks."""
    wl = small(layers=2, batch=3, hq=hq, hkv=hkv, d=d, dtype=dtype, m=m, W=6, rank=16 if dtype == "bf16" else 0)
    T = m + 2 * chunk + 5
    p = Parity(wl, seed=60 + m, ragged=[T, m - chunk // 2, 2 * chunk + 3])
    p.prefill(T, chunk=chunk, bulk=True, all_layers=all_layers)
    p.compare_state()
    p.decode(12)
    p.compare_state()
    p.close()


def test_bulk_prefill_rejects_misaligned_rows():
    wl = small(batch=1, hq=2, hkv=2, d=64, dtype="bf16", m=16, W=2, rank=16)
    ctx = binding.Context(1, 1, 2, 2, 64, 16, 2, dtype=binding.WKV_BF16)
    buf = torch.zeros(1 * 8 * 2 * 64 + 8, dtype=torch.bfloat16, device="cuda:0")
    good = buf[:1024].view(1, 8, 2, 64)
    odd = buf[4:1028].view(1, 8, 2, 64)                 # 8 bytes past a 16-byte boundary
    with pytest.raises(binding.WkvError) as e:
        ctx.wkv_prefill_bulk(0, odd, good, good)
    assert e.value.code == binding.WKV_ERR_INVALID
    ctx.wkv_prefill_bulk(0, good, good, good)            # the context is still usable
    assert ctx.wkv_status() == 0 and ctx.wkv_export_state(0, 0, 0)["len"] == 8
    ctx.close()


def test_bulk_prefill_llama7b_layer_shape():
    """32 heads x 128, bf16, budget 2048: 2048 dense + 2048 streamed prompt tokens, sampled lanes against the oracle."""
    wl = WORKLOADS["llama7b_layer"]
    p = Parity(wl, sample=6)
    p.prefill(wl.prefill, chunk=wl.prefill, bulk=True)
    p.compare_state()
    p.decode(64)
    p.compare_state()
    p.close()


@pytest.mark.parametrize("name,n_sample", [("serving_b16", 6), ("gqa_b32", 4)])
def test_bulk_prefill_full_budget_shapes(name, n_sample):
    """Full batch, full budget and head layout of the large workloads (two of their layers): the whole dense phase
    (4096 / 3277 tokens, 32 / 26 key tiles) plus a ragged streamed tail, sampled lanes against the oracle."""
    wl = WORKLOADS[name].scaled(n_layers=2)
    n_prompt = wl.budget + 48
    rng = np.random.default_rng(5)
    lens = rng.integers(wl.budget - 40, n_prompt + 1, wl.batch)        # some prompts end inside the dense phase
    lens[0] = n_prompt
    lens[1] = wl.budget - 33
    p = Parity(wl, sample=n_sample, ragged=lens.tolist())
    p.prefill(n_prompt, chunk=n_prompt, bulk=True)
    p.compare_state()
    p.decode(6)
    p.compare_state()
    p.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("layers,batch,m,T,schedule", [(3, 2, 60, 150, binding.WKV_SCHEDULE_SPLIT), (2, 1, 40, 90, binding.WKV_SCHEDULE_SPLIT),
                                                       (1, 2, 33, 70, binding.WKV_SCHEDULE_SPLIT), (4, 1, 50, 50, binding.WKV_SCHEDULE_CLUSTER)])
def test_all_layers_prompt_call_matches_per_layer_calls(layers, batch, m, T, schedule):
    """wkv_prefill_bulk_layers (dense phase over the lanes of all layers, streamed tail with the layers interleaved)
    against wkv_prefill layer by layer: identical state, removed positions and (bf16-rounded) outputs."""
    wl = small(layers=layers, batch=batch, hq=4, hkv=2, d=128, dtype="bf16", m=m, W=4, rank=16)
    st = TokenStream(wl, 77, "cuda:0")
    Q, K, V = st.tokens(0, T)
    lens = torch.tensor([T, max(1, T - 37)][:batch], dtype=torch.int32, device="cuda:0")
    res = []
    for all_layers in (False, True):
        ctx = binding.Context(layers, batch, 4, 2, 128, m, 4, dtype=binding.WKV_BF16, schedule=schedule, n_splits=2)
        out = torch.zeros(layers, batch, T, 4, 128, dtype=torch.bfloat16, device="cuda:0")
        ev = torch.full((layers, batch, T, 2), -7, dtype=torch.int32, device="cuda:0")
        if all_layers:
            ctx.wkv_prefill_bulk_layers(Q, K, V, lens, out, ev)
        else:
            for layer in range(layers):
                ctx.wkv_prefill(layer, Q[layer], K[layer], V[layer], lens, out[layer], ev[layer])
        assert ctx.wkv_status() == 0
        res.append(([ctx.wkv_export_state(l, b, h) for l in range(layers) for b in range(batch) for h in range(2)],
                    out.float().cpu(), ev.cpu()))
        ctx.close()
    for s0, s1 in zip(res[0][0], res[1][0]):
        assert s0["len"] == s1["len"] and s0["tokens"] == s1["tokens"]
        for key in ("pos", "a", "K", "V"):
            assert torch.equal(s0[key], s1[key]), key
    assert torch.equal(res[0][2], res[1][2])
    torch.testing.assert_close(res[1][1], res[0][1], rtol=2e-2, atol=1e-3)


def test_all_layers_prompt_paper_cache_setting():
    """The paper's 256-entry cache (4 initial tokens, 124 recent) on the Llama-2-7B KV shape, one sequence: a
    1024-token prompt for all 32 layers in one call (dense phase over 1024 lanes, then one launch per token over all
    layers), sampled lanes against the oracle, then decode."""
    wl = WORKLOADS["paper_cache256"]
    p = Parity(wl, sample=10, ragged=[1024])
    p.prefill(1024, chunk=1024, all_layers=True)
    p.compare_state()
    p.decode(12, layers_entry=True)
    p.compare_state()
    p.close()


def test_all_layers_prompt_many_lanes_interleaves_layers():
    """16 layers of the serving shape at half its budget (8192 lanes, 72 MB of logit scratch): too much for one launch
    over all layers, so the dense phase runs layer by layer and the streamed tail interleaves the layers (a layer's scan
    alongside the previous layer's epilogues)."""
    wl = WORKLOADS["serving_b16"].scaled(n_layers=16, budget=2048, window=64)
    n_prompt = wl.budget + 40
    lens = [n_prompt - (3 * i) % 50 for i in range(wl.batch)]
    lens[0] = n_prompt
    p = Parity(wl, sample=8, ragged=lens)
    assert p.ctx.wkv_device_bytes() > 0
    p.prefill(n_prompt, chunk=n_prompt, all_layers=True)
    p.compare_state()
    p.decode(6)
    p.compare_state()
    p.close()
    torch.cuda.empty_cache()


def test_large_budget_dense_prompt_then_decode():
    """A budget of 8192 entries (256 cache tiles per lane, 128 key tiles in the dense phase), fp32: the whole budget
    filled by the dense kernel, then decode steps that compress, every token against the oracle.  With thousands of
    keys per output the 1e-5 output tolerance only holds if the products are not summed in one sequential chain."""
    wl = small(batch=1, hq=2, hkv=2, d=64, dtype="f32", m=8192, W=32)
    p = Parity(wl, seed=123, ragged=[8192])
    assert p.ctx.wkv_splits() > 1
    p.prefill(8192, chunk=8192, bulk=True)
    p.compare_state()
    p.decode(24)
    p.compare_state()
    assert p.n_evictions == wl.lanes * 24
    p.close()


@pytest.mark.parametrize("kind", ["zero_q", "huge_q"])
def test_bulk_prefill_degenerate_scores(kind):
    """Uniform attention (zero queries) and a saturated softmax (queries x25: most exponentials cut off to exactly 0)
    through the dense kernel and the streamed tail."""
    wl = small(batch=2, hq=4, hkv=2, d=128, dtype="bf16", m=140, W=6, rank=16)
    p = Parity(wl, seed=19, ragged=[230, 131])
    draw = p.stream.token

    def token(t):
        q, k, v = draw(t)
        return (torch.zeros_like(q) if kind == "zero_q" else (q.float() * 25.0).to(q.dtype)), k, v

    p.stream.token = token
    p.prefill(230, chunk=230, bulk=True)
    p.compare_state()
    p.decode(20)
    p.compare_state()
    p.close()


def test_bulk_prefill_eviction_ablation_and_stream_switch():
    """merge = 0 (plain eviction with the same picks) through the dense phase and the streamed tail; halfway the
    context is moved to another CUDA stream (wkv_set_stream) and must carry on from the same state."""
    wl = small(layers=2, batch=2, hq=4, hkv=4, d=64, dtype="f32", m=48, W=4)
    p = Parity(wl, seed=15, merge=0, ragged=[120, 77])
    p.prefill(120, chunk=120, bulk=True)
    p.compare_state()
    p.decode(10)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    p.ctx.wkv_set_stream(side.cuda_stream)
    with torch.cuda.stream(side):
        p.decode(25)
        p.compare_state()
    side.synchronize()
    p.ctx.wkv_set_stream(torch.cuda.current_stream().cuda_stream)
    p.decode(5)
    p.compare_state()
    p.close()


@pytest.mark.parametrize("dtype,d,hq,hkv,m,W,S,T,chunk", [
    ("bf16", 128, 4, 4, 70, 9, 0, 150, 150),     # one head per key: blocks of 8 tokens, the smallest window that allows them; last block of 8 full
    ("bf16", 128, 4, 4, 70, 12, 2, 149, 149),    # ... last block of 7 tokens, sinks
    ("f32", 64, 2, 2, 33, 10, 0, 100, 29),       # fp32 rows; the prompt in chunks that end inside blocks (blocks restart per call)
    ("bf16", 64, 8, 4, 100, 16, 1, 171, 171),    # two heads per key: blocks of 4
    ("bf16", 128, 8, 2, 95, 16, 0, 170, 60),     # four heads per key: blocks of 2, chunked
    ("f32", 128, 4, 1, 40, 6, 0, 90, 90),        # four heads per key on fp32 rows
])
def test_blocked_prompt_tail_every_token(dtype, d, hq, hkv, m, W, S, T, chunk):
    """The tokens of a prompt beyond the budget, in blocks that share two sweeps of the cache (two-kernel schedule forced,
    so that small shapes take that path): removed positions bit for bit and outputs within tolerance for every token,
    state afterwards, then decode.  Ragged lengths end sequences inside a block and leave one sequence below the budget."""
    wl = small(batch=4, hq=hq, hkv=hkv, d=d, dtype=dtype, m=m, W=W, S=S, rank=16 if dtype == "bf16" else 0)
    lens = [T, T - 3, m - 5, m + 11]
    p = Parity(wl, seed=70 + m, ragged=lens, schedule=binding.WKV_SCHEDULE_SPLIT)
    before = p.ctx.wkv_launch_count()
    p.prefill(T, chunk=chunk, bulk=True)
    launches = p.ctx.wkv_launch_count() - before
    # what the blocked path launches: per call the dense kernel (if the layer is still below the budget), then per block
    # one logit sweep, one lane-epilogue launch for the block's tokens, the value sweep and the output kernel
    B, expected, consumed = 8 // (hq // hkv), 0, 0
    for t0 in range(0, T, chunk):
        tc = min(chunk, T - t0)
        n0 = min(tc, max(0, m - consumed))
        tail = tc - n0
        expected += (1 if n0 > 0 else 0) + (2 * tail if tail < 2 else 4 * ((tail + B - 1) // B))
        consumed += tc
    assert launches == expected, "the tail did not go through the blocked path"
    p.compare_state()
    p.decode(m // 2 + 3)
    p.compare_state()
    p.close()


def test_blocked_prompt_tail_without_outputs_and_all_layers():
    """Outputs not requested (the value sweep is skipped) and the all-layers call: same state as the streamed prompt."""
    wl = small(layers=3, batch=2, hq=4, hkv=4, d=128, dtype="bf16", m=60, W=10, S=1, rank=16)
    st = TokenStream(wl, 33, "cuda:0")
    Q, K, V = st.tokens(0, 140)
    lens = torch.tensor([140, 97], dtype=torch.int32, device="cuda:0")
    states = []
    for mode in ("streamed", "blocked", "blocked_layers"):
        ctx = binding.Context(wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.budget, wl.window,
                              wl.sink, binding.WKV_BF16, schedule=binding.WKV_SCHEDULE_SPLIT)
        if mode == "blocked_layers":
            ctx.wkv_prefill_bulk_layers(Q, K, V, lens)
        else:
            for layer in range(wl.n_layers):
                (ctx.wkv_prefill if mode == "streamed" else ctx.wkv_prefill_bulk)(layer, Q[layer], K[layer], V[layer], lens)
        assert ctx.wkv_status() == 0
        states.append([ctx.wkv_export_state(l, b, h) for l in range(wl.n_layers) for b in range(wl.batch) for h in range(wl.n_kv_heads)])
        ctx.close()
    for other in states[1:]:
        for s0, s1 in zip(states[0], other):
            assert s0["len"] == s1["len"] and s0["tokens"] == s1["tokens"]
            assert torch.equal(s0["pos"], s1["pos"]) and torch.equal(s0["a"], s1["a"])
            assert torch.equal(s0["K"], s1["K"]) and torch.equal(s0["V"], s1["V"])
