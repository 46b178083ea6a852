"""Parity at the full shapes of the large workloads (all layers, full batch, full budget) in the launch
configuration bench.py times, on sampled lanes the oracle computes one by one.  Two kinds of test: the configurations'
stated decode lengths (2048 / 512 / 512 steps) behind a prompt shortened to budget + 160 tokens -- every cache is then
full and has compressed 160 times, which is the state the decode phase runs in -- and the configurations' stated
prompt lengths (8192 / 16384 ragged / 32768 tokens) followed by a few decode steps."""
import numpy as np
import pytest
import torch

from paper_2503_01330_b200.synth import WORKLOADS

from parity_util import Parity, check_all_lanes

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,n_sample,decode,schedule", [("llama7b_b8", 12, 2048, 0), ("serving_b16", 12, 512, 0),
                                                           ("gqa_b32", 10, 512, 0), ("llama7b_b8", 6, 8, 2)])
def test_full_shape_sampled_lanes(name, n_sample, decode, schedule):
    wl = WORKLOADS[name]
    n_prefill = wl.budget + 160
    rng = np.random.default_rng(11)
    lens = rng.integers(n_prefill - 60, n_prefill + 1, wl.batch)       # ragged prompt ends, all beyond the budget
    lens[0] = n_prefill
    lens[-1] = n_prefill - 60
    p = Parity(wl, sample=n_sample, ragged=lens.tolist(), schedule=schedule)      # 0: the schedule bench.py gets
    assert p.ctx.wkv_device_bytes() > 0.9 * 2 * wl.lanes * (wl.budget + 1) * wl.head_dim * wl.elem_bytes
    p.prefill(n_prefill, chunk=32)
    p.compare_state()
    p.decode(decode)
    p.decode(4, layers_entry=True)
    p.compare_state()
    assert p.n_evictions >= len(p.lanes) * (100 + decode)
    # ... and what holds at any size, on every lane of the context (not only the sampled ones)
    check_all_lanes(p.ctx, wl, (p.lens + decode + 4).tolist(), p.ev)
    p.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["paper_cache1024", "paper_cache256"])
def test_paper_cache_settings(name):
    """The cache settings of the paper's Experiments section (4 initial tokens kept, 1024 / 508 recent and 256 / 124
    recent), Llama-2-7B KV shape: streamed prompt, per-layer decode calls and the all-layers call (one launch)."""
    wl = WORKLOADS[name]
    p = Parity(wl, sample=16, ragged=[wl.budget + 300])
    p.prefill(wl.budget + 300, chunk=64)
    p.compare_state()
    p.decode(16)
    p.decode(48, layers_entry=True)
    p.decode(8)
    p.compare_state()
    for ln in p.lanes:                                     # the four initial tokens are never removed
        assert p.ctx.wkv_export_state(*ln)["pos"][:4].tolist() == [0, 1, 2, 3]
    p.close()


def test_llama7b_b8_full_prompt_length():
    """The 32-layer, batch-8 configuration with its whole 8192-token prompt (budget 1638: 6554 compressions per lane
    before the first decode step), fed in chunks of 256 tokens for all layers at once -- dense while the lanes are below
    the budget, streamed with interleaved layers afterwards -- then decode; sampled lanes against the oracle."""
    wl = WORKLOADS["llama7b_b8"]
    p = Parity(wl, sample=6, ragged=[wl.prefill] * wl.batch)
    p.prefill(wl.prefill, chunk=256, all_layers=True)
    p.compare_state()
    p.decode(24)
    p.compare_state()
    assert p.n_evictions == len(p.lanes) * (wl.prefill + 24 - wl.budget)
    p.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name,n_sample,decode", [("serving_b16", 12, 16), ("gqa_b32", 8, 16)])
def test_serving_and_gqa_full_prompt_lengths(name, n_sample, decode):
    """The two largest configurations with their whole prompts (16384 tokens with per-sequence lengths drawn from
    8192..16384, and 32768 tokens), in chunks of 256 tokens for all layers at once, then decode; sampled lanes against
    the oracle.  Tens of thousands of compressions per lane, every removed position compared; the attention output on
    every 64th prompt token and on every decode step."""
    wl = WORKLOADS[name]
    p = Parity(wl, sample=n_sample)
    assert int(p.lens.max()) == wl.prefill and int(p.lens.min()) >= wl.prefill_min
    p.prefill(wl.prefill, chunk=256, all_layers=True, out_every=64)
    p.compare_state()
    p.decode(decode)
    p.compare_state()
    assert p.n_evictions >= sum(int(p.lens[b]) - wl.budget for _, b, _ in p.lanes)
    check_all_lanes(p.ctx, wl, (p.lens + decode).tolist(), p.ev)
    p.close()
    torch.cuda.empty_cache()
