"""Parity at the full shapes of the large workloads (all layers, full batch, full budget) in the launch
configuration bench.py times, on sampled lanes the oracle computes one by one.  The streamed prompt is shortened
to budget + 160 tokens: every cache is then full and has compressed 160 times, which is the state the decode phase
runs in."""
import numpy as np
import pytest
import torch

from paper_2503_01330_b200.synth import WORKLOADS

from parity_util import Parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,n_sample,decode,schedule", [("llama7b_b8", 12, 256, 0), ("serving_b16", 12, 96, 0),
                                                           ("gqa_b32", 10, 64, 0), ("llama7b_b8", 6, 8, 2)])
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
