"""Seeded random configurations through the CUDA library and the CPU oracle: shapes, budgets, windows, sinks, prompt
lengths (ragged or not), schedules, split counts and entry points drawn together, so that combinations no hand-written
case names are covered too.  Each configuration runs a prompt (dense part and tail, or streamed), compares the state,
decodes some steps and compares the state again; removed positions, retained positions and scores bit for bit, outputs
and merged values within the stated tolerances (parity_util)."""
import numpy as np
import pytest
import torch

from paper_2503_01330_b200.synth import Workload
from parity_util import Parity

pytestmark = pytest.mark.gpu


def _draw(rng, budget_max):
    G = int(rng.choice([1, 1, 2, 4, 4, 8]))
    Hk = int(rng.choice([1, 2, 4]))
    budget = int(rng.integers(8, budget_max))
    sink = int(rng.choice([0, 0, 1, 4]))
    window = int(rng.integers(1, max(2, budget - sink - 1)))
    if rng.random() < 0.3:
        window = int(rng.integers(1, min(window, 12) + 1))
    prefill = int(rng.integers(1, min(2 * budget + 40, budget + 700)))
    pmin = int(rng.integers(1, prefill + 1)) if rng.random() < 0.5 else prefill
    wl = Workload("random", int(rng.choice([1, 2, 3])), int(rng.choice([1, 2, 3])), G * Hk, Hk, int(rng.choice([64, 128])),
                  str(rng.choice(["f32", "bf16", "bf16"])), budget, window, sink, prefill, pmin, int(rng.integers(1, 60)),
                  int(rng.choice([0, 16])), 0.05, bool(rng.random() < 0.5))
    bulk = bool(rng.random() < 0.7)
    how = dict(schedule=int(rng.choice([0, 0, 1, 2, 3])), n_splits=int(rng.choice([0, 0, 1, 2, 3, 4])),
               merge=int(rng.choice([1, 1, 1, 0])), bulk=bulk, all_layers=bool(bulk and rng.random() < 0.5),
               chunk=int(rng.choice([7, 32, 100, 4096])), layers_entry=bool(rng.random() < 0.4),
               host_entry=bool(rng.random() < 0.15))
    return wl, how


@pytest.mark.parametrize("seed,n_cfg,budget_max", [(11, 40, 420), (12, 12, 2600)])
def test_random_configurations_against_the_oracle(seed, n_cfg, budget_max):
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    rng = np.random.default_rng(seed)
    ran = 0
    for it in range(n_cfg):
        wl, how = _draw(rng, budget_max)
        what = f"configuration {it} of seed {seed}: {wl} {how}"
        try:
            p = Parity(wl, seed=seed * 1000 + it, n_splits=how["n_splits"], sink=wl.sink, merge=how["merge"],
                       schedule=how["schedule"])
        except RuntimeError as e:
            # the one refusal these draws can meet: the cluster schedule with a split count that is no cluster size
            assert how["schedule"] == 2 and "invalid" in str(e), what
            continue
        try:
            p.prefill(wl.prefill, chunk=how["chunk"], bulk=how["bulk"], all_layers=how["all_layers"])
            p.compare_state()
            p.decode(wl.decode, host_entry=how["host_entry"], layers_entry=how["layers_entry"])
            p.compare_state()
            assert p.ctx.wkv_status() == 0, what
        except AssertionError as e:
            raise AssertionError(f"{what}\n{e}") from e
        finally:
            p.close()
        ran += 1
    assert ran >= n_cfg * 3 // 4
