"""The N > 1 path on CPU: two gloo ranks run as replicas (independent lanes, no data-path collective) and agree on
the slowest rank's time, as bench.py does on GPUs."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2503_01330_b200.multi import aggregate_steps_per_s, max_over_ranks, rank_seed


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2503_01330_b200.synth import BASE_SEED, TokenStream, WORKLOADS
    wl = WORKLOADS["tiny"].scaled(budget=12, window=2)
    seed = rank_seed(BASE_SEED, rank)
    ref = oracle.Oracle(wl.lanes, wl.head_dim, wl.budget, window=wl.window, mode=oracle.MODE_PINNED)
    stream = TokenStream(wl, seed, "cpu")
    evs = []
    for t in range(30):                                  # each replica decodes its own batch
        q, k, v = stream.token(t)
        _, ev, _ = ref.step(q[0].reshape(wl.lanes, 1, -1).numpy(), k[0].reshape(wl.lanes, -1).numpy(),
                            v[0].reshape(wl.lanes, -1).numpy())
        evs.append(ev.copy())
    local_ms = 10.0 + 5.0 * rank                          # stand-in for the device-measured time of this rank
    dist.barrier()
    slowest = max_over_ranks(local_ms, dist, "cpu")
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.concatenate([[slowest, seed], np.stack(evs).ravel()]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_are_independent_replicas(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(world))
    assert r0[0] == r1[0] == 15.0                        # both ranks report the maximum over ranks
    assert r0[1] != r1[1]                                # different streams per rank
    assert (r0[2:] != r1[2:]).any()                      # ... hence different eviction sequences
    assert aggregate_steps_per_s(world, 30, r0[0]) == 2 * 30 / 0.015


def test_single_process_is_identity():
    assert max_over_ranks(3.5) == 3.5
    assert rank_seed(100, 0) != rank_seed(100, 1)
