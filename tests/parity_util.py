"""Shared driver of the GPU-vs-oracle parity tests: feeds ONE seeded stream to the CUDA library (all lanes) and
to the CPU oracle (all or sampled lanes) and compares every step."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2503_01330_b200 import binding
from paper_2503_01330_b200.synth import BASE_SEED, TokenStream, sequence_lengths

# Tolerances of the comparison (attention outputs, merged values):
#   fp32 : |x - y| <= 1e-5 * max(|y|, rms of y's row)   -- 1e-5 relative; the row rms keeps components that
#          cancel to almost zero from demanding more than fp32 accumulation can give
#   bf16 : |x - y| <= 1e-3 + 2e-2 * |y|                  -- bf16 storage, fp32 accumulation
# Eviction positions, retained positions and accumulated scores a are compared bit for bit.


def assert_close(got, want, dtype, what):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    if dtype == "f32":
        rms = np.sqrt((want ** 2).mean(axis=-1, keepdims=True))
        bound = 1e-5 * np.maximum(np.abs(want), rms) + 1e-30
    else:
        bound = 1e-3 + 2e-2 * np.abs(want)
    bad = np.abs(got - want) > bound
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} beyond tolerance, worst ratio {(np.abs(got - want) / bound).max():.3g}"


def pick_lanes(wl, n, seed):
    """n distinct (layer, b, kv_head) triples, always including the first and the last lane."""
    total = wl.lanes
    if n is None or n >= total:
        ids = np.arange(total)
    else:
        rng = np.random.default_rng(seed)
        ids = np.unique(np.concatenate([[0, total - 1], rng.choice(total, size=n, replace=False)]))[:max(n, 2)]
    per_layer = wl.batch * wl.n_kv_heads
    return [(int(i // per_layer), int((i % per_layer) // wl.n_kv_heads), int(i % wl.n_kv_heads)) for i in ids]


class Parity:
    def __init__(self, wl, seed=BASE_SEED, sample=None, n_splits=0, sink=None, merge=1, device="cuda:0", ragged=None,
                 check_probs=False, schedule=0, scale=0.0):
        self.wl, self.dev = wl, torch.device(device)
        self.sink = wl.sink if sink is None else sink
        self.dtype_code = binding.WKV_F32 if wl.dtype == "f32" else binding.WKV_BF16
        self.ctx = binding.Context(wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.budget, wl.window,
                                   self.sink, self.dtype_code, merge=merge, n_splits=n_splits, device=self.dev,
                                   schedule=schedule, scale=scale)
        self.lanes = pick_lanes(wl, sample, seed)
        self.li = torch.tensor([l for l, _, _ in self.lanes], device=self.dev)
        self.bi = torch.tensor([b for _, b, _ in self.lanes], device=self.dev)
        self.hi = torch.tensor([h for _, _, h in self.lanes], device=self.dev)
        self.ref = oracle.Oracle(len(self.lanes), wl.head_dim, wl.budget, window=wl.window, sink=self.sink,
                                 group=wl.group, dtype=oracle.F32 if wl.dtype == "f32" else oracle.BF16,
                                 mode=oracle.MODE_PINNED, merge=merge, scale=scale)
        self.stream = TokenStream(wl, seed, self.dev)
        self.lens = sequence_lengths(wl, seed) if ragged is None else torch.as_tensor(ragged, dtype=torch.int32)
        self.t = 0
        self.n_evictions = 0
        self.check_probs = check_probs
        L, B, Hq, Hk, d = wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        self.out = torch.empty(L, B, Hq, d, dtype=wl.torch_dtype, device=self.dev)
        self.ev = torch.empty(L, B, Hk, dtype=torch.int32, device=self.dev)
        self.probs = torch.empty(L, B, Hq, wl.budget + 1, device=self.dev) if check_probs else None

    # ---- oracle side of one token --------------------------------------------------------------
    def _oracle_token(self, q, k, v, active, out_gpu, ev_gpu, what, probs_gpu=None, check_out=True):
        """q [n, G, d], k, v [n, d], out_gpu [n, G, d], ev_gpu [n] already gathered for the sampled lanes (CPU).
        check_out = False: the removed positions are compared, the attention output is not (and the oracle is not asked
        for it, which spares it the fp64 pass over the cache)."""
        o_ref, ev_ref, p_ref = self.ref.step(q.float().numpy(), k.float().numpy(), v.float().numpy(), active=active,
                                             want_out=check_out, want_probs=probs_gpu is not None)
        act = np.ones(len(self.lanes), bool) if active is None else np.asarray(active, bool)
        np.testing.assert_array_equal(ev_gpu.numpy()[act], ev_ref[act], err_msg=f"{what}: eviction positions")
        self.n_evictions += int((ev_ref[act] >= 0).sum())
        if act.any() and check_out:
            assert_close(out_gpu.float().numpy()[act], o_ref[act], self.wl.dtype, f"{what}: attention output")
        return p_ref

    def _gather(self, q, k, v):
        wl = self.wl
        qs = q.view(wl.n_layers, wl.batch, wl.n_kv_heads, wl.group, wl.head_dim)[self.li, self.bi, self.hi]
        return qs.cpu(), k[self.li, self.bi, self.hi].cpu(), v[self.li, self.bi, self.hi].cpu()

    # ---- prefill through wkv_prefill, chunked ------------------------------------------------------
    def prefill(self, n_tokens, chunk=32, compare=True, bulk=False, all_layers=False, out_every=1):
        """out_every = k > 1: the attention output is compared on every k-th prompt token only (and on the last token);
        removed positions are compared on every token either way, and the state afterwards by compare_state."""
        wl = self.wl
        lens_dev = self.lens.to(self.dev)
        t_end = self.t + n_tokens

        def launch(t0):
            """Issues one chunk on the GPU (asynchronous) and returns what the comparison needs, still on the device."""
            tc = min(chunk, t_end - t0)
            Q, K, V = self.stream.tokens(t0, tc)                          # [L, B, tc, H, d]
            rel = (lens_dev - t0).clamp(min=0, max=tc).to(torch.int32)
            out = torch.empty(wl.n_layers, wl.batch, tc, wl.n_q_heads, wl.head_dim, dtype=wl.torch_dtype, device=self.dev)
            ev = torch.empty(wl.n_layers, wl.batch, tc, wl.n_kv_heads, dtype=torch.int32, device=self.dev)
            if all_layers:
                self.ctx.wkv_prefill_bulk_layers(Q, K, V, rel, out, ev)
            for layer in range(0 if all_layers else wl.n_layers):
                (self.ctx.wkv_prefill_bulk if bulk else self.ctx.wkv_prefill)(layer, Q[layer], K[layer], V[layer], rel,
                                                                              out[layer], ev[layer])
            Qs = Q.view(wl.n_layers, wl.batch, tc, wl.n_kv_heads, wl.group, wl.head_dim)[self.li, self.bi, :, self.hi]
            Ks, Vs = K[self.li, self.bi, :, self.hi], V[self.li, self.bi, :, self.hi]
            Os = out.view(wl.n_layers, wl.batch, tc, wl.n_kv_heads, wl.group, wl.head_dim)[self.li, self.bi, :, self.hi]
            Es = ev[self.li, self.bi, :, self.hi]
            return t0, tc, (Qs, Ks, Vs, Os, Es), (Q, K, V, rel, out, ev)     # the last tuple keeps the kernels' buffers alive

        # the GPU works on chunk c + 1 while the oracle checks chunk c
        pending = launch(self.t) if self.t < t_end else None
        while pending is not None:
            t0, tc, dev_parts, _keep = pending
            Qs, Ks, Vs, Os, Es = (x.cpu() for x in dev_parts)             # waits for chunk c
            pending = launch(t0 + tc) if t0 + tc < t_end else None
            lens_s = self.lens[self.bi.cpu()].numpy()
            for i in range(tc):
                tok = t0 + i
                active = tok < lens_s
                self._oracle_token(Qs[:, i], Ks[:, i], Vs[:, i], active.astype(np.uint8), Os[:, i], Es[:, i],
                                   f"prefill token {tok}", check_out=out_every <= 1 or tok % out_every == 0 or tok == t_end - 1)
            self.t = t0 + tc

    # ---- decode through wkv_decode_step --------------------------------------------------------------
    def decode(self, n_steps, host_entry=False, layers_entry=False):
        wl = self.wl
        for s in range(n_steps):
            q, k, v = self.stream.token(self.t)
            if host_entry:
                qh, kh, vh = (x.cpu().pin_memory() for x in (q, k, v))
                oh = torch.empty_like(self.out, device="cpu").pin_memory()
                eh = torch.empty_like(self.ev, device="cpu").pin_memory()
                if layers_entry:
                    self.ctx.wkv_decode_step_layers_host(qh, kh, vh, oh, eh)
                else:
                    for layer in range(wl.n_layers):
                        self.ctx.wkv_decode_step_host(layer, qh[layer], kh[layer], vh[layer], oh[layer], eh[layer])
                self.out.copy_(oh)
                self.ev.copy_(eh)
            elif layers_entry:
                self.ctx.wkv_decode_step_layers(q, k, v, self.out, self.ev)
            else:
                for layer in range(wl.n_layers):
                    self.ctx.wkv_decode_step(layer, q[layer], k[layer], v[layer], self.out[layer], self.ev[layer],
                                             None if self.probs is None else self.probs[layer])
            qs, ks, vs = self._gather(q, k, v)
            os_ = self.out.view(wl.n_layers, wl.batch, wl.n_kv_heads, wl.group, wl.head_dim)[self.li, self.bi, self.hi].cpu()
            es = self.ev[self.li, self.bi, self.hi].cpu()
            pg = None
            if self.probs is not None:
                pg = self.probs.view(wl.n_layers, wl.batch, wl.n_kv_heads, wl.group, wl.budget + 1)[self.li, self.bi, self.hi].cpu()
                before = [(self.ref.export(i)["pos"], self.ref.tokens(i)) for i in range(len(self.lanes))]
            p_ref = self._oracle_token(qs, ks, vs, None, os_, es, f"decode step {self.t}", probs_gpu=pg)
            if pg is not None:
                # GPU: slot order; oracle: order of the list as attended (new token last, victim not yet removed)
                for i, ln in enumerate(self.lanes):
                    pos_list = [int(p) for p in before[i][0]] + [before[i][1]]
                    slot_pos = self.ctx.wkv_export_slots(*ln).numpy()          # after the step: the freed slot shows -1
                    ev_pos = int(es[i])
                    got = pg[i].numpy()
                    for g in range(wl.group):
                        by_pos = {p: np.float32(p_ref[i, g, j]) for j, p in enumerate(pos_list)}
                        for sl, p in enumerate(slot_pos):
                            if p >= 0:
                                assert got[g, sl] == by_pos[int(p)], (self.t, ln, g, sl)
                            elif sl < len(pos_list):
                                assert ev_pos >= 0 and got[g, sl] == by_pos[ev_pos], (self.t, ln, g, sl)
                            else:
                                assert got[g, sl] == 0.0
            self.t += 1
        assert self.ctx.wkv_status() == 0

    # ---- exported state ----------------------------------------------------------------------------
    def compare_state(self):
        worst_v_mismatch = 0
        for i, ln in enumerate(self.lanes):
            g = self.ctx.wkv_export_state(*ln)          # also validates the slot chain on the host
            r = self.ref.export(i)
            assert g["len"] == len(r["pos"]) and g["tokens"] == self.ref.tokens(i), f"lane {ln}: length / token count"
            np.testing.assert_array_equal(g["pos"].numpy(), r["pos"], err_msg=f"lane {ln}: retained positions")
            np.testing.assert_array_equal(g["a"].numpy().view(np.uint32), r["a"].astype(np.float32).view(np.uint32),
                                          err_msg=f"lane {ln}: accumulated scores (bitwise)")
            np.testing.assert_array_equal(g["K"].float().numpy(), r["K"], err_msg=f"lane {ln}: keys")
            assert_close(g["V"].float().numpy(), r["V"], self.wl.dtype, f"lane {ln}: merged values")
            worst_v_mismatch = max(worst_v_mismatch, int((g["V"].float().numpy() != r["V"]).sum()))
        return worst_v_mismatch

    def close(self):
        self.ctx.close()
        self.ref.close()


def check_all_lanes(ctx, wl, tokens_per_seq, evicted=None):
    """Properties of Algorithm 1's bookkeeping that hold at any size, checked on EVERY lane of the context at once, on the
    device arrays themselves (the context's memory comes from this process's provider, in the order the library asks for
    it: K, V, a, pos, next, prev, lane state).  tokens_per_seq [batch]: tokens each sequence has consumed.
    evicted [n_layers, batch, n_kv_heads] (optional): the removed positions of the last step."""
    bufs = list(ctx._bufs.values())
    lanes, m, W, S = wl.lanes, wl.budget, wl.window, wl.sink
    cap = (m + 1 + 3) // 4 * 4
    a = bufs[2].view(torch.float32)[:lanes * cap].view(lanes, cap)
    pos, nxt, prv = (bufs[i].view(torch.int32)[:lanes * cap].view(lanes, cap) for i in (3, 4, 5))
    st = bufs[6].view(torch.int32)[:lanes * 8].view(lanes, 8)
    dev = a.device
    t = torch.as_tensor(tokens_per_seq, dtype=torch.int32, device=dev).repeat_interleave(wl.n_kv_heads).repeat(wl.n_layers)  # [lanes]
    length, tok, head, tail, free = (st[:, i] for i in range(5))
    assert torch.equal(tok, t), "tokens consumed"
    assert torch.equal(length, torch.minimum(t, torch.full_like(t, m))), "entries held = min(tokens, budget)"
    used = pos[:, :m + 1] >= 0
    assert torch.equal(used.sum(1).to(torch.int32), length), "occupied slots = entries held"
    p64 = pos[:, :m + 1].to(torch.int64)
    # positions are distinct and below the token count
    srt = torch.where(used, p64, torch.full_like(p64, -1)).sort(dim=1).values
    dup = (srt[:, 1:] == srt[:, :-1]) & (srt[:, 1:] >= 0)
    assert not dup.any() and (p64.max(dim=1).values < t.to(torch.int64)).all(), "distinct positions below the token count"
    # the protected regions are whole: the newest `window` tokens and the first `sink` tokens are all still there
    newest = torch.minimum(t, torch.full_like(t, W)).to(torch.int64)
    kept_recent = (used & (p64 >= (t.to(torch.int64) - newest)[:, None])).sum(1)
    assert torch.equal(kept_recent, newest), "recent window retained"
    if S > 0:
        assert torch.equal((used & (p64 < S)).sum(1), torch.minimum(t, torch.full_like(t, S)).to(torch.int64)), "initial tokens retained"
    # the chain: next and prev are inverse on occupied slots, positions increase along it, one head and one tail
    idx = torch.arange(m + 1, device=dev)[None, :].expand(lanes, -1)
    n64, q64 = nxt[:, :m + 1].to(torch.int64), prv[:, :m + 1].to(torch.int64)
    has_next, has_prev = used & (n64 >= 0), used & (q64 >= 0)
    assert torch.equal(has_next.sum(1), (length - 1).clamp(min=0).to(torch.int64)), "every entry but the tail has a right neighbour"
    assert torch.equal(has_prev.sum(1), (length - 1).clamp(min=0).to(torch.int64)), "every entry but the head has a left neighbour"
    back = torch.gather(q64, 1, n64.clamp(min=0))
    pos_next = torch.gather(p64, 1, n64.clamp(min=0))
    assert (back[has_next] == idx[has_next]).all(), "prev[next[s]] = s"
    assert (pos_next[has_next] > p64[has_next]).all(), "positions increase along the chain"
    nonempty = length > 0
    hs, ts = head[nonempty].to(torch.int64), tail[nonempty].to(torch.int64)
    rows = torch.nonzero(nonempty)[:, 0]
    assert (q64[rows, hs] == -1).all() and (n64[rows, ts] == -1).all() and used[rows, hs].all() and used[rows, ts].all(), "head and tail"
    assert (p64[rows, ts] == t[nonempty].to(torch.int64) - 1).all(), "the tail is the newest token"
    full = t > m
    assert (~used[full, :][torch.arange(int(full.sum()), device=dev), free[full].to(torch.int64)]).all(), "the free slot is free"
    # accumulated scores: non-negative, each at most the steps its entry has been attended, all of a lane at most the steps
    n_att = (t.to(torch.int64)[:, None] - p64).clamp(min=0)
    av = torch.where(used, a[:, :m + 1], torch.zeros_like(a[:, :m + 1]))
    assert (av >= 0).all() and (av <= n_att.to(torch.float32) * (1 + 1e-5) + 1e-6).all(), "0 <= a <= n"
    assert (av.sum(1, dtype=torch.float64) <= t.to(torch.float64) * (1 + 1e-5)).all(), "sum of a <= steps"
    if evicted is not None:
        ev = evicted.reshape(-1).to(torch.int64)
        comp = full
        assert (ev[~comp] == -1).all() and (ev[comp] >= S).all() and (ev[comp] <= t[comp].to(torch.int64) - 1 - W).all(), "removed position in range"
        assert not (used & (p64 == ev[:, None]) & comp[:, None]).any(), "the removed position is gone"
