"""Seeded synthetic q/k/v streams and the named workloads.

This module only draws random tensors; it holds none of the method's arithmetic, so both the CUDA
library's callers and the CPU oracle's callers may use it.  The public text corpora and the trained
Llama-2-7B weights the paper evaluates on are not available offline; these streams stand in for them.
They take Llama-2-7B's KV shape (32 layers x 32 heads x 128 channels) and the paper's singular-value
finding (Introduction, Fig. 1): keys are close to low rank, values are not.

A stream is deterministic per (seed, token index) on a given device; CPU and CUDA generators draw
different numbers, so a comparison always feeds both sides the bytes of ONE stream.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str            # "f32" | "bf16": storage type of q, k, v, out and the cache
    budget: int           # m
    window: int           # W
    sink: int
    prefill: int          # tokens consumed before the timed / compared decode phase (max over sequences)
    prefill_min: int      # ragged batches: per-sequence prefill length ~ U{prefill_min..prefill}
    decode: int           # decode steps
    key_rank: int         # 0: full-rank keys with a few boosted channels; r > 0: rank-r keys plus noise
    key_noise: float
    unit_scale: bool      # True: q, k, v ~ N(0,1)/sqrt(head_dim);  False: ~ N(0,1)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def lanes(self) -> int:
        return self.n_layers * self.batch * self.n_kv_heads

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    # 1 layer, batch 1, 4 heads x 64, fp32; skewed scores through a few high-variance key channels
    "tiny": Workload("tiny", 1, 1, 4, 4, 64, "f32", 128, 16, 0, 256, 256, 256, 0, 0.0, True),
    # one Llama-2-7B-shaped layer, batch 1
    "llama7b_layer": Workload("llama7b_layer", 1, 1, 32, 32, 128, "bf16", 2048, 64, 0, 4096, 4096, 1024, 16, 0.05,
                              False),
    # full 32-layer KV shape, batch 8, budget ratio 20 %
    "llama7b_b8": Workload("llama7b_b8", 32, 8, 32, 32, 128, "bf16", 1638, 64, 0, 8192, 8192, 2048, 16, 0.05, False),
    # serving batch, ragged prefill lengths
    "serving_b16": Workload("serving_b16", 32, 16, 32, 32, 128, "bf16", 4096, 128, 0, 16384, 8192, 512, 16, 0.05,
                            False),
    # the paper's own cache settings (Experiments section): 4 initial tokens kept, cache 1024 with 508 recent tokens
    # and cache 256 with 124 recent tokens, Llama-2-7B KV shape, one sequence, 4k context
    "paper_cache1024": Workload("paper_cache1024", 32, 1, 32, 32, 128, "bf16", 1024, 508, 4, 4096, 4096, 512, 16, 0.05,
                                False),
    "paper_cache256": Workload("paper_cache256", 32, 1, 32, 32, 128, "bf16", 256, 124, 4, 4096, 4096, 512, 16, 0.05,
                               False),
    # grouped-query variant: 32 query heads share 8 kv heads
    "gqa_b32": Workload("gqa_b32", 32, 32, 32, 8, 128, "bf16", 3277, 128, 0, 32768, 32768, 512, 16, 0.05, False),
}

BASE_SEED = 20250301


def sequence_lengths(wl: Workload, seed: int) -> torch.Tensor:
    """Per-sequence prefill lengths [batch] (int32, CPU): uniform on {prefill_min..prefill}."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 7919 + 17)
    if wl.prefill_min >= wl.prefill:
        return torch.full((wl.batch,), wl.prefill, dtype=torch.int32)
    lens = torch.randint(wl.prefill_min, wl.prefill + 1, (wl.batch,), generator=g, dtype=torch.int32)
    lens[0] = wl.prefill          # the longest sequence defines the token count of the prefill call
    return lens


class TokenStream:
    """q, k, v for token index t of every (layer, sequence, head) of a workload."""

    def __init__(self, wl: Workload, seed: int = BASE_SEED, device="cpu"):
        self.wl, self.seed, self.device = wl, int(seed), torch.device(device)
        g = self._gen(-1)
        L, H, d = wl.n_layers, wl.n_kv_heads, wl.head_dim
        if wl.key_rank > 0:
            # fixed rank-r basis per (layer, kv head); each key channel keeps unit variance
            self.basis = torch.randn(L, H, wl.key_rank, d, generator=g, device=self.device) / (wl.key_rank ** 0.5)
        else:
            # 4 boosted key channels per (layer, kv head)
            boost = torch.ones(L, H, d, device=self.device)
            idx = torch.rand(L, H, d, generator=g, device=self.device).argsort(dim=-1)[..., :4]
            boost.scatter_(-1, idx, 8.0)
            self.boost = boost

    def _gen(self, t: int) -> torch.Generator:
        g = torch.Generator(device=self.device)
        g.manual_seed((self.seed * 1_000_003 + (t + 1)) & 0x7FFFFFFFFFFF)
        return g

    def token(self, t: int):
        """Returns q [n_layers, B, Hq, d], k, v [n_layers, B, Hkv, d] in the workload's storage type."""
        wl, g, dev = self.wl, self._gen(t), self.device
        L, B, Hq, Hk, d = wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        q = torch.randn(L, B, Hq, d, generator=g, device=dev)
        v = torch.randn(L, B, Hk, d, generator=g, device=dev)
        if wl.key_rank > 0:
            z = torch.randn(L, B, Hk, wl.key_rank, generator=g, device=dev)
            k = torch.einsum("lbhr,lhrd->lbhd", z, self.basis)
            k = k + wl.key_noise * torch.randn(L, B, Hk, d, generator=g, device=dev)
        else:
            k = torch.randn(L, B, Hk, d, generator=g, device=dev) * self.boost[:, None]
        if wl.unit_scale:
            s = d ** -0.5
            q, k, v = q * s, k * s, v * s
        dt = wl.torch_dtype
        return q.to(dt).contiguous(), k.to(dt).contiguous(), v.to(dt).contiguous()

    def tokens(self, t0: int, n: int):
        """n consecutive tokens, token-major per sequence: q [n_layers, B, n, Hq, d], k, v [n_layers, B, n, Hkv, d]."""
        qs, ks, vs = zip(*(self.token(t) for t in range(t0, t0 + n)))
        return torch.stack(qs, 2).contiguous(), torch.stack(ks, 2).contiguous(), torch.stack(vs, 2).contiguous()

    def prompt(self, layer: int, n: int):
        """A whole prompt of n tokens for ONE layer, token-major per sequence: q [B, n, Hq, d], k, v [B, n, Hkv, d].
        Same distributions as token(), drawn with a few large calls (its own random stream, keyed by the layer)."""
        wl, dev = self.wl, self.device
        g = torch.Generator(device=dev)
        g.manual_seed((self.seed * 1_000_003 + 7_000_000_007 + layer) & 0x7FFFFFFFFFFF)
        B, Hq, Hk, d = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        q = torch.randn(B, n, Hq, d, generator=g, device=dev)
        v = torch.randn(B, n, Hk, d, generator=g, device=dev)
        if wl.key_rank > 0:
            z = torch.randn(B, n, Hk, wl.key_rank, generator=g, device=dev)
            k = torch.einsum("bnhr,hrd->bnhd", z, self.basis[layer])
            k = k + wl.key_noise * torch.randn(B, n, Hk, d, generator=g, device=dev)
        else:
            k = torch.randn(B, n, Hk, d, generator=g, device=dev) * self.boost[layer][None, None]
        if wl.unit_scale:
            s = d ** -0.5
            q, k, v = q * s, k * s, v * s
        dt = wl.torch_dtype
        return q.to(dt).contiguous(), k.to(dt).contiguous(), v.to(dt).contiguous()
