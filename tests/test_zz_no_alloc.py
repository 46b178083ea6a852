"""wkv_decode_step_static: the decode step for callers that may not allocate device memory.

A host that has promised a fixed device footprint (a serving loop that must not stall in the allocator, a
plug-in that may only touch buffers it was handed) cannot let a library call cudaMalloc on its behalf.  This
entry point keeps the kernel's scratch in an array that is part of the library image, so nothing is allocated.
The test drives two contexts with the same inputs, one through wkv_decode_step and one through the static
variant, and requires the same results on consecutive calls -- and the same removed positions and outputs as the CPU
oracle -- while neither the memory provider nor torch's allocator sees a request.  It is collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_01330_b200 import binding
from paper_2503_01330_b200.synth import TokenStream, Workload
from parity_util import assert_close

pytestmark = pytest.mark.gpu


def _pair(wl, splits):
    mk = lambda: binding.Context(wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.budget, wl.window,
                                 wl.sink, binding.WKV_BF16 if wl.dtype == "bf16" else binding.WKV_F32, n_splits=splits)
    return mk(), mk()


@pytest.mark.parametrize("dtype,d,hq,hkv,m,splits", [("bf16", 128, 8, 4, 70, 3), ("f32", 64, 4, 4, 45, 2)])
def test_static_scratch_matches_regular_entry_point(dtype, d, hq, hkv, m, splits):
    wl = Workload("noalloc", 2, 3, hq, hkv, d, dtype, m, 4, 1, 0, 0, 0, 16 if dtype == "bf16" else 0, 0.05, dtype == "f32")
    ref, sta = _pair(wl, splits)
    stream = TokenStream(wl, 77, "cuda:0")
    shape_o = (wl.n_layers, wl.batch, wl.n_q_heads, wl.head_dim)
    o_ref = torch.empty(shape_o, dtype=wl.torch_dtype, device="cuda")
    o_sta = torch.empty_like(o_ref)
    e_ref = torch.empty(wl.n_layers, wl.batch, wl.n_kv_heads, dtype=torch.int32, device="cuda")
    e_sta = torch.empty_like(e_ref)
    lanes = wl.lanes
    cpu = oracle.Oracle(lanes, wl.head_dim, wl.budget, window=wl.window, sink=wl.sink, group=wl.group,
                        dtype=oracle.BF16 if dtype == "bf16" else oracle.F32, mode=oracle.MODE_PINNED)
    toks = [stream.token(t) for t in range(m + 40)]
    # one step of this shape outside the watched region: the first launch of a kernel may make the runtime load its code
    q, k, v = toks[0]
    for layer in range(wl.n_layers):
        ref.wkv_decode_step(layer, q[layer], k[layer], v[layer], o_ref[layer], e_ref[layer])
        sta.wkv_decode_step_static(layer, q[layer], k[layer], v[layer], o_sta[layer], e_sta[layer])
    ref.wkv_reset()
    sta.wkv_reset()
    torch.cuda.synchronize()
    provider_bytes, n_blocks = sta.wkv_device_bytes(), len(sta._bufs)
    for t in range(m + 40):                      # growth, then 40 compressing steps; every step is a pair of calls
        q, k, v = toks[t]
        requests, torch_reserved = torch.cuda.memory_stats()["allocation.all.allocated"], torch.cuda.memory_reserved()
        for layer in range(wl.n_layers):         # two static calls in a row share the array: layer 0 then layer 1
            sta.wkv_decode_step_static(layer, q[layer], k[layer], v[layer], o_sta[layer], e_sta[layer])
        # the static calls asked nobody for memory: not the provider, not torch's allocator
        assert sta.wkv_device_bytes() == provider_bytes and len(sta._bufs) == n_blocks
        # (the count of requests, not the bytes in use: the collector may free other tests' tensors at any moment)
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == requests and torch.cuda.memory_reserved() <= torch_reserved
        for layer in range(wl.n_layers):
            ref.wkv_decode_step(layer, q[layer], k[layer], v[layer], o_ref[layer], e_ref[layer])
        assert torch.equal(e_ref, e_sta), f"step {t}: eviction positions"
        # ... and against the oracle
        qo = q.view(wl.n_layers, wl.batch, wl.n_kv_heads, wl.group, wl.head_dim).reshape(lanes, wl.group, -1).float().cpu().numpy()
        want_o, want_e, _ = cpu.step(qo, k.reshape(lanes, -1).float().cpu().numpy(), v.reshape(lanes, -1).float().cpu().numpy())
        np.testing.assert_array_equal(e_sta.cpu().numpy().reshape(-1), want_e, err_msg=f"step {t}: removed positions vs oracle")
        assert_close(o_sta.view(lanes, wl.group, -1).float().cpu().numpy(), want_o, dtype, f"step {t}: output vs oracle")
        if dtype == "f32":
            rms = o_ref.float().pow(2).mean(-1, keepdim=True).sqrt()
            bound = 1e-5 * torch.maximum(o_ref.float().abs(), rms)
        else:
            bound = 1e-3 + 2e-2 * o_ref.float().abs()
        assert ((o_sta.float() - o_ref.float()).abs() <= bound).all(), f"step {t}: attention output"
    assert (e_ref >= 0).all()
    for layer in range(wl.n_layers):
        for b in range(wl.batch):
            for h in range(wl.n_kv_heads):
                a, s = ref.wkv_export_state(layer, b, h), sta.wkv_export_state(layer, b, h)
                assert torch.equal(a["pos"], s["pos"]) and torch.equal(a["a"], s["a"]) and torch.equal(a["V"], s["V"])
    assert ref.wkv_status() == 0 and sta.wkv_status() == 0
    ref.close()
    sta.close()
    cpu.close()


def test_static_scratch_rejects_oversized_shapes():
    # 64 sequences x 32 heads x 4097 logits x 4 bytes is far beyond the 4 MiB array
    ctx = binding.Context(1, 64, 32, 32, 128, 4096, 64, dtype=binding.WKV_BF16)
    x = torch.zeros(64, 32, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.WkvError) as e:
        ctx.wkv_decode_step_static(0, x, x, x, torch.empty_like(x))
    assert e.value.code == binding.WKV_ERR_INVALID and "WKV_STATIC_SCRATCH_BYTES" in str(e.value)
    ctx.wkv_decode_step(0, x, x, x, torch.empty_like(x))     # the context stays usable
    assert ctx.wkv_status() == 0
    ctx.close()
