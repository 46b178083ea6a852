"""Error paths of the boundary that need a CUDA device but fault nothing: a memory provider that fails, and
bookkeeping that the host finds inconsistent.  Every failure is made on the host."""
import ctypes as C

import pytest
import torch

from paper_2503_01330_b200 import binding

pytestmark = pytest.mark.gpu


class Provider:
    """A memory provider over torch tensors that returns NULL on chosen requests and counts what it handed out."""

    def __init__(self, fail_at=(), fail_bytes_over=None):
        self.fail_at, self.fail_bytes_over = set(fail_at), fail_bytes_over
        self.calls, self.live, self.released = 0, {}, 0

        def alloc(nbytes, _user):
            k = self.calls
            self.calls += 1
            if k in self.fail_at or (self.fail_bytes_over is not None and nbytes > self.fail_bytes_over):
                return None
            buf = torch.empty(int(nbytes), dtype=torch.uint8, device="cuda:0")
            self.live[buf.data_ptr()] = buf
            return buf.data_ptr()

        def release(ptr, _user):
            assert ptr in self.live, "release of a block the provider never handed out (or handed back twice)"
            del self.live[ptr]
            self.released += 1

        self.alloc_cb, self.release_cb = binding.ALLOC_FN(alloc), binding.RELEASE_FN(release)

    def config(self, **kw):
        args = dict(n_layers=2, batch=2, n_q_heads=4, n_kv_heads=4, head_dim=64, budget=40, window=4, sink=0,
                    dtype=binding.WKV_BF16)
        args.update(kw)
        cfg = binding.make_config(**args)
        cfg.stream = torch.cuda.current_stream().cuda_stream
        cfg.alloc, cfg.release = self.alloc_cb, self.release_cb
        return cfg


def test_provider_failure_at_every_request_of_create():
    """wkv_create with a provider that returns NULL on its k-th request, for every k: WKV_ERR_ALLOC, no context, and
    every block obtained before the failure handed back."""
    torch.cuda.init()
    L = binding.lib()
    ok = Provider()
    h = C.c_void_p()
    assert L.wkv_create(C.byref(ok.config()), C.byref(h)) == binding.WKV_OK
    n_requests = ok.calls
    assert n_requests >= 15 and len(ok.live) == n_requests
    L.wkv_destroy(h)
    assert not ok.live and ok.released == n_requests
    for k in range(n_requests):
        p = Provider(fail_at=[k])
        h = C.c_void_p(1234)
        rc = L.wkv_create(C.byref(p.config()), C.byref(h))
        assert rc == binding.WKV_ERR_ALLOC, (k, rc)
        assert h.value is None, "no context on failure"
        assert not p.live and p.released == k, f"request {k} failed: {p.released} of {k} earlier blocks were handed back"
    assert L.wkv_strerror(binding.WKV_ERR_ALLOC).decode() == "device memory provider failed"


def test_provider_failure_for_the_dense_prompt_scratch_leaves_the_context_usable():
    """The dense prompt phase takes its scratch on first use.  If the provider refuses it the call returns WKV_ERR_ALLOC
    with a text, nothing has been launched, and the context decodes and -- once the provider gives in -- prefills."""
    L = binding.lib()
    p = Provider()
    cfg = p.config(n_layers=1, budget=64)
    h = C.c_void_p()
    assert L.wkv_create(C.byref(cfg), C.byref(h)) == binding.WKV_OK
    n_create = p.calls
    g = torch.Generator(device="cuda:0").manual_seed(3)
    Q = torch.randn(2, 48, 4, 64, generator=g, device="cuda:0").to(torch.bfloat16)
    K = torch.randn(2, 48, 4, 64, generator=g, device="cuda:0").to(torch.bfloat16)
    V = torch.randn(2, 48, 4, 64, generator=g, device="cuda:0").to(torch.bfloat16)
    dp = lambda t: C.c_void_p(t.data_ptr())
    p.fail_at = {n_create}                                  # the next request is the scratch of the dense phase
    launches = L.wkv_launch_count(h)
    rc = L.wkv_prefill_bulk(h, 0, dp(Q), dp(K), dp(V), None, 48, None, None)
    assert rc == binding.WKV_ERR_ALLOC and b"provider returned NULL" in L.wkv_last_error(h)
    assert L.wkv_launch_count(h) == launches and p.calls == n_create + 1
    # the context is where it was: empty lanes; one decode step works
    out = torch.empty(2, 4, 64, dtype=torch.bfloat16, device="cuda:0")
    ev = torch.empty(2, 4, dtype=torch.int32, device="cuda:0")
    assert L.wkv_decode_step(h, 0, dp(Q[:, 0].contiguous()), dp(K[:, 0].contiguous()), dp(V[:, 0].contiguous()), dp(out),
                             dp(ev), None) == binding.WKV_OK
    assert L.wkv_status(h) == binding.WKV_OK and (ev == -1).all()
    assert L.wkv_reset(h) == binding.WKV_OK
    # second try, provider willing: the prompt goes through and the lanes hold 48 entries
    assert L.wkv_prefill_bulk(h, 0, dp(Q), dp(K), dp(V), None, 48, None, None) == binding.WKV_OK
    n, tok = C.c_int32(), C.c_int32()
    assert L.wkv_export_state(h, 0, 1, 3, C.byref(n), C.byref(tok), None, None, None, None) == binding.WKV_OK
    assert (n.value, tok.value) == (48, 48) and L.wkv_status(h) == binding.WKV_OK
    L.wkv_destroy(h)
    assert not p.live


def test_inconsistent_bookkeeping_is_reported_as_state_error():
    """WKV_ERR_STATE: the host check of an exported lane.  The test owns the device memory (it is the provider), so it
    can damage one lane's state words and links in place; the export of that lane must refuse, the others must not."""
    L = binding.lib()
    p = Provider()
    cfg = p.config(n_layers=1, batch=1, budget=16, window=2, dtype=binding.WKV_F32)
    h = C.c_void_p()
    assert L.wkv_create(C.byref(cfg), C.byref(h)) == binding.WKV_OK
    blocks = list(p.live.values())                          # in request order: K, V, a, pos, next, prev, lane state, ...
    lanes, cap = 4, 20
    nxt = blocks[4].view(torch.int32)[:lanes * cap].view(lanes, cap)
    state = blocks[6].view(torch.int32)[:lanes * 8].view(lanes, 8)
    g = torch.Generator(device="cuda:0").manual_seed(5)
    dp = lambda t: C.c_void_p(t.data_ptr())
    out = torch.empty(1, 4, 64, device="cuda:0")
    for _ in range(24):
        q, k, v = (torch.randn(1, 4, 64, generator=g, device="cuda:0") for _ in range(3))
        assert L.wkv_decode_step(h, 0, dp(q), dp(k), dp(v), dp(out), None, None) == binding.WKV_OK
    n = C.c_int32()
    for lane in range(lanes):
        assert L.wkv_export_state(h, 0, 0, lane, C.byref(n), None, None, None, None, None) == binding.WKV_OK and n.value == 16
    torch.cuda.synchronize()
    assert int(state[1, 0]) == 16 and int(state[1, 1]) == 24      # the blocks are the ones we think they are
    state[1, 0] = 17                                         # lane 1: a length beyond the budget
    head2 = int(state[2, 2])
    nxt[2, head2] = head2                                    # lane 2: the chain loops on its first entry
    torch.cuda.synchronize()
    assert L.wkv_export_state(h, 0, 0, 1, C.byref(n), None, None, None, None, None) == binding.WKV_ERR_STATE
    assert b"length" in L.wkv_last_error(h)
    assert L.wkv_export_state(h, 0, 0, 2, C.byref(n), None, None, None, None, None) == binding.WKV_ERR_STATE
    assert L.wkv_export_state(h, 0, 0, 0, C.byref(n), None, None, None, None, None) == binding.WKV_OK
    assert L.wkv_export_state(h, 0, 0, 3, C.byref(n), None, None, None, None, None) == binding.WKV_OK
    assert L.wkv_strerror(binding.WKV_ERR_STATE).decode().startswith("inconsistent")
    L.wkv_destroy(h)                                         # no further step runs on the damaged lanes
    assert not p.live


def test_provider_refusing_the_blocked_tail_scratch_falls_back_to_streaming():
    """The blocked prompt tail takes its scratch on first use, after the dense part of the prompt has been launched.  A
    refusal there must not lose the prompt: the tail is streamed token by token instead, with the same results."""
    L = binding.lib()
    g = torch.Generator(device="cuda:0").manual_seed(11)
    Q, K, V = (torch.randn(2, 120, 4, 64, generator=g, device="cuda:0").to(torch.bfloat16) for _ in range(3))
    dp = lambda t: C.c_void_p(t.data_ptr())
    states = []
    for refuse in (False, True):
        p = Provider()
        cfg = p.config(n_layers=1, budget=64, window=12, schedule=binding.WKV_SCHEDULE_SPLIT)
        h = C.c_void_p()
        assert L.wkv_create(C.byref(cfg), C.byref(h)) == binding.WKV_OK
        n_create = p.calls
        if refuse:
            p.fail_at = {n_create + 1}                      # request n_create is the dense phase's scratch, the next one the tail's
        launches = L.wkv_launch_count(h)
        assert L.wkv_prefill_bulk(h, 0, dp(Q), dp(K), dp(V), None, 120, None, None) == binding.WKV_OK
        launches = L.wkv_launch_count(h) - launches
        # 64 tokens dense, 56 in blocks of 8 (one sweep + one lane-epilogue launch each) -- or streamed, two launches per token
        assert launches == (1 + 56 * 2 if refuse else 1 + 7 * 2) and p.calls == (n_create + 2 if refuse else n_create + 7)
        assert L.wkv_status(h) == binding.WKV_OK
        pos = torch.empty(64, dtype=torch.int32)
        a = torch.empty(64)
        n = C.c_int32()
        lane_states = []
        for b in range(2):
            for hd in range(4):
                assert L.wkv_export_state(h, 0, b, hd, C.byref(n), None, dp(pos), dp(a), None, None) == binding.WKV_OK
                lane_states.append((n.value, pos.clone(), a.clone()))
        states.append(lane_states)
        L.wkv_destroy(h)
        assert not p.live
    for (n0, p0, a0), (n1, p1, a1) in zip(*states):
        assert n0 == n1 == 64 and torch.equal(p0, p1) and torch.equal(a0, a1)
