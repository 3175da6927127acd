"""GPU tests of the cache's life around the hot path: snapshot by copying the arena and attaching
to the copy, checkpoint / rollback of a live cache, the safe-step budget against a tiny pool, and
the debug aids (range checks on page indices, canary blocks).  Failures are planted on the host
and nothing here can make a kernel touch memory outside the arena: a planted page index names a
ring page of the same arena, and the range check is on."""
import ctypes as C
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import D, Workload, assert_attn_close, compare_state, dev, load, oracle_units, to_dev_bf16

pytestmark = pytest.mark.gpu


def feed(cache, wl, t0, t1, seq=0):
    ids = torch.full((1,), seq, dtype=torch.int32, device=dev())
    K, V = to_dev_bf16(wl.K), to_dev_bf16(wl.V)
    lg = torch.from_numpy(wl.logit).to(dev())
    for t in range(t0, t1):
        cache.spkv_append_evict(0, ids, K[t, :1].contiguous(), V[t, :1].contiguous(), lg[t, :1].contiguous())


def test_attach_to_a_copy_of_the_arena_continues_where_the_original_was():
    spkv = load()
    w, Hq, Hkv, G, T = 32, 4, 2, 2, 400
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=24, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(600, T, 1, Hq, Hkv, [0.3, 0.8], tl)
    feed(cache, wl, 0, 300)
    torch.cuda.synchronize()
    # snapshot = a plain copy of the arena, placed somewhere else (here through the host)
    copy = cache.arena.cpu().to(dev())
    hnd = C.c_void_p()
    s0 = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    # which heads are local-only is part of the layout: an attach that declares some is refused
    flags = np.array([[1, 0]], np.uint8)
    wrong = spkv.Config.from_buffer_copy(cache.cfg)
    wrong.h_local_only = flags.ctypes.data
    assert spkv.lib().spkv_cache_attach(C.byref(wrong), C.c_void_p(copy.data_ptr()), copy.numel(), s0, C.byref(hnd)) == -15
    twin = spkv.Cache.attach(copy, cache.cfg)
    feed(twin, wl, 300, T)
    feed(cache, wl, 300, T)
    units = oracle_units(wl, w, tl)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    q = to_dev_bf16(wl.q[T - 1])
    for c in (cache, twin):
        assert c.spkv_status() == 0
        out = spkv.bits_from_bf16(c.spkv_decode_attention(0, ids, q[:1].contiguous()))[0]
        for h in range(Hkv):
            compare_state(c, 0, 0, h, units[0][h])
            ref = units[0][h].attend(np.ascontiguousarray(wl.q[T - 1, 0, h * G:(h + 1) * G]), 1.0 / math.sqrt(D))
            assert_attn_close(out[h * G:(h + 1) * G], ref, f"kvh {h}")
    # an arena of another configuration, or one that never held a cache, is refused
    other = spkv.Config.from_buffer_copy(cache.cfg)
    other.window = 64
    n = C.c_size_t()
    assert spkv.lib().spkv_arena_bytes(C.byref(other), C.byref(n)) == 0
    big = torch.zeros(max(n.value, copy.numel()), dtype=torch.uint8, device=dev())
    big[:copy.numel()] = copy
    assert spkv.lib().spkv_cache_attach(C.byref(other), C.c_void_p(big.data_ptr()), big.numel(), s0, C.byref(hnd)) == -15
    blank = torch.zeros(copy.numel(), dtype=torch.uint8, device=dev())
    assert spkv.lib().spkv_cache_attach(C.byref(cache.cfg), C.c_void_p(blank.data_ptr()), blank.numel(), s0,
                                        C.byref(hnd)) == -15
    assert spkv.lib().spkv_cache_attach(C.byref(cache.cfg), C.c_void_p(copy.data_ptr()), 1024, s0, C.byref(hnd)) == -2


def test_rollback_replays_the_same_steps_bit_for_bit():
    spkv = load()
    w, Hq, Hkv, G, T = 64, 8, 2, 4, 900
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=40, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(610, T, 1, Hq, Hkv, [0.4, 1.0], tl)
    other = Workload(611, T, 1, Hq, Hkv, [0.9, 0.1], tl)      # what gets rolled back
    feed(cache, wl, 0, 500)
    free0 = cache.spkv_cache_stats().pages_free
    ck = cache.spkv_cache_checkpoint()
    feed(cache, other, 500, 800)                                # crosses page boundaries, pops pages
    assert cache.spkv_cache_stats().pages_free < free0
    cache.spkv_cache_rollback(ck)
    assert cache.spkv_cache_stats().pages_free == free0
    feed(cache, wl, 500, T)
    assert cache.spkv_status() == 0
    units = oracle_units(wl, w, tl)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    out = spkv.bits_from_bf16(cache.spkv_decode_attention(0, ids, to_dev_bf16(wl.q[T - 1])[:1].contiguous()))[0]
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[0][h])
        ref = units[0][h].attend(np.ascontiguousarray(wl.q[T - 1, 0, h * G:(h + 1) * G]), 1.0 / math.sqrt(D))
        assert_attn_close(out[h * G:(h + 1) * G], ref, f"kvh {h}")
    small = torch.empty(16, dtype=torch.uint8, device=dev())
    with pytest.raises(spkv.SpkvError) as e:
        cache.spkv_cache_rollback(small)
    assert e.value.code == -7


def test_safe_step_budget_on_a_tiny_pool():
    """Every evicted pair is kept (tau = -inf, the worst case the budget assumes): the pool runs
    out exactly one step after the budget says zero, never before."""
    spkv = load()
    w, Hkv = 8, 2
    cache = spkv.Cache(n_layers=2, max_seqs=2, n_q_heads=2, n_kv_heads=Hkv, max_context=4096,
                       pool_pages=9, window=w, tau=-math.inf)
    ids = torch.tensor([1], dtype=torch.int32, device=dev())
    k = torch.zeros((1, Hkv, 128), dtype=torch.bfloat16, device=dev())
    lg = torch.zeros((1, Hkv), dtype=torch.float32, device=dev())
    # 4 units (2 layers x 2 heads) of sequence 1 share 9 pages: two pages each, the ninth goes to the
    # first unit that asks: w + 2 * 64 steps are safe, the step after that needs 4 pages and finds 1
    assert cache.spkv_safe_steps([1]) == w + 128
    assert cache.spkv_safe_steps() == w + 64                # all 8 units counted: one page each, the ninth is not enough for a second round
    steps = 0
    while cache.spkv_safe_steps([1]) > 0:
        budget = cache.spkv_safe_steps([1])
        for _ in range(budget):
            for layer in range(2):
                cache.spkv_append_evict(layer, ids, k, k, lg)
        steps += budget
        assert cache.spkv_status() == 0, steps
    assert steps == w + 128
    for layer in range(2):
        cache.spkv_append_evict(layer, ids, k, k, lg)
    assert cache.spkv_status() == -5                        # SPKV_E_POOL_EXHAUSTED, one step past the budget
    with pytest.raises(spkv.SpkvError):
        cache.spkv_safe_steps([2])                          # not a sequence slot


def test_debug_bounds_catch_a_bad_page_index_and_a_trampled_canary():
    spkv = load()
    w, Hq, Hkv, G, T = 64, 4, 2, 2, 700
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=30, window=w, tau=0.5, flags=spkv.FLAG_DEBUG_BOUNDS)
    tl = cache.spkv_tau_logit()
    wl = Workload(620, T, 1, Hq, Hkv, [0.5, 0.9], tl)
    feed(cache, wl, 0, T)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    q = to_dev_bf16(wl.q[T - 1])[:1].contiguous()
    good = cache.spkv_decode_attention(0, ids, q).clone()
    assert cache.spkv_status() == 0                         # checks on, nothing to report
    units = oracle_units(wl, w, tl)
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[0][h])
    # plant a page index that names no pool page (index 0 is a ring page of this same arena, so even
    # an unchecked read would stay inside it) into unit 1's page table
    n_can = C.c_int32()
    offs = (C.c_size_t * 16)()
    assert spkv.lib().spkv_arena_canaries(C.byref(cache.cfg), offs, 16, C.byref(n_can)) == 0
    table_off = offs[2] + 256                               # the page tables follow the third canary
    table = cache.arena[table_off:table_off + 2 * 32 * 4].view(torch.int32)      # 2 units x 32 entries
    saved = int(table[32 + 1].item())
    table[32 + 1] = 0
    cache.spkv_decode_attention(0, ids, q)
    assert cache.spkv_status() == -13                       # SPKV_E_BOUNDS_PAGE, no fault
    table[32 + 1] = saved
    cache.spkv_clear_status()
    again = cache.spkv_decode_attention(0, ids, q)
    assert cache.spkv_status() == 0 and torch.equal(again, good)
    # a canary block that something wrote over is reported by spkv_status
    cache.arena[offs[4] + 17] = 0
    assert cache.spkv_status() == -14
    cache.arena[offs[4] + 17] = 0xC5
    assert cache.spkv_status() == 0
    # without the flag nothing is checked (and nothing was wrong)
    plain = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=30, window=w, tau=0.5)
    feed(plain, wl, 0, T)
    assert torch.equal(plain.spkv_decode_attention(0, ids, q), good) and plain.spkv_status() == 0
