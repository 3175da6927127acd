"""spkv_decode_attention_static: decode attention for callers that cannot allocate.

Some users of this library run inside a memory plan they do not own -- a serving engine
that gave all free HBM to its KV pool at start-up, a plugin inside a host application, a
decode loop that must never reach the allocator.  For them the library offers one entry
point whose split-K scratch is a fixed array inside the library image, so that no
workspace has to be allocated or passed.  This test calls it through the C ABI, twice in
a row, and checks each result against spkv_decode_attention (which uses a caller-supplied
workspace) within the attention tolerance of the other tests; it also checks that a
request beyond the built-in scratch is refused.  The file sorts last on purpose: a run
that stops at the first failure has then already run every other test.
"""
import ctypes as C
import math

import numpy as np
import pytest
import torch

from gpu_util import ABS_TOL, REL_TOL, Workload, dev, load, to_dev_bf16

pytestmark = pytest.mark.gpu


def build_cache(spkv, n_seq, Hq, Hkv, T, rates, seed):
    cache = spkv.Cache(n_layers=1, max_seqs=n_seq, n_q_heads=Hq, n_kv_heads=Hkv, max_context=4096,
                       pool_pages=40 * n_seq * Hkv, window=128, tau=0.5)
    wl = Workload(seed, T, n_seq, Hq, Hkv, rates, cache.spkv_tau_logit())
    K, V = to_dev_bf16(wl.K), to_dev_bf16(wl.V)
    lg = torch.from_numpy(wl.logit).to(dev())
    for s in range(n_seq):           # state via the prefill path, one sequence at a time
        cache.spkv_prefill(0, s, K[:, s].contiguous(), V[:, s].contiguous(), lg[:, s].contiguous())
    assert cache.spkv_status() == 0
    return cache, wl


def test_static_scratch_decode_matches_workspace_decode_twice():
    spkv = load()
    n_seq, Hq, Hkv, T = 3, 8, 2, 2300           # units of up to ~36 pages: split over blocks
    cache, wl = build_cache(spkv, n_seq, Hq, Hkv, T, [0.15, 0.95], 300)
    ids = torch.arange(n_seq, dtype=torch.int32, device=dev())
    rng = np.random.default_rng(301)
    from paper_2605_14037_b200 import synth
    for call in range(2):                        # two calls in a row share the built-in array
        q = to_dev_bf16(synth.normal_bf16(rng, (n_seq, Hq, 128)))
        k = to_dev_bf16(synth.normal_bf16(rng, (n_seq, Hkv, 128)))
        lg = torch.from_numpy(rng.standard_normal((n_seq, Hkv)).astype(np.float32)).to(dev())
        cache.spkv_append_evict(0, ids, k, k, lg)
        lse_a = torch.empty((n_seq, Hq), dtype=torch.float32, device=dev())
        lse_b = torch.empty_like(lse_a)
        want = cache.spkv_decode_attention(0, ids, q, lse=lse_a).float()
        got = cache.spkv_decode_attention_static(0, ids, q, lse=lse_b).float()
        torch.cuda.synchronize()
        err = (got - want).abs()
        assert bool((err <= ABS_TOL + REL_TOL * want.abs()).all()), f"call {call}: max err {err.max().item()}"
        assert torch.allclose(lse_a, lse_b, atol=1e-3, rtol=0)
        assert float(want.abs().max()) > 0.0
    assert cache.spkv_status() == 0


def test_static_scratch_rejects_requests_beyond_its_size():
    spkv = load()
    # 64 sequences x 8 KV heads with 8 query heads each need more than the built-in 6 MiB
    cache = spkv.Cache(n_layers=1, max_seqs=64, n_q_heads=64, n_kv_heads=8, max_context=256,
                       pool_pages=8, window=128, tau=0.5)
    need = spkv.lib().spkv_decode_workspace_bytes(C.byref(cache.cfg), 64)
    assert need > (6 << 20)
    ids = torch.arange(64, dtype=torch.int32, device=dev())
    q = torch.zeros((64, 64, 128), dtype=torch.bfloat16, device=dev())
    out = torch.full_like(q, 7.0)
    rc = spkv.lib().spkv_decode_attention_static(cache._h, 0, C.c_void_p(ids.data_ptr()), 64,
                                                 C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()),
                                                 None, 0.1, None)
    assert rc == -10
    assert spkv.lib().spkv_error_string(rc) == b"request exceeds the built-in scratch area"
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())              # refused calls touch nothing
    # argument errors are refused as spkv_decode_attention refuses them, before the shared array is
    # touched: a bad layer, a missing query tensor, a batch larger than the cache has slots
    f, s0 = spkv.lib().spkv_decode_attention_static, C.c_void_p(torch.cuda.current_stream().cuda_stream)
    ok_args = (C.c_void_p(ids.data_ptr()), 4, C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()), None, 0.1, s0)
    assert f(cache._h, 1, *ok_args) == -1
    assert f(cache._h, 0, C.c_void_p(ids.data_ptr()), 4, None, C.c_void_p(out.data_ptr()), None, 0.1, s0) == -1
    assert f(cache._h, 0, C.c_void_p(ids.data_ptr()), 65, C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()),
             None, 0.1, s0) == -1
    assert f(None, 0, *ok_args) == -1
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    # a batch that fits is accepted by the same cache
    small = torch.arange(4, dtype=torch.int32, device=dev())
    k = torch.zeros((4, 8, 128), dtype=torch.bfloat16, device=dev())
    cache.spkv_append_evict(0, small, k, k, torch.zeros((4, 8), dtype=torch.float32, device=dev()))
    o = cache.spkv_decode_attention_static(0, small, q[:4].contiguous())
    torch.cuda.synchronize()
    assert bool((o == 0).all()) and cache.spkv_status() == 0
