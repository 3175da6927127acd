"""spkv_decode_stack: one decode step of the whole layer stack in two launches (the appends of
every layer, then one persistent decode-attention kernel over all layers).  Checked against the
oracle's streaming form unit by unit (state bit-exact, outputs at the attention tolerance), and
against the per-layer calls it replaces on a second cache with the same flags (same state,
logits and outputs, bit for bit)."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import D, assert_attn_close, compare_state, dev, load, to_dev_bf16
from paper_2605_14037_b200 import synth

pytestmark = pytest.mark.gpu


def make_stack(spkv, rng, L, B, Hq, Hkv, T0, w, rates, d_in, tau=0.5, flags=0, max_context=8192, pool_pages=None):
    """Two caches in the same state after T0 tokens per sequence (built by the prefill path from
    logits of the layers' linear predictors), the predictors, and the oracle units [L][B][Hkv]."""
    pool = pool_pages if pool_pages is not None else L * B * Hkv * ((T0 + 200) // 64 + 3)
    mk = lambda f: spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=max_context,
                              pool_pages=pool, window=w, tau=tau, flags=f)
    ca, cb = mk(flags), mk(flags)
    tl = ca.spkv_tau_logit()
    preds, units = [], [[[oracle.Unit(w, D) for _ in range(Hkv)] for _ in range(B)] for _ in range(L)]
    for l in range(L):
        W = synth.linear_predictor(rng, Hkv, d_in)
        r = np.roll(np.asarray(rates, dtype=np.float64), l)[:Hkv]
        b = synth.bias_for_keep_rate(W, r, tl if math.isfinite(tl) else 0.0)
        pred = spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev()))
        preds.append(pred)
        for s in range(B):
            T_s = max(0, T0 - 37 * s)          # ragged contexts
            if T_s == 0:
                continue
            x = synth.normal_bf16(rng, (T_s, d_in))
            K, V = synth.normal_bf16(rng, (T_s, Hkv, D)), synth.normal_bf16(rng, (T_s, Hkv, D))
            lg = ca.spkv_score(pred, to_dev_bf16(x))
            for cache in (ca, cb):
                cache.spkv_prefill(l, s, to_dev_bf16(K), to_dev_bf16(V), lg)
            lgh = lg.cpu().numpy()
            for h in range(Hkv):
                units[l][s][h].prefill(np.ascontiguousarray(K[:, h]), np.ascontiguousarray(V[:, h]),
                                       np.ascontiguousarray(lgh[:, h]), tl)
    return ca, cb, preds, units, tl


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("L,B,Hq,Hkv,T0,w,rates,steps", [
    (3, 2, 8, 2, 700, 128, [0.3, 0.9], 3),                       # a few units, split over many blocks
    (5, 3, 8, 2, 300, 16, [0.0, 1.0], 4),                        # local-only and keep-all heads, tiny window
    (2, 4, 32, 8, 2500, 128, [0.0, 0.02, 0.1, 0.2, 0.35, 0.5, 0.8, 1.0], 2),   # the benchmark's head layout
    (4, 1, 16, 1, 1500, 128, [0.6], 2),                          # 16 query heads per KV head
    (1, 2, 6, 2, 400, 100, [0.4, 0.7], 3),                       # one layer, odd group, odd window
    (7, 2, 4, 4, 0, 128, [0.5, 0.5, 0.5, 0.5], 5),               # from an empty cache
    (33, 1, 4, 1, 0, 16, [0.5], 40),                             # many tiny layers: the plan buffers wrap many times
    (12, 2, 8, 2, 90, 16, [0.0, 1.0], 6),                        # layers of a page or two: most blocks visit them empty-handed
])
def test_stack_step_matches_oracle_and_per_layer_calls(L, B, Hq, Hkv, T0, w, rates, steps, flags):
    spkv = load()
    rng = np.random.default_rng(1000 + L * 7 + B)
    d_in, G = 64, Hq // Hkv
    ca, cb, preds, units, tl = make_stack(spkv, rng, L, B, Hq, Hkv, T0, w, rates, d_in, flags=flags)
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    scale = 1.0 / math.sqrt(D)
    for t in range(steps):
        x = synth.normal_bf16(rng, (L, B, d_in))
        q = synth.normal_bf16(rng, (L, B, Hq, D))
        k, v = synth.normal_bf16(rng, (L, B, Hkv, D)), synth.normal_bf16(rng, (L, B, Hkv, D))
        xd, qd, kd, vd = (to_dev_bf16(a) for a in (x, q, k, v))
        lg_a = torch.empty((L, B, Hkv), dtype=torch.float32, device=dev())
        lse_a = torch.empty((L, B, Hq), dtype=torch.float32, device=dev())
        out_a = ca.spkv_decode_stack(preds, ids, xd, qd, kd, vd, logits_out=lg_a, lse=lse_a)
        lg_b = torch.empty_like(lg_a)
        out_b = torch.empty_like(out_a)
        for l in range(L):
            cb.spkv_score_append_evict(l, preds[l], ids, xd[l], kd[l], vd[l], logits_out=lg_b[l])
            cb.spkv_decode_attention(l, ids, qd[l], out=out_b[l])
        torch.cuda.synchronize()
        assert torch.equal(lg_a.view(torch.int32), lg_b.view(torch.int32)), "logits differ from the per-layer call"
        assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)), f"step {t}: outputs differ"
        got, got_lse, lgh = spkv.bits_from_bf16(out_a), lse_a.cpu().numpy(), lg_a.cpu().numpy()
        for l in range(L):
            for s in range(B):
                for h in range(Hkv):
                    u = units[l][s][h]
                    u.append(k[l, s, h], v[l, s, h], lgh[l, s, h], tl)
                    ref, ref_lse = u.attend(np.ascontiguousarray(q[l, s, h * G:(h + 1) * G]), scale, want_lse=True)
                    assert_attn_close(got[l, s, h * G:(h + 1) * G], ref, f"step {t} layer {l} seq {s} kvh {h}")
                    assert np.abs(got_lse[l, s, h * G:(h + 1) * G] - ref_lse).max() < 1e-3
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0
    for l in range(L):
        assert np.array_equal(ca.spkv_read_lengths(l)[0], cb.spkv_read_lengths(l)[0])
        for s in range(B):
            for h in range(Hkv):
                compare_state(ca, l, s, h, units[l][s][h])


def test_stack_step_repeats_bit_for_bit_and_refuses_bad_arguments():
    """The same step from the same state twice gives the same bits (ranges are handed out in a
    different order every time; the results must not depend on it), the range counter is left at
    zero, and argument errors are refused before anything is launched."""
    import ctypes as C
    spkv = load()
    rng = np.random.default_rng(77)
    L, B, Hq, Hkv, d_in = 4, 3, 8, 2, 64
    ca, cb, preds, units, tl = make_stack(spkv, rng, L, B, Hq, Hkv, 900, 128, [0.2, 0.8], d_in)
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    x, q = to_dev_bf16(synth.normal_bf16(rng, (L, B, d_in))), to_dev_bf16(synth.normal_bf16(rng, (L, B, Hq, D)))
    k = to_dev_bf16(synth.normal_bf16(rng, (L, B, Hkv, D)))
    o1 = ca.spkv_decode_stack(preds, ids, x, q, k, k).clone()
    o2 = cb.spkv_decode_stack(preds, ids, x, q, k, k).clone()
    torch.cuda.synchronize()
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    ws = ca._ws["decode_stack"]
    assert int(ws[:4].view(torch.int32).item()) == 0          # the last claim cleared the counter
    f = spkv.lib().spkv_decode_stack
    arr = (spkv.Predictor * L)(*preds)
    p = lambda t: C.c_void_p(t.data_ptr())
    args = lambda **kw: [kw.get("cache", ca._h), C.cast(arr, C.c_void_p), p(ids), kw.get("B", B), kw.get("x", p(x)), p(q),
                         p(k), p(k), p(o1), None, None, 0.1, kw.get("ws", p(ws)), kw.get("nbytes", ws.numel()), None]
    assert f(*args(cache=None)) == -1
    assert f(*args(B=B + 1)) == -1
    assert f(*args(x=None)) == -1
    assert f(*args(nbytes=1024)) == spkv.lib().spkv_decode_attention(ca._h, 0, p(ids), B, p(q), p(o1), None, 0.1,
                                                                     p(ws), 16, None)   # the workspace error code
    assert f(*args(B=0)) == 0
    torch.cuda.synchronize()
    assert ca.spkv_status() == 0


def test_stack_step_with_sinks_local_only_heads_and_per_head_thresholds():
    """The variants of the cache go through the stack step unchanged: sink tokens, a head declared
    local-only at creation (no page table), per-head thresholds set at run time, range checks on.
    Compared bit for bit with the per-layer calls (which test_gpu_sinks / test_gpu_hybrid hold
    against the oracle) from an empty cache over enough steps for evictions and second pages."""
    spkv = load()
    rng = np.random.default_rng(5)
    L, B, Hq, Hkv, w, d_in, steps = 3, 2, 8, 4, 16, 64, 150
    local = np.zeros((L, Hkv), dtype=np.uint8)
    local[1, 2] = 1
    mk = lambda: spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=512, pool_pages=96,
                            window=w, tau=0.5, sink_tokens=3, local_only=local, flags=spkv.FLAG_DEBUG_BOUNDS)
    ca, cb = mk(), mk()
    for c_ in (ca, cb):
        c_.spkv_set_head_tau(0, 1, 1.0)        # a local-only head declared at run time
        c_.spkv_set_head_tau(2, 0, 0.0)        # a full-attention head
    tl = ca.spkv_tau_logit()
    preds = []
    for l in range(L):
        W = synth.linear_predictor(rng, Hkv, d_in)
        preds.append(spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(
            synth.bias_for_keep_rate(W, [0.2, 0.5, 0.8, 0.4], tl)).to(dev())))
    ids = torch.tensor([1, 0], dtype=torch.int32, device=dev())
    for t in range(steps):
        x, q = to_dev_bf16(synth.normal_bf16(rng, (L, B, d_in))), to_dev_bf16(synth.normal_bf16(rng, (L, B, Hq, D)))
        k, v = to_dev_bf16(synth.normal_bf16(rng, (L, B, Hkv, D))), to_dev_bf16(synth.normal_bf16(rng, (L, B, Hkv, D)))
        out_a = ca.spkv_decode_stack(preds, ids, x, q, k, v)
        for l in range(L):
            cb.spkv_score_append_evict(l, preds[l], ids, x[l], k[l], v[l])
            out_b = cb.spkv_decode_attention(l, ids, q[l])
            assert torch.equal(out_a[l].view(torch.int16), out_b.view(torch.int16)), (t, l)
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0
    for l in range(L):
        la, lb = ca.spkv_read_lengths(l)[0], cb.spkv_read_lengths(l)[0]
        assert np.array_equal(la, lb)
    assert ca.spkv_read_lengths(1)[0][:, 2].max() == 0                   # declared local-only: not even the sinks
    assert (ca.spkv_read_lengths(0)[0][:, 1] == 3).all()                 # threshold 1 at run time: the sinks only
    assert ca.spkv_read_lengths(2)[0][:, 0].min() == steps - w          # the full-attention head kept every evictee
    for h in (0, 3):
        assert ca.spkv_read_kept(1, 1, h)[0][:3].tolist() == [0, 1, 2]   # the sinks lead the cache


def test_stack_step_with_two_layer_predictors_makes_the_per_layer_calls():
    """Two-layer predictors are scored by a kernel of their own, so the stack call falls back to the
    per-layer calls inside the library: same results as making them oneself, logits required."""
    spkv = load()
    rng = np.random.default_rng(11)
    L, B, Hq, Hkv, w, d_in, hidden, steps = 3, 2, 8, 2, 16, 64, 32, 40
    mk = lambda: spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=256, pool_pages=48,
                            window=w, tau=0.5)
    ca, cb = mk(), mk()
    preds = []
    for l in range(L):
        W1 = to_dev_bf16(synth.normal_bf16(rng, (hidden, d_in)))
        W2 = to_dev_bf16(synth.normal_bf16(rng, (Hkv, hidden)))
        b1 = torch.from_numpy(rng.standard_normal(hidden).astype(np.float32)).to(dev())
        b2 = torch.from_numpy(rng.standard_normal(Hkv).astype(np.float32)).to(dev())
        preds.append(spkv.make_predictor(W1, b1, W2, b2))
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    for t in range(steps):
        x, q = to_dev_bf16(synth.normal_bf16(rng, (L, B, d_in))), to_dev_bf16(synth.normal_bf16(rng, (L, B, Hq, D)))
        k, v = to_dev_bf16(synth.normal_bf16(rng, (L, B, Hkv, D))), to_dev_bf16(synth.normal_bf16(rng, (L, B, Hkv, D)))
        lg_a = torch.empty((L, B, Hkv), dtype=torch.float32, device=dev())
        out_a = ca.spkv_decode_stack(preds, ids, x, q, k, v, logits_out=lg_a)
        for l in range(L):
            lg_b = torch.empty((B, Hkv), dtype=torch.float32, device=dev())
            cb.spkv_score_append_evict(l, preds[l], ids, x[l], k[l], v[l], logits_out=lg_b)
            out_b = cb.spkv_decode_attention(l, ids, q[l])
            assert torch.equal(lg_a[l].view(torch.int32), lg_b.view(torch.int32)), (t, l)
            assert torch.equal(out_a[l].view(torch.int16), out_b.view(torch.int16)), (t, l)
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0
    with pytest.raises(spkv.SpkvError):                       # two-layer predictors need the logits buffer
        ca.spkv_decode_stack(preds, ids, x, q, k, v)


def test_stack_step_replayed_from_a_cuda_graph_matches_eager_calls():
    """bench.py replays the stack step as a CUDA graph: a captured step, replayed with fresh inputs
    copied into its buffers, against eager calls on a second cache -- outputs and final lengths,
    bit for bit, over enough steps for evictions."""
    spkv = load()
    rng = np.random.default_rng(21)
    L, B, Hq, Hkv, d_in, steps = 4, 3, 8, 2, 64, 12
    ca, cb, preds, units, tl = make_stack(spkv, rng, L, B, Hq, Hkv, 600, 128, [0.3, 0.8], d_in, flags=1)
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    bufs = [torch.zeros(shape, dtype=torch.bfloat16, device=dev())
            for shape in ((L, B, d_in), (L, B, Hq, D), (L, B, Hkv, D), (L, B, Hkv, D))]
    out_g = torch.zeros((L, B, Hq, D), dtype=torch.bfloat16, device=dev())
    ca.spkv_decode_stack(preds, ids, *bufs, out=out_g)          # warm-up outside the capture (same step on both caches)
    cb.spkv_decode_stack(preds, ids, *bufs)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):                                    # capturing runs nothing
        ca.spkv_decode_stack(preds, ids, *bufs, out=out_g)
    for t in range(steps):
        fresh = [to_dev_bf16(synth.normal_bf16(rng, tuple(b.shape))) for b in bufs]
        for b, f in zip(bufs, fresh):
            b.copy_(f)
        g.replay()
        want = cb.spkv_decode_stack(preds, ids, *fresh)
        torch.cuda.synchronize()
        assert torch.equal(out_g.view(torch.int16), want.view(torch.int16)), t
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0
    for l in range(L):
        assert np.array_equal(ca.spkv_read_lengths(l)[0], cb.spkv_read_lengths(l)[0])
