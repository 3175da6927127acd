"""GPU parity, step 3 (decode attention): outputs against the oracle's streaming form
within |gpu - ref| <= 2e-3 + 1e-2 |ref| per element (bf16 inputs and output, fp32
accumulation), log-sum-exp within 1e-3."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import D, Workload, assert_attn_close, dev, load, to_dev_bf16
from paper_2605_14037_b200 import spkv as _unused  # noqa: F401  (fails loudly if the library is missing)
from paper_2605_14037_b200 import synth

pytestmark = pytest.mark.gpu


def run_and_check(spkv, w, T, Hq, Hkv, n_seq, tau, rates, check_steps, seed, sm_scale=None,
                  pool_pages=200, max_context=8192, tweak=None):
    cache = spkv.Cache(n_layers=2, max_seqs=n_seq + 1, n_q_heads=Hq, n_kv_heads=Hkv,
                       max_context=max_context, pool_pages=pool_pages, window=w, tau=tau)
    tl = cache.spkv_tau_logit()
    G = Hq // Hkv
    wl = Workload(seed, T, n_seq, Hq, Hkv, rates, tl)
    if tweak is not None:
        tweak(wl)
    seq_ids = list(range(n_seq, 0, -1))          # slots n_seq..1, reversed order
    ids = torch.tensor(seq_ids, dtype=torch.int32, device=dev())
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    units = [[oracle.Unit(w, D) for _ in range(Hkv)] for _ in range(n_seq)]
    scale = 1.0 / math.sqrt(D) if sm_scale is None else sm_scale
    layer = 1
    lse = torch.empty((n_seq, Hq), dtype=torch.float32, device=dev())
    worst = 0.0
    for t in range(T):
        cache.spkv_append_evict(layer, ids, K[t], V[t], lg[t])
        for s in range(n_seq):
            for h in range(Hkv):
                units[s][h].append(wl.K[t, s, h], wl.V[t, s, h], wl.logit[t, s, h], tl)
        if t in check_steps:
            out = cache.spkv_decode_attention(layer, ids, Q[t], lse=lse, sm_scale=sm_scale)
            got = spkv.bits_from_bf16(out)                      # [n_seq, Hq, D]
            got_lse = lse.cpu().numpy()
            for s in range(n_seq):
                for h in range(Hkv):
                    ref, ref_lse = units[s][h].attend(
                        np.ascontiguousarray(wl.q[t, s, h * G:(h + 1) * G]), scale, want_lse=True)
                    worst = max(worst, assert_attn_close(got[s, h * G:(h + 1) * G], ref,
                                                         f"t={t} seq={s} kvh={h}"))
                    assert np.abs(got_lse[s, h * G:(h + 1) * G] - ref_lse).max() < 1e-3
    assert cache.spkv_status() == 0
    return worst


@pytest.mark.parametrize("w,G,Hkv", [(128, 4, 2), (128, 1, 2), (128, 8, 1), (4, 4, 2), (1, 4, 1),
                                     (100, 2, 2), (128, 16, 1), (128, 3, 2)])
def test_decode_small_every_phase(w, G, Hkv):
    """From the first token (t < w, partially filled ring) across page boundaries."""
    spkv = load()
    T = 330
    steps = set(range(0, 8)) | {w - 2, w - 1, w, w + 1, 63, 64, 65, 127, 128, 129, 191, 192, 193,
                                255, 256, 257, T - 1}
    run_and_check(spkv, w, T, G * Hkv, Hkv, 2, 0.5, np.linspace(0.2, 0.9, Hkv), steps, 50 + w + G)


@pytest.mark.parametrize("tau,rates", [(-math.inf, [0.3, 0.3]), (math.inf, [0.7, 0.7]),
                                       (0.5, [0.0, 1.0]), (0.9, [0.05, 0.5])])
def test_decode_limits(tau, rates):
    """tau = -inf: full causal attention; tau = +inf: sliding window; r = 0 and r = 1 heads."""
    spkv = load()
    run_and_check(spkv, 128, 700, 8, 2, 2, tau, rates, {0, 127, 128, 300, 699}, 60)


def test_decode_many_segments_and_ragged_batch():
    """Units from 2 to ~80 pages in one call: ranges cut inside units, several merges."""
    spkv = load()
    run_and_check(spkv, 128, 5200, 32, 8, 2, 0.5,
                  [0.0, 0.02, 0.1, 0.2, 0.35, 0.5, 0.8, 1.0], {4000, 5199}, 70,
                  pool_pages=700, max_context=8192)


@pytest.mark.parametrize("direction", [1.0, -1.0])
def test_decode_scores_that_grow_or_fall_with_position(direction):
    """Raw scores +-0.4 t for every other query head: the running maximum moves on every tile
    (or never after the first), and the partial results of a unit's page ranges carry maxima
    hundreds apart into the log-sum-exp merge.  The other heads keep ordinary scores."""
    spkv = load()

    def tweak(wl):
        Kf = synth.bf16_bits_to_f32(wl.K)
        Kf[..., 0] = (direction * 0.05 * np.arange(wl.T, dtype=np.float32))[:, None, None]
        wl.K = synth.to_bf16_bits(Kf)
        qf = synth.bf16_bits_to_f32(wl.q)
        qf[:, :, 0::2, :] = 0.0
        qf[:, :, 0::2, 0] = 8.0
        wl.q = synth.to_bf16_bits(qf)

    run_and_check(spkv, 128, 5200, 32, 8, 2, 0.5, [0.0, 0.02, 0.1, 0.2, 0.35, 0.5, 0.8, 1.0],
                  {130, 4000, 5199}, 71, pool_pages=700, max_context=8192, tweak=tweak)


def test_decode_scale_and_batch_of_one():
    spkv = load()
    run_and_check(spkv, 16, 400, 4, 1, 1, 0.5, [0.5], {0, 15, 16, 399}, 80, sm_scale=0.3)


def test_decode_output_is_deterministic_and_repeatable():
    spkv = load()
    cache = spkv.Cache(n_layers=1, max_seqs=2, n_q_heads=8, n_kv_heads=2, max_context=4096,
                       pool_pages=100, window=128, tau=0.5)
    wl = Workload(90, 1500, 2, 8, 2, [0.4, 0.9], 0.0)
    ids = torch.tensor([0, 1], dtype=torch.int32, device=dev())
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    for t in range(wl.T):
        cache.spkv_append_evict(0, ids, K[t], V[t], lg[t])
    a = cache.spkv_decode_attention(0, ids, Q[-1]).clone()
    for _ in range(3):
        b = cache.spkv_decode_attention(0, ids, Q[-1])
        assert torch.equal(a, b)
    # a sub-batch cuts the page ranges elsewhere: same rows up to summation order
    one = cache.spkv_decode_attention(0, ids[1:], Q[-1][1:].contiguous())
    assert torch.allclose(one[0].float(), a[1].float(), atol=2e-3, rtol=1e-2)


def test_decode_workspace_checked():
    spkv = load()
    import ctypes as C
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=2, n_kv_heads=1, max_context=64,
                       pool_pages=1, window=4)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    q = torch.zeros((1, 2, 128), dtype=torch.bfloat16, device=dev())
    rc = spkv.lib().spkv_decode_attention(cache._h, 0, C.c_void_p(ids.data_ptr()), 1,
                                          C.c_void_p(q.data_ptr()), C.c_void_p(q.data_ptr()), None,
                                          0.1, None, 0, None)
    assert rc == -7


@pytest.mark.parametrize("flags", [0, 1])
def test_decode_step_host_pipeline_matches_device_calls(flags):
    """spkv_decode_step_host (pinned host buffers, copies on the cache's own streams, two
    slots in flight) gives bit for bit what the device-pointer calls give, layer after layer
    and step after step, and its outputs are complete after flush + synchronize."""
    spkv = load()
    rng = np.random.default_rng(91)
    L, B, Hq, Hkv, d_in, w, steps = 3, 5, 8, 2, 64, 16, 40
    mk = lambda f: spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=512,
                              pool_pages=L * B * Hkv * 2, window=w, tau=0.5, flags=f)
    ca, cb = mk(flags), mk(0)
    tl = ca.spkv_tau_logit()
    preds = []
    for l in range(L):
        W = synth.linear_predictor(rng, Hkv, d_in)
        b = synth.bias_for_keep_rate(W, [0.3, 0.6], tl)
        preds.append(spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev())))
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    bf = lambda shape: torch.from_numpy(synth.normal_bf16(rng, shape).view(np.int16)).view(torch.bfloat16)
    for t in range(steps):
        hx, hq = bf((L, B, d_in)).pin_memory(), bf((L, B, Hq, D)).pin_memory()
        hk, hv = bf((L, B, Hkv, D)).pin_memory(), bf((L, B, Hkv, D)).pin_memory()
        hout = torch.zeros((L, B, Hq, D), dtype=torch.bfloat16).pin_memory()
        for l in range(L):
            ca.spkv_decode_step_host(l, preds[l], ids, hx[l], hq[l], hk[l], hv[l], hout[l])
        ca.spkv_decode_step_host_flush()
        torch.cuda.current_stream().synchronize()
        for l in range(L):
            cb.spkv_score_append_evict(l, preds[l], ids, hx[l].to(dev()), hk[l].to(dev()), hv[l].to(dev()))
            want = cb.spkv_decode_attention(l, ids, hq[l].to(dev())).cpu()
            assert torch.equal(hout[l].view(torch.int16), want.view(torch.int16)), (t, l)
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0
    for l in range(L):
        la, _ = ca.spkv_read_lengths(l)
        lb, _ = cb.spkv_read_lengths(l)
        assert np.array_equal(la, lb)


@pytest.mark.parametrize("T", [40000, 8 * 64 * 20 + 70])
def test_units_split_over_dozens_of_blocks_merge_on_two_levels(T):
    """Two full-attention units of tens of thousands of pairs are the whole launch: each is cut
    into dozens of block ranges, more than one first-level merge group holds, so the partial
    results are merged group by group and then across groups.  Output and log-sum-exp against
    the oracle; repeated launches are bit-identical (the counters reset themselves)."""
    spkv = load()
    rng = np.random.default_rng(5 + T)
    w, Hq, Hkv, G, B, C = 128, 4, 1, 4, 2, 8192
    cache = spkv.Cache(n_layers=1, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=T + 64,
                       pool_pages=B * (T // 64 + 2), window=w, tau=-math.inf)
    tl = cache.spkv_tau_logit()
    K = synth.normal_bf16(rng, (B, T, Hkv, D))
    V = synth.normal_bf16(rng, (B, T, Hkv, D))
    q = synth.normal_bf16(rng, (B, Hq, D))
    lg = torch.zeros((C, Hkv), dtype=torch.float32, device=dev())
    units = []
    for s in range(B):
        Kd, Vd = to_dev_bf16(K[s]), to_dev_bf16(V[s])
        for a in range(0, T, C):
            n = min(C, T - a)
            cache.spkv_prefill(0, s, Kd[a:a + n], Vd[a:a + n], lg[:n])
        u = oracle.Unit(w, D)
        u.prefill(np.ascontiguousarray(K[s, :, 0]), np.ascontiguousarray(V[s, :, 0]),
                  np.zeros(T, np.float32), tl)
        units.append(u)
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    lse = torch.empty((B, Hq), dtype=torch.float32, device=dev())
    scale = 1.0 / math.sqrt(D)
    out = cache.spkv_decode_attention(0, ids, to_dev_bf16(q), lse=lse).clone()
    again = cache.spkv_decode_attention(0, ids, to_dev_bf16(q))
    assert torch.equal(out.view(torch.int16), again.view(torch.int16))
    assert cache.spkv_status() == 0
    got = spkv.bits_from_bf16(out)
    for s in range(B):
        ref, ref_lse = units[s].attend(q[s], scale, want_lse=True)
        assert_attn_close(got[s], ref, f"long unit {s}")
        assert np.abs(lse[s].cpu().numpy() - ref_lse).max() < 1e-3


@pytest.mark.parametrize("L,B,steps", [(4, 16, 24), (3, 2, 24), (2, 3, 24), (1, 2, 24), (8, 16, 200)])
def test_overlap_mode_is_bit_identical_to_stream_ordered_launches(L, B, steps):
    """SPKV_FLAG_OVERLAP: appends and decodes skip the wait for the whole stream and order
    themselves by per-layer block counters.  A multi-layer decode loop (inputs staged before
    each step, launches back to back, as the benchmark issues them) must give, bit for bit,
    the outputs and cache state of a cache that launches everything stream-ordered.  Two and
    one layer(s) exercise the fall-back when a workspace half comes back to the same layer; the
    long case is there for the orderings that only show up now and then (a dependency wait that
    runs out sets the status word)."""
    spkv = load()
    rng = np.random.default_rng(300 + L * 10 + B)
    Hq, Hkv, d_in, w, T0 = 8, 2, 64, 128, 700
    mk = lambda flags: spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                                  pool_pages=L * B * Hkv * 14, window=w, tau=0.5, flags=flags)
    ca, cb = mk(spkv.FLAG_OVERLAP), mk(0)
    tl = ca.spkv_tau_logit()
    preds = []
    for l in range(L):
        W = synth.linear_predictor(rng, Hkv, d_in)
        b = synth.bias_for_keep_rate(W, [0.2, 0.9], tl)
        preds.append(spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev())))
    bf = lambda shape: to_dev_bf16(synth.normal_bf16(rng, shape))
    for l in range(L):                       # some history, so that units span several blocks
        for s in range(B):
            k, v = bf((T0, Hkv, D)), bf((T0, Hkv, D))
            lg = torch.from_numpy(synth.logits_with_keep_rate(rng, (T0, Hkv), 0.6, tl)).to(dev())
            for c in (ca, cb):
                c.spkv_prefill(l, s, k, v, lg)
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    for t in range(steps):
        x, q = bf((L, B, d_in)), bf((L, B, Hq, D))
        k, v = bf((L, B, Hkv, D)), bf((L, B, Hkv, D))
        outs = []
        for c in (ca, cb):
            o = torch.empty((L, B, Hq, D), dtype=torch.bfloat16, device=dev())
            torch.cuda.synchronize()         # the step's inputs are complete before its first launch
            for l in range(L):
                c.spkv_score_append_evict(l, preds[l], ids, x[l], k[l], v[l])
                c.spkv_decode_attention(l, ids, q[l], out=o[l])
            outs.append(o)
        torch.cuda.synchronize()
        assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16)), t
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0
    for l in range(L):
        la, ta = ca.spkv_read_lengths(l)
        lb, tb = cb.spkv_read_lengths(l)
        assert np.array_equal(la, lb) and np.array_equal(ta, tb)
        for s in range(B):
            for h in range(Hkv):
                pa, ka, va = ca.spkv_read_kept(l, s, h)
                pb, kb, vb = cb.spkv_read_kept(l, s, h)
                assert np.array_equal(pa, pb) and np.array_equal(ka, kb) and np.array_equal(va, vb)


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("L", [1, 3, 4, 5, 9, 33])
def test_decode_stack_host_matches_device_calls(flags, L):
    """spkv_decode_stack_host (the layers in chunks -- head, bulk, tail -- each with its copies in,
    its kernels back to back and its copy out) against the device-pointer calls, bit for bit,
    with and without overlap mode, for stacks too short for three chunks, just long enough, and
    long enough for a head and tail of two layers."""
    spkv = load()
    rng = np.random.default_rng(123 + flags)
    B, Hq, Hkv, d_in, w, steps = 3, 8, 2, 64, 16, 30
    mk = lambda f: spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=512,
                              pool_pages=L * B * Hkv * 2, window=w, tau=0.5, flags=f)
    ca, cb = mk(flags), mk(0)
    tl = ca.spkv_tau_logit()
    preds = []
    for l in range(L):
        W = synth.linear_predictor(rng, Hkv, d_in)
        b = synth.bias_for_keep_rate(W, [0.3, 0.6], tl)
        preds.append(spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev())))
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    bf = lambda shape: torch.from_numpy(synth.normal_bf16(rng, shape).view(np.int16)).view(torch.bfloat16)
    for t in range(steps):
        hx, hq = bf((L, B, d_in)).pin_memory(), bf((L, B, Hq, D)).pin_memory()
        hk, hv = bf((L, B, Hkv, D)).pin_memory(), bf((L, B, Hkv, D)).pin_memory()
        hout = torch.zeros((L, B, Hq, D), dtype=torch.bfloat16).pin_memory()
        ca.spkv_decode_stack_host(preds, ids, hx, hq, hk, hv, hout)
        torch.cuda.current_stream().synchronize()
        for l in range(L):
            cb.spkv_score_append_evict(l, preds[l], ids, hx[l].to(dev()), hk[l].to(dev()), hv[l].to(dev()))
            want = cb.spkv_decode_attention(l, ids, hq[l].to(dev())).cpu()
            assert torch.equal(hout[l].view(torch.int16), want.view(torch.int16)), (t, l)
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0


@pytest.mark.parametrize("kernel_rows", [(128, 5200, 32, 8, [0.0, 0.02, 0.1, 0.2, 0.35, 0.5, 0.8, 1.0], 700),
                                         (16, 700, 8, 2, [0.3, 0.9], 60)])
def test_decode_float32_output_at_2e_5(kernel_rows):
    """spkv_decode_attention_f32 returns the rows before their rounding to bf16, which lets the
    kernel be held to 2e-5 (bf16 output rounding alone is up to 2^-9 |o|): what is left is the
    hi + lo split of P (at most 2^-17 = 7.6e-6 of sum p |v| / l), the exp2 approximation (~2^-22)
    and fp32 accumulation order.  Measured worst: 2.7e-6 (tensor-core kernel), 3e-7 (CUDA-core one).
    The bf16 rows of the same call must be exactly the rounded float32 rows."""
    spkv = load()
    w, T, Hq, Hkv, rates, pool = kernel_rows
    G = Hq // Hkv
    cache = spkv.Cache(n_layers=1, max_seqs=2, n_q_heads=Hq, n_kv_heads=Hkv, max_context=8192,
                       pool_pages=pool, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(91, T, 2, Hq, Hkv, rates, tl)
    ids = torch.tensor([1, 0], dtype=torch.int32, device=dev())
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    units = [[oracle.Unit(w, D) for _ in range(Hkv)] for _ in range(2)]
    scale = 1.0 / math.sqrt(D)
    worst = 0.0
    for t in range(T):
        cache.spkv_append_evict(0, ids, K[t], V[t], lg[t])
        for s in range(2):
            for h in range(Hkv):
                units[s][h].append(wl.K[t, s, h], wl.V[t, s, h], wl.logit[t, s, h], tl)
        if t in (0, w - 1, w, T // 2, T - 1):
            out, out32 = cache.spkv_decode_attention_f32(0, ids, Q[t])
            assert torch.equal(out, out32.to(torch.bfloat16))
            got = out32.cpu().numpy().astype(np.float64)
            for s in range(2):
                for h in range(Hkv):
                    ref = units[s][h].attend(np.ascontiguousarray(wl.q[t, s, h * G:(h + 1) * G]), scale)
                    err = np.abs(got[s, h * G:(h + 1) * G] - ref)
                    assert (err <= 2e-5 + 2e-5 * np.abs(ref)).all(), (t, s, h, float(err.max()))
                    worst = max(worst, float(err.max()))
    assert cache.spkv_status() == 0
    print("worst abs error of the float32 rows:", worst)


@pytest.mark.parametrize("L,B", [(4, 16), (2, 3), (3, 5), (1, 2)])
def test_graph_replay_in_overlap_mode_matches_eager_launches(L, B):
    """The benchmark's launch configuration: one step of the layer stack (fused score + append,
    decode, per layer) captured once into a CUDA graph on an overlap-mode cache and replayed
    step after step, the step's inputs copied into fixed staging tensors before each replay.
    Outputs and final cache state must equal, bit for bit, those of a plain cache that launches
    every kernel eagerly and stream-ordered."""
    spkv = load()
    rng = np.random.default_rng(900 + L + B)
    Hq, Hkv, d_in, w, T0, steps = 8, 2, 64, 128, 500, 40
    mk = lambda flags: spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                                  pool_pages=L * B * Hkv * 12, window=w, tau=0.5, flags=flags)
    ca, cb = mk(spkv.FLAG_OVERLAP), mk(0)
    tl = ca.spkv_tau_logit()
    preds = []
    for l in range(L):
        W = synth.linear_predictor(rng, Hkv, d_in)
        b = synth.bias_for_keep_rate(W, [0.3, 0.8], tl)
        preds.append(spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev())))
    bf = lambda shape: to_dev_bf16(synth.normal_bf16(rng, shape))
    for l in range(L):
        for s in range(B):
            k, v = bf((T0, Hkv, D)), bf((T0, Hkv, D))
            lg = torch.from_numpy(synth.logits_with_keep_rate(rng, (T0, Hkv), 0.5, tl)).to(dev())
            for c in (ca, cb):
                c.spkv_prefill(l, s, k, v, lg)
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    xs, qs = torch.empty((L, B, d_in), dtype=torch.bfloat16, device=dev()), torch.empty((L, B, Hq, D), dtype=torch.bfloat16, device=dev())
    ks, vs = torch.empty((L, B, Hkv, D), dtype=torch.bfloat16, device=dev()), torch.empty((L, B, Hkv, D), dtype=torch.bfloat16, device=dev())
    out_a = torch.empty((L, B, Hq, D), dtype=torch.bfloat16, device=dev())
    ca.decode_workspace(B)                  # allocate before the capture

    def layer_calls(c, x, q, k, v, o):
        for l in range(L):
            c.spkv_score_append_evict(l, preds[l], ids, x[l], k[l], v[l])
            c.spkv_decode_attention(l, ids, q[l], out=o[l])

    inputs = [(bf((L, B, d_in)), bf((L, B, Hq, D)), bf((L, B, Hkv, D)), bf((L, B, Hkv, D))) for _ in range(steps + 1)]

    def stage(i):
        x, q, k, v = inputs[i]
        xs.copy_(x); qs.copy_(q); ks.copy_(k); vs.copy_(v)

    # warm-up step outside the capture (both caches take it), then capture one step
    stage(0)
    side = torch.cuda.Stream(device=dev())
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        layer_calls(ca, xs, qs, ks, vs, out_a)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    out_b = torch.empty_like(out_a)
    layer_calls(cb, *inputs[0], out_b)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        layer_calls(ca, xs, qs, ks, vs, out_a)
    # the capture itself launched nothing: replay it for steps 1..n
    for i in range(1, steps + 1):
        stage(i)
        graph.replay()
        layer_calls(cb, *inputs[i], out_b)
        torch.cuda.synchronize()
        assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)), i
    assert ca.spkv_status() == 0 and cb.spkv_status() == 0
    for l in range(L):
        la, ta = ca.spkv_read_lengths(l)
        lb, tb = cb.spkv_read_lengths(l)
        assert np.array_equal(la, lb) and np.array_equal(ta, tb)
        for s in range(B):
            for h in range(Hkv):
                pa, ka, va = ca.spkv_read_kept(l, s, h)
                pb, kb, vb = cb.spkv_read_kept(l, s, h)
                assert np.array_equal(pa, pb) and np.array_equal(ka, kb) and np.array_equal(va, vb)
