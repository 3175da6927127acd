"""GPU parity, step 1 (score + threshold): float32 logits against the double-precision
oracle, and decisions that agree wherever the logit is not within rounding of tau."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev, load, to_dev_bf16
from paper_2605_14037_b200 import synth

pytestmark = pytest.mark.gpu

# bf16 products are exact in float32; a length-d float32 accumulation of O(1) terms errs
# by about d * 2^-24 * |partial sums| -- far below 1e-3 for d <= 8192.
LOGIT_TOL = 1e-3


def make_cache(spkv, Hkv, tau=0.5):
    return spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hkv, n_kv_heads=Hkv, max_context=64,
                      pool_pages=1, window=4, tau=tau)


@pytest.mark.parametrize("n_tok,d_in,Hkv", [(1, 512, 2), (16, 512, 8), (1000, 512, 8),
                                            (37, 8, 1), (5, 4096, 3)])
def test_linear_predictor(n_tok, d_in, Hkv):
    spkv = load()
    rng = np.random.default_rng(20 + n_tok)
    cache = make_cache(spkv, Hkv, tau=0.7)
    tl = cache.spkv_tau_logit()
    x = synth.normal_bf16(rng, (n_tok, d_in))
    W = synth.linear_predictor(rng, Hkv, d_in)
    b = synth.bias_for_keep_rate(W, np.linspace(0.1, 0.9, Hkv), tl)
    pred = spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev()))
    flags = torch.zeros((n_tok, Hkv), dtype=torch.uint8, device=dev())
    got = cache.spkv_score(pred, to_dev_bf16(x), flags=flags).cpu().numpy()
    ref = oracle.score_linear(x, W, b)
    assert np.abs(got - ref).max() < LOGIT_TOL
    f = flags.cpu().numpy().astype(bool)
    assert np.array_equal(f, got >= np.float32(tl))            # flag == decision on the fp32 logit
    differ = f != (ref >= float(tl))
    assert (np.abs(ref[differ] - float(tl)) < LOGIT_TOL).all()  # only inside the rounding band


# 64 tokens and more go to the tensor-core kernel when hidden is a multiple of 16 up to 256 and
# hidden x heads (rounded up to 8) <= 4096; the other cases run on the CUDA cores
@pytest.mark.parametrize("n_tok,d_in,hidden,Hkv", [(1, 512, 64, 2), (16, 512, 256, 8),
                                                   (300, 256, 64, 4), (3, 1024, 8, 1),
                                                   (2000, 4096, 256, 8),     # model width, ragged last tile
                                                   (129, 520, 48, 3),        # d_in not a multiple of 64
                                                   (64, 64, 16, 16), (1000, 512, 128, 32),
                                                   (500, 512, 256, 24),      # second layer too big for shared memory
                                                   (256, 8192, 240, 5)])
def test_mlp_predictor(n_tok, d_in, hidden, Hkv):
    spkv = load()
    rng = np.random.default_rng(30 + n_tok)
    cache = make_cache(spkv, Hkv)
    tl = cache.spkv_tau_logit()
    x = synth.normal_bf16(rng, (n_tok, d_in))
    W1, b1, W2, b2 = synth.mlp_predictor(rng, Hkv, d_in, hidden)
    pred = spkv.make_predictor(to_dev_bf16(W1), torch.from_numpy(b1).to(dev()),
                               to_dev_bf16(W2), torch.from_numpy(b2).to(dev()))
    flags = torch.zeros((n_tok, Hkv), dtype=torch.uint8, device=dev())
    got = cache.spkv_score(pred, to_dev_bf16(x), flags=flags).cpu().numpy()
    ref = oracle.score_mlp(x, W1, b1, W2, b2)
    assert np.abs(got - ref).max() < LOGIT_TOL
    f = flags.cpu().numpy().astype(bool)
    assert np.array_equal(f, got >= np.float32(tl))
    differ = f != (ref >= float(tl))
    assert (np.abs(ref[differ] - float(tl)) < LOGIT_TOL).all()


def test_score_then_append_chain_is_bit_exact_outside_the_guard_band():
    """Tokens whose oracle logit lies within the rounding band of tau are resampled, after
    which GPU-scored logits drive the same keep decisions as oracle-scored ones."""
    spkv = load()
    rng = np.random.default_rng(40)
    Hkv, d_in, T, w = 2, 512, 500, 16
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hkv, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=20, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    W = synth.linear_predictor(rng, Hkv, d_in)
    b = synth.bias_for_keep_rate(W, [0.2, 0.5], tl)
    x = synth.normal_bf16(rng, (T, d_in))
    for _ in range(10):
        ref = oracle.score_linear(x, W, b)
        near = (np.abs(ref - float(tl)) < LOGIT_TOL).any(axis=1)
        if not near.any():
            break
        x[near] = synth.normal_bf16(rng, (int(near.sum()), d_in))
    K, V = synth.normal_bf16(rng, (T, Hkv, 128)), synth.normal_bf16(rng, (T, Hkv, 128))
    pred = spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev()))
    xd, Kd, Vd = to_dev_bf16(x), to_dev_bf16(K), to_dev_bf16(V)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    for t in range(T):
        lg = cache.spkv_score(pred, xd[t:t + 1])
        cache.spkv_append_evict(0, ids, Kd[t:t + 1], Vd[t:t + 1], lg)
    for h in range(Hkv):
        u = oracle.Unit(w, 128)
        u.prefill(np.ascontiguousarray(K[:, h]), np.ascontiguousarray(V[:, h]),
                  ref[:, h].astype(np.float32), tl)
        pos, k, v = cache.spkv_read_kept(0, 0, h)
        assert np.array_equal(pos, u.kept()[0]) and np.array_equal(k, u.kept()[1])


@pytest.mark.parametrize("kind", ["linear", "mlp"])
def test_fused_score_append_equals_separate_calls(kind):
    """spkv_score_append_evict == spkv_score followed by spkv_append_evict, bit for bit."""
    spkv = load()
    rng = np.random.default_rng(41)
    Hkv, d_in, T, w, B = 4, 512, 300, 8, 3
    mk = lambda: spkv.Cache(n_layers=1, max_seqs=B, n_q_heads=Hkv, n_kv_heads=Hkv, max_context=1024,
                            pool_pages=40, window=w, tau=0.5)
    a, b = mk(), mk()
    if kind == "linear":
        W = synth.linear_predictor(rng, Hkv, d_in)
        bias = synth.bias_for_keep_rate(W, [0.1, 0.3, 0.6, 0.9], 0.0)
        pred = spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(bias).to(dev()))
    else:
        W1, b1, W2, b2 = synth.mlp_predictor(rng, Hkv, d_in, 64)
        pred = spkv.make_predictor(to_dev_bf16(W1), torch.from_numpy(b1).to(dev()),
                                   to_dev_bf16(W2), torch.from_numpy(b2).to(dev()))
    x = to_dev_bf16(synth.normal_bf16(rng, (T, B, d_in)))
    K = to_dev_bf16(synth.normal_bf16(rng, (T, B, Hkv, 128)))
    V = to_dev_bf16(synth.normal_bf16(rng, (T, B, Hkv, 128)))
    ids = torch.tensor([2, 0, 1], dtype=torch.int32, device=dev())
    lg_f = torch.empty((B, Hkv), dtype=torch.float32, device=dev())
    for t in range(T):
        lg = a.spkv_score(pred, x[t])
        a.spkv_append_evict(0, ids, K[t], V[t], lg)
        b.spkv_score_append_evict(0, pred, ids, x[t], K[t], V[t], logits_out=lg_f)
        assert torch.equal(lg, lg_f)
    for s in range(B):
        for h in range(Hkv):
            for p, q in zip(a.spkv_read_kept(0, s, h), b.spkv_read_kept(0, s, h)):
                assert np.array_equal(p, q)
            for p, q in zip(a.spkv_read_window(0, s, h), b.spkv_read_window(0, s, h)):
                assert np.array_equal(p, q)
    assert a.spkv_status() == 0 and b.spkv_status() == 0
