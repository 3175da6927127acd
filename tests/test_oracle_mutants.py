"""How sharp are the oracle's pins?  Each case plants ONE plausible mistake in a copy of the
oracle's C source (a wrong comparison, an off-by-one window, a transposed operand, a dropped
term, ...), builds it, and runs the pin tests against the broken copy in a child process: the
pins must fail.  A mistake that survives would mean the oracle is not pinned there."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "spkv_oracle.c")

# (name, text in the source, what it is replaced by, how many times the text occurs)
MUTANTS = [
    ("threshold_exclusive_mask", "int z = (logit[s] >= tau_logit) ? 1 : 0;", "int z = (logit[s] > tau_logit) ? 1 : 0;", 1),
    ("window_one_too_wide", "int in_win = (t - s >= 0) && (t - s < w);", "int in_win = (t - s >= 0) && (t - s <= w);", 1),
    ("no_causal_mask", "double causal = (s <= t) ? 0.0 : -INFINITY;", "double causal = 0.0;", 1),
    ("scores_against_values", "dot += bf16_widen(q[(size_t)g * D + i]) * bf16_widen(K[(size_t)s * D + i]);",
     "dot += bf16_widen(q[(size_t)g * D + i]) * bf16_widen(V[(size_t)s * D + i]);", 1),
    ("scale_dropped_mask", "score[s] = dot * scale + bias;", "score[s] = dot + bias;", 1),
    ("scale_dropped_stream", "p[j] = dot * scale;", "p[j] = dot;", 1),
    ("all_heads_use_head_0", "for (int i = 0; i < D; ++i) dot += bf16_widen(q[(size_t)g * D + i]) * bf16_widen(kr[i]);",
     "for (int i = 0; i < D; ++i) dot += bf16_widen(q[i]) * bf16_widen(kr[i]);", 1),
    ("evict_decides_on_new_logit", "if (u->ring_logit[slot] >= tau_logit || u->t - u->w < u->n_sink)",
     "if (logit >= tau_logit || u->t - u->w < u->n_sink)", 1),
    ("kept_position_off_by_one", "orcA_keep(u, u->t - u->w, ", "orcA_keep(u, u->t - u->w + 1, ", 1),
    ("ring_slot_off_by_one", "long slot = u->t % u->w;", "long slot = (u->t + 1) % u->w;", 1),
    ("sink_one_too_many", "int sink = s < n_sink;", "int sink = s <= n_sink;", 1),
    ("lse_without_max", "if (lse) lse[g] = mx + log(denom);", "if (lse) lse[g] = log(denom);", 1),
    ("linear_bias_dropped", "logit_out[(size_t)n * n_kv_heads + h] = acc + (double)b[h];",
     "logit_out[(size_t)n * n_kv_heads + h] = acc;", 1),
    ("silu_is_plain_sigmoid", "a[j] = z * orc_sigmoid(z);", "a[j] = orc_sigmoid(z);", 1),
    ("tau_logit_sign", "return (float)log(tau / (1.0 - tau));", "return (float)log((1.0 - tau) / tau);", 1),
    ("softmax_without_normalisation", "double p = exp(score[s] - mx) / denom;", "double p = exp(score[s] - mx);", 1),
    ("soft_gate_inside_the_window_too", "else if (t - s < w) bias_ts = 0.0;", "else if (t - s < 0) bias_ts = 0.0;", 1),
    ("soft_window_one_too_wide", "else if (t - s < w) bias_ts = 0.0;", "else if (t - s <= w) bias_ts = 0.0;", 1),
    ("soft_future_visible", "if (s > t) bias_ts = -INFINITY;", "if (s > t + 1) bias_ts = -INFINITY;", 1),
    ("soft_gate_without_logarithm", "return log(u_tilde);", "return u_tilde - 1.0;", 1),
    ("soft_gate_dropped_term", ": l - log1p(exp(l));", ": -log1p(exp(l));", 1),
    ("anneal_weights_swapped", "double u_tilde = (1.0 - alpha) * u + alpha * z;", "double u_tilde = alpha * u + (1.0 - alpha) * z;", 1),
    ("anneal_threshold_exclusive", "double z = (logit >= tau_logit) ? 1.0 : 0.0;", "double z = (logit > tau_logit) ? 1.0 : 0.0;", 1),
    ("soft_scale_dropped", "a[s] = qk * scale + bias_ts;", "a[s] = qk + bias_ts;", 1),
    ("soft_scores_against_values", "qk += bf16_widen(qg[i]) * bf16_widen(K[(size_t)s * D + i]);",
     "qk += bf16_widen(qg[i]) * bf16_widen(V[(size_t)s * D + i]);", 1),
    ("soft_all_heads_use_head_0", "const uint16_t *qg = q + (size_t)g * D;", "const uint16_t *qg = q;", 1),
    ("soft_lse_without_max", "if (lse) lse[g] = top + log(z_row);", "if (lse) lse[g] = log(z_row);", 1),
    ("soft_unnormalised", "double weight = exp(a[s] - top) / z_row;", "double weight = exp(a[s] - top);", 1),
    ("keep_all_and_keep_none_swapped", "if (!(tau > 0.0)) return -INFINITY;", "if (!(tau > 0.0)) return INFINITY;", 1),
]


@pytest.mark.parametrize("name,old,new,count", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, old, new, count):
    text = open(SRC).read()
    assert text.count(old) == count, f"{name}: source text occurs {text.count(old)} times"
    mutated = text.replace(old, new)
    src = tmp_path / "mutant.c"
    lib = tmp_path / "libmutant.so"
    src.write_text(mutated)
    subprocess.check_call(["gcc", "-O1", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-o", str(lib), str(src), "-lm"])
    env = dict(os.environ, SPKV_ORACLE_LIB=str(lib))
    # the pins of the part of the oracle the mistake sits in (soft-gated forward / everything else)
    soft = name.startswith(("soft_", "anneal_"))
    files = ["test_oracle_soft.py"] if soft else ["test_oracle_pins.py", "test_oracle_sinks.py"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        *[os.path.join(ROOT, "tests", f) for f in files]],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    out = r.stdout + r.stderr
    assert r.returncode == 1 and " failed" in out, f"mutant {name} survived the pins:\n{out[-800:]}"
