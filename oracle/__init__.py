"""CPU oracle for SP-KV inference attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``spkv_oracle.c`` (plain C, double precision).
Nothing in the product package imports this module; only tests, the smoke
check and the benchmark's CPU-baseline leg do.  It shares no code with the
CUDA library.

Array conventions: bfloat16 data travel as ``numpy.uint16`` bit patterns,
logits as ``float32``, results as ``float64``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spkv_oracle.c")
_LIB = os.path.join(_HERE, "libspkv_oracle.so")

_u16p = np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP for the unit loop only).  SPKV_ORACLE_LIB names a
    ready-made library to load instead (the mutation tests point it at deliberately broken
    copies to show that the pins catch them)."""
    override = os.environ.get("SPKV_ORACLE_LIB")
    if override:
        return override
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        l = C.CDLL(build())
        l.orc_bf16_to_double.restype = C.c_double
        l.orc_bf16_to_double.argtypes = [C.c_uint16]
        l.orc_sigmoid.restype = C.c_double
        l.orc_sigmoid.argtypes = [C.c_double]
        l.orc_tau_logit.restype = C.c_float
        l.orc_tau_logit.argtypes = [C.c_double]
        l.orc_score_linear.restype = None
        l.orc_score_linear.argtypes = [_u16p, C.c_int, C.c_int, _u16p, _f32p, C.c_int, _f64p]
        l.orc_score_mlp.restype = None
        l.orc_score_mlp.argtypes = [_u16p, C.c_int, C.c_int, _u16p, _f32p, C.c_int, _u16p, _f32p,
                                    C.c_int, _f64p]
        l.orcB_attend_row.restype = None
        l.orcB_attend_row.argtypes = [_u16p, _u16p, _f32p, C.c_int, C.c_int, C.c_int, C.c_float,
                                      _u16p, C.c_int, C.c_int, C.c_double, _f64p, C.c_void_p]
        l.orcB_attend_row_sinks.restype = None
        l.orcB_attend_row_sinks.argtypes = [_u16p, _u16p, _f32p, C.c_int, C.c_int, C.c_int, C.c_float,
                                            C.c_int, _u16p, C.c_int, C.c_int, C.c_double, _f64p,
                                            C.c_void_p]
        l.orcB_attend_all_sinks.restype = None
        l.orcB_attend_all_sinks.argtypes = [_u16p, _u16p, _f32p, C.c_int, C.c_int, C.c_float, C.c_int,
                                            _u16p, C.c_int, C.c_int, C.c_double, _f64p]
        l.orcA_set_sinks.restype = None
        l.orcA_set_sinks.argtypes = [C.c_void_p, C.c_int]
        l.orcB_attend_all.restype = None
        l.orcB_attend_all.argtypes = [_u16p, _u16p, _f32p, C.c_int, C.c_int, C.c_float, _u16p,
                                      C.c_int, C.c_int, C.c_double, _f64p]
        l.orcB_density.restype = None
        l.orc_gate_log_bias.argtypes = [C.c_float, C.c_double, C.c_float]
        l.orc_gate_log_bias.restype = C.c_double
        l.orcB_attend_row_soft.argtypes = [_u16p, _u16p, _f32p, C.c_int, C.c_int, C.c_int, C.c_double, C.c_float,
                                           _u16p, C.c_int, C.c_int, C.c_double, _f64p, C.c_void_p]
        l.orcB_attend_row_soft.restype = None
        l.orcB_attend_all_soft.argtypes = [_u16p, _u16p, _f32p, C.c_int, C.c_int, C.c_double, C.c_float, _u16p,
                                           C.c_int, C.c_int, C.c_double, _f64p, C.c_void_p]
        l.orcB_attend_all_soft.restype = None
        l.orcB_density.argtypes = [_f32p, C.c_int, C.c_int, C.c_float, C.POINTER(C.c_double),
                                   C.POINTER(C.c_double)]
        l.orcA_new.restype = C.c_void_p
        l.orcA_new.argtypes = [C.c_int, C.c_int]
        l.orcA_free.restype = None
        l.orcA_free.argtypes = [C.c_void_p]
        l.orcA_append.restype = None
        l.orcA_append.argtypes = [C.c_void_p, _u16p, _u16p, C.c_float, C.c_float]
        l.orcA_attend.restype = None
        l.orcA_attend.argtypes = [C.c_void_p, _u16p, C.c_int, C.c_double, _f64p, C.c_void_p]
        l.orcA_prefill.restype = None
        l.orcA_prefill.argtypes = [C.c_void_p, C.c_int, _u16p, _u16p, _f32p, C.c_float,
                                   C.c_void_p, C.c_int, C.c_double, C.c_void_p]
        l.orcA_t.restype = C.c_long
        l.orcA_t.argtypes = [C.c_void_p]
        l.orcA_len.restype = C.c_long
        l.orcA_len.argtypes = [C.c_void_p]
        l.orcA_get_kept.restype = None
        l.orcA_get_kept.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.orcA_get_window.restype = None
        l.orcA_get_window.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.orcA_step_batch.restype = None
        l.orcA_step_batch.argtypes = [C.c_void_p, C.c_int, _u16p, _u16p, _f32p, C.c_float, _u16p,
                                      C.c_int, C.c_double, _f64p]
        l.orcA_prefill_batch.restype = None
        l.orcA_prefill_batch.argtypes = [C.c_void_p, C.c_int, C.c_int, _u16p, _u16p, _f32p,
                                         C.c_float]
        l.orc_threads.restype = C.c_int
        l.orc_threads.argtypes = []
        _lib = l
    return _lib


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def threads() -> int:
    return int(lib().orc_threads())


def sigmoid(z: float) -> float:
    return float(lib().orc_sigmoid(float(z)))


def tau_logit(tau: float) -> np.float32:
    return np.float32(lib().orc_tau_logit(float(tau)))


def bf16_to_double(bits) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    l = lib()
    return np.array([l.orc_bf16_to_double(int(b)) for b in bits.ravel()]).reshape(bits.shape)


def score_linear(x, W, b) -> np.ndarray:
    """Eq. 1 logits, linear predictor: x [n,d] bf16 bits, W [H,d] bf16 bits, b [H] f32."""
    x, W, b = _u16(x), _u16(W), _f32(b)
    n, d = x.shape
    H = W.shape[0]
    out = np.empty((n, H), np.float64)
    lib().orc_score_linear(x, n, d, W, b, H, out)
    return out


def score_mlp(x, W1, b1, W2, b2) -> np.ndarray:
    """Eq. 1 logits, two-layer perceptron with SiLU (the paper's listing)."""
    x, W1, W2, b1, b2 = _u16(x), _u16(W1), _u16(W2), _f32(b1), _f32(b2)
    n, d = x.shape
    hidden, H = W1.shape[0], W2.shape[0]
    out = np.empty((n, H), np.float64)
    lib().orc_score_mlp(x, n, d, W1, b1, hidden, W2, b2, H, out)
    return out


def mask_attend_row(K, V, logit, t, w, tau_l, q, scale, want_lse=False, n_sink=0):
    """Mask form (Eq. 2-5), one query position t.  K,V [T,D]; q [G,D] -> [G,D].
    n_sink > 0: the sink-token variant (first n_sink positions always retained)."""
    K, V, q, logit = _u16(K), _u16(V), _u16(q), _f32(logit)
    T, D = K.shape
    G = q.shape[0]
    out = np.empty((G, D), np.float64)
    lse = np.empty(G, np.float64)
    lib().orcB_attend_row_sinks(K, V, logit, T, int(t), int(w), float(tau_l), int(n_sink), q, G, D,
                                float(scale), out, lse.ctypes.data)
    return (out, lse) if want_lse else out


def mask_attend_all(K, V, logit, w, tau_l, q, scale, n_sink=0):
    """Mask form for every position.  q [T,G,D] -> [T,G,D] (O(T^2))."""
    K, V, q, logit = _u16(K), _u16(V), _u16(q), _f32(logit)
    T, D = K.shape
    G = q.shape[1]
    out = np.empty((T, G, D), np.float64)
    lib().orcB_attend_all_sinks(K, V, logit, T, int(w), float(tau_l), int(n_sink), q, G, D,
                                float(scale), out)
    return out


def gate_log_bias(logit, alpha=0.0, tau_l=0.0) -> float:
    """log of the (annealed) gate of one position: Eq. 6 with the gate of Eq. 7."""
    return float(lib().orc_gate_log_bias(float(np.float32(logit)), float(alpha), float(tau_l)))


def soft_attend_row(K, V, logit, t, w, q, scale, alpha=0.0, tau_l=0.0, want_lse=False):
    """Soft-gated forward (Eq. 6; alpha > 0: the annealed gate of Eq. 7), one query position t.
    K,V [T,D]; q [G,D] -> [G,D]."""
    K, V, q, logit = _u16(K), _u16(V), _u16(q), _f32(logit)
    T, D = K.shape
    G = q.shape[0]
    out = np.empty((G, D), np.float64)
    lse = np.empty(G, np.float64)
    lib().orcB_attend_row_soft(K, V, logit, T, int(t), int(w), float(alpha), float(tau_l), q, G, D,
                               float(scale), out, lse.ctypes.data)
    return (out, lse) if want_lse else out


def soft_attend_all(K, V, logit, w, q, scale, alpha=0.0, tau_l=0.0, want_lse=False):
    """Soft-gated forward for every position.  q [T,G,D] -> [T,G,D] (O(T^2))."""
    K, V, q, logit = _u16(K), _u16(V), _u16(q), _f32(logit)
    T, D = K.shape
    G = q.shape[1]
    out = np.empty((T, G, D), np.float64)
    lse = np.empty((T, G), np.float64)
    lib().orcB_attend_all_soft(K, V, logit, T, int(w), float(alpha), float(tau_l), q, G, D, float(scale),
                               out, lse.ctypes.data)
    return (out, lse) if want_lse else out


def density(logit, w, tau_l):
    """Eq. 8 for one (layer, head): (mean of z over all T, kept / left-the-window)."""
    logit = _f32(logit)
    a, b = C.c_double(), C.c_double()
    lib().orcB_density(logit, logit.shape[0], int(w), float(tau_l), C.byref(a), C.byref(b))
    return a.value, b.value


class Unit:
    """Streaming form: ring of w pairs + append-only kept list, one (layer, seq, KV head)."""

    def __init__(self, w: int, D: int = 128, n_sink: int = 0):
        self.w, self.D, self.n_sink = int(w), int(D), int(n_sink)
        self._h = C.c_void_p(lib().orcA_new(self.w, self.D))
        if self.n_sink:
            lib().orcA_set_sinks(self._h, self.n_sink)

    def __del__(self):
        try:
            if self._h:
                lib().orcA_free(self._h)
                self._h = None
        except Exception:
            pass

    @property
    def t(self) -> int:
        return int(lib().orcA_t(self._h))

    def __len__(self) -> int:
        return int(lib().orcA_len(self._h))

    def append(self, k, v, logit, tau_l):
        lib().orcA_append(self._h, _u16(k).reshape(-1), _u16(v).reshape(-1), float(logit),
                          float(tau_l))

    def attend(self, q, scale, want_lse=False):
        q = _u16(q)
        G = q.shape[0]
        out = np.empty((G, self.D), np.float64)
        lse = np.empty(G, np.float64)
        lib().orcA_attend(self._h, q, G, float(scale), out, lse.ctypes.data)
        return (out, lse) if want_lse else out

    def prefill(self, k, v, logit, tau_l, q=None, scale=0.0):
        """C x (append, attend); returns [C,G,D] outputs when q is given."""
        k, v, logit = _u16(k), _u16(v), _f32(logit)
        Cn = k.shape[0]
        if q is None:
            lib().orcA_prefill(self._h, Cn, k, v, logit, float(tau_l), None, 0, 0.0, None)
            return None
        q = _u16(q)
        G = q.shape[1]
        out = np.empty((Cn, G, self.D), np.float64)
        lib().orcA_prefill(self._h, Cn, k, v, logit, float(tau_l), q.ctypes.data, G, float(scale),
                           out.ctypes.data)
        return out

    def kept(self):
        n = len(self)
        pos = np.empty(n, np.int32)
        k = np.empty((n, self.D), np.uint16)
        v = np.empty((n, self.D), np.uint16)
        lib().orcA_get_kept(self._h, pos.ctypes.data, k.ctypes.data, v.ctypes.data)
        return pos, k, v

    def window(self):
        n = min(self.t, self.w)
        pos = np.empty(n, np.int32)
        k = np.empty((n, self.D), np.uint16)
        v = np.empty((n, self.D), np.uint16)
        lg = np.empty(n, np.float32)
        lib().orcA_get_window(self._h, pos.ctypes.data, k.ctypes.data, v.ctypes.data,
                              lg.ctypes.data)
        return pos, k, v, lg


def _handles(units):
    arr = (C.c_void_p * len(units))(*[u._h for u in units])
    return arr


def step_batch(units, k, v, logit, tau_l, q, scale):
    """One decode step (append, attend) on many units; k,v [n,D], logit [n], q [n,G,D]."""
    k, v, q, logit = _u16(k), _u16(v), _u16(q), _f32(logit)
    n, G, D = q.shape
    out = np.empty((n, G, D), np.float64)
    lib().orcA_step_batch(_handles(units), n, k, v, logit, float(tau_l), q, G, float(scale), out)
    return out


def prefill_batch(units, k, v, logit, tau_l):
    """State build: unit i receives k[i], v[i] ([C,D]) and logit[i] ([C])."""
    k, v, logit = _u16(k), _u16(v), _f32(logit)
    n, Cn, _ = k.shape
    lib().orcA_prefill_batch(_handles(units), n, Cn, k, v, logit, float(tau_l))
