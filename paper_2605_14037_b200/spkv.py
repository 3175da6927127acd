"""ctypes binding of libspkv.so: the same entry points as include/spkv.h.

Argument marshalling only -- every step of the path runs in the CUDA kernels of the
library.  PyTorch supplies device memory and streams.  There is no CPU fallback: if
the library cannot be loaded, importing this module raises.

Low level: ``lib()`` returns the ctypes handle with prototypes set; the ``spkv_*``
functions below mirror the C names and accept torch tensors.
High level: ``Cache`` owns an arena tensor and workspaces and forwards to them.
"""
from __future__ import annotations

import ctypes as C
import math
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libspkv.so")

SPKV_OK = 0
ERRORS = {
    -1: "SPKV_E_INVALID", -2: "SPKV_E_ARENA_TOO_SMALL", -3: "SPKV_E_UNSUPPORTED", -4: "SPKV_E_CUDA",
    -5: "SPKV_E_POOL_EXHAUSTED", -6: "SPKV_E_CONTEXT_OVERFLOW", -7: "SPKV_E_WORKSPACE",
    -8: "SPKV_E_TIMEOUT", -9: "SPKV_E_BOUNDS", -10: "SPKV_E_SCRATCH_LIMIT", -11: "SPKV_E_ORDER_DECODE",
    -12: "SPKV_E_ORDER_APPEND", -13: "SPKV_E_BOUNDS_PAGE", -14: "SPKV_E_CANARY", -15: "SPKV_E_ATTACH",
}


FLAG_OVERLAP = 1          # SPKV_FLAG_OVERLAP
FLAG_PREFILL_PV_BF16 = 2  # SPKV_FLAG_PREFILL_PV_BF16
FLAG_DEBUG_BOUNDS = 4      # SPKV_FLAG_DEBUG_BOUNDS


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("max_seqs", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("window", C.c_int32),
                ("page_tokens", C.c_int32), ("max_context", C.c_int32), ("pool_pages", C.c_int64),
                ("tau", C.c_float), ("flags", C.c_int32), ("sink_tokens", C.c_int32),
                ("h_local_only", C.c_void_p)]


class Predictor(C.Structure):
    _fields_ = [("kind", C.c_int32), ("d_in", C.c_int32), ("hidden", C.c_int32),
                ("reserved", C.c_int32), ("d_W1", C.c_void_p), ("d_b1", C.c_void_p),
                ("d_W2", C.c_void_p), ("d_b2", C.c_void_p)]


class Stats(C.Structure):
    _fields_ = [("units", C.c_int64), ("pairs_seen", C.c_int64), ("pairs_kept", C.c_int64),
                ("pairs_in_window", C.c_int64), ("pairs_evicted", C.c_int64),
                ("gates_open", C.c_int64), ("pages_in_use", C.c_int64), ("pages_free", C.c_int64),
                ("bytes_resident", C.c_int64), ("density_all", C.c_double),
                ("density_cache", C.c_double)]


class SpkvError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {ERRORS.get(code, code)} ({lib().spkv_error_string(code).decode()})")


_lib = None


def lib():
    """Loads libspkv.so (fails loudly when it is missing) and declares prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} not found: build it with "
                          "`python -m paper_2605_14037_b200.build` (there is no fallback path)")
    l = C.CDLL(_LIB_PATH)
    vp, i32, sz, f32 = C.c_void_p, C.c_int32, C.c_size_t, C.c_float
    cfgp, pp = C.POINTER(Config), C.POINTER(Predictor)
    protos = {
        "spkv_arena_bytes": (C.c_int, [cfgp, C.POINTER(sz)]),
        "spkv_cache_create": (C.c_int, [cfgp, vp, sz, vp, C.POINTER(vp)]),
        "spkv_cache_attach": (C.c_int, [cfgp, vp, sz, vp, C.POINTER(vp)]),
        "spkv_cache_checkpoint_bytes": (sz, [vp]),
        "spkv_cache_checkpoint": (C.c_int, [vp, vp, sz, vp]),
        "spkv_cache_rollback": (C.c_int, [vp, vp, sz, vp]),
        "spkv_note_foreign_work": (C.c_int, [vp]),
        "spkv_safe_steps": (C.c_int, [vp, vp, i32, vp, C.POINTER(C.c_int64)]),
        "spkv_safe_steps_from_lengths": (C.c_int, [cfgp, vp, vp, C.c_int64, C.c_int64, C.POINTER(C.c_int64)]),
        "spkv_arena_canaries": (C.c_int, [cfgp, C.POINTER(sz), i32, C.POINTER(i32)]),
        "spkv_cache_destroy": (C.c_int, [vp]),
        "spkv_cache_reset_seq": (C.c_int, [vp, i32, vp]),
        "spkv_set_tau": (C.c_int, [vp, f32]),
        "spkv_set_head_tau": (C.c_int, [vp, i32, i32, f32, vp]),
        "spkv_score": (C.c_int, [vp, pp, vp, i32, vp, vp, vp]),
        "spkv_append_evict": (C.c_int, [vp, i32, vp, i32, vp, vp, vp, vp]),
        "spkv_score_append_evict": (C.c_int, [vp, i32, pp, vp, i32, vp, vp, vp, vp, vp]),
        "spkv_decode_workspace_bytes": (sz, [cfgp, i32]),
        "spkv_decode_attention": (C.c_int, [vp, i32, vp, i32, vp, vp, vp, f32, vp, sz, vp]),
        "spkv_stream_read": (C.c_int, [vp, sz, vp, vp, vp]),
        "spkv_wait_selftest": (C.c_int, [vp, C.c_longlong, vp, vp]),
        "spkv_decode_attention_f32": (C.c_int, [vp, i32, vp, i32, vp, vp, vp, vp, f32, vp, sz, vp]),
        "spkv_decode_attention_static": (C.c_int, [vp, i32, vp, i32, vp, vp, vp, f32, vp]),
        "spkv_prefill_workspace_bytes": (sz, [cfgp, i32]),
        "spkv_prefill": (C.c_int, [vp, i32, i32, i32, vp, vp, vp, vp, vp, f32, vp, sz, vp]),
        "spkv_softgate_workspace_bytes": (sz, [i32, i32, i32]),
        "spkv_softgate_forward": (C.c_int, [i32, i32, i32, i32, vp, vp, vp, vp, f32, f32, f32, i32, vp, vp, vp, sz,
                                            vp, vp]),
        "spkv_decode_step_staging_bytes": (sz, [cfgp, i32, i32]),
        "spkv_decode_step_host": (C.c_int, [vp, i32, pp, vp, i32, vp, vp, vp, vp, vp, f32, vp, sz, vp]),
        "spkv_decode_step_host_flush": (C.c_int, [vp, vp]),
        "spkv_decode_stack_staging_bytes": (sz, [cfgp, i32, i32]),
        "spkv_decode_stack_host": (C.c_int, [vp, vp, vp, i32, vp, vp, vp, vp, vp, f32, vp, sz, vp]),
        "spkv_decode_stack_workspace_bytes": (sz, [cfgp, i32]),
        "spkv_decode_stack": (C.c_int, [vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, f32, vp, sz, vp]),
        "spkv_status": (C.c_int, [vp, vp]),
        "spkv_clear_status": (C.c_int, [vp, vp]),
        "spkv_cache_stats": (C.c_int, [vp, vp, C.POINTER(Stats)]),
        "spkv_read_lengths": (C.c_int, [vp, i32, vp, vp, vp]),
        "spkv_read_kept": (C.c_int, [vp, i32, i32, i32, vp, vp, vp, i32, C.POINTER(i32), vp]),
        "spkv_read_window": (C.c_int, [vp, i32, i32, i32, vp, vp, vp, vp, C.POINTER(i32), vp]),
        "spkv_tau_logit": (f32, [vp]),
        "spkv_error_string": (C.c_char_p, [C.c_int]),
    }
    for name, (res, args) in protos.items():
        fn = getattr(l, name)
        fn.restype, fn.argtypes = res, args
    _lib = l
    return l


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _ptr(t, dtype=None):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensor, contiguous"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return C.c_void_p(t.data_ptr())


def _check(rc, where):
    if rc != SPKV_OK:
        raise SpkvError(rc, where)


def make_predictor(W1, b1, W2=None, b2=None) -> Predictor:
    """Linear predictor (W1 [Hkv,d_in], b1 [Hkv]) or two-layer perceptron
    (W1 [hidden,d_in], b1 [hidden], W2 [Hkv,hidden], b2 [Hkv]); bf16 weights, f32 biases."""
    p = Predictor()
    p.kind = 0 if W2 is None else 1
    p.d_in = W1.shape[1]
    p.hidden = 0 if W2 is None else W1.shape[0]
    p.d_W1, p.d_b1 = _ptr(W1, torch.bfloat16), _ptr(b1, torch.float32)
    p.d_W2 = _ptr(W2, torch.bfloat16) if W2 is not None else None
    p.d_b2 = _ptr(b2, torch.float32) if b2 is not None else None
    p._keep = (W1, b1, W2, b2)
    return p


class Cache:
    """An SP-KV cache inside one torch-owned arena tensor, plus the workspaces the
    attention calls need.  Methods carry the names of the C entry points."""

    def __init__(self, n_layers, max_seqs, n_q_heads, n_kv_heads, max_context, pool_pages,
                 window=128, tau=0.5, device="cuda:0", head_dim=128, page_tokens=64, sink_tokens=0,
                 flags=0, local_only=None):
        """local_only: optional [n_layers, n_kv_heads] array, non-zero = that head is declared
        local-only (window attention, no page table, not scored by the fused append)."""
        import numpy as np
        self._local_only = None
        if local_only is not None:
            self._local_only = np.ascontiguousarray(np.asarray(local_only) != 0, dtype=np.uint8)
            assert self._local_only.shape == (n_layers, n_kv_heads)
        self.cfg = Config(n_layers, max_seqs, n_q_heads, n_kv_heads, head_dim, window, page_tokens,
                          max_context, pool_pages, tau, flags, sink_tokens,
                          self._local_only.ctypes.data if self._local_only is not None else None)
        self.device = torch.device(device)
        n = C.c_size_t()
        _check(lib().spkv_arena_bytes(C.byref(self.cfg), C.byref(n)), "spkv_arena_bytes")
        self.arena_bytes = n.value
        with torch.cuda.device(self.device):
            self.arena = torch.empty(self.arena_bytes, dtype=torch.uint8, device=self.device)
            h = C.c_void_p()
            _check(lib().spkv_cache_create(C.byref(self.cfg), _ptr(self.arena), self.arena_bytes,
                                           _stream(), C.byref(h)), "spkv_cache_create")
        self._h = h
        self._ws = {}
        self.G = n_q_heads // n_kv_heads
        self.default_scale = 1.0 / math.sqrt(head_dim)

    @classmethod
    def attach(cls, arena, cfg, tau=None, flags=None, local_only=None):
        """A Cache over an arena tensor that already holds one (a copy of another cache's arena):
        spkv_cache_attach.  `cfg` is the Config the arena was created with; tau / flags override;
        local_only as at creation (it is part of the layout and has to be given again)."""
        import numpy as np
        self = cls.__new__(cls)
        self.cfg = Config.from_buffer_copy(cfg)
        self._local_only = None
        if local_only is not None:
            self._local_only = np.ascontiguousarray(np.asarray(local_only) != 0, dtype=np.uint8)
            assert self._local_only.shape == (cfg.n_layers, cfg.n_kv_heads)
        self.cfg.h_local_only = self._local_only.ctypes.data if self._local_only is not None else None
        if tau is not None:
            self.cfg.tau = tau
        if flags is not None:
            self.cfg.flags = flags
        self.device = arena.device
        self.arena, self.arena_bytes = arena, arena.numel()
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib().spkv_cache_attach(C.byref(self.cfg), _ptr(arena), arena.numel(), _stream(), C.byref(h)),
                   "spkv_cache_attach")
        self._h, self._ws = h, {}
        self.G = self.cfg.n_q_heads // self.cfg.n_kv_heads
        self.default_scale = 1.0 / math.sqrt(self.cfg.head_dim)
        return self

    def spkv_cache_checkpoint(self, buf=None, stream=None):
        """Saves metadata + ring pages into `buf` (allocated when None); returns the buffer."""
        n = lib().spkv_cache_checkpoint_bytes(self._h)
        if buf is None:
            buf = torch.empty(n, dtype=torch.uint8, device=self.device)
        _check(lib().spkv_cache_checkpoint(self._h, _ptr(buf), buf.numel(), _stream(stream)), "spkv_cache_checkpoint")
        return buf

    def spkv_cache_rollback(self, buf, stream=None):
        _check(lib().spkv_cache_rollback(self._h, _ptr(buf), buf.numel(), _stream(stream)), "spkv_cache_rollback")

    def spkv_note_foreign_work(self):
        _check(lib().spkv_note_foreign_work(self._h), "spkv_note_foreign_work")

    def spkv_safe_steps(self, seq_ids=None, stream=None) -> int:
        """Decode steps the listed sequences (host ints; None = all) can take before the pool or a
        page table could run out, every evicted pair assumed kept."""
        import numpy as np
        ids = np.ascontiguousarray(np.asarray([] if seq_ids is None else seq_ids, dtype=np.int32))
        out = C.c_int64()
        _check(lib().spkv_safe_steps(self._h, ids.ctypes.data if ids.size else None, int(ids.size),
                                     _stream(stream), C.byref(out)), "spkv_safe_steps")
        return int(out.value)

    def close(self):
        if getattr(self, "_h", None):
            lib().spkv_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- workspaces (zero-filled once, as the C interface asks) -----------------------
    def _workspace(self, kind, nbytes):
        ws = self._ws.get(kind)
        if ws is None or ws.numel() < nbytes:
            ws = torch.zeros(max(nbytes, 256), dtype=torch.uint8, device=self.device)
            self._ws[kind] = ws
        return ws

    def decode_workspace(self, B):
        return self._workspace("decode", lib().spkv_decode_workspace_bytes(C.byref(self.cfg), B))

    # -- hot path -----------------------------------------------------------------------
    def spkv_score(self, pred, x, logits=None, flags=None, stream=None):
        n_tok = x.shape[0]
        if logits is None:
            logits = torch.empty((n_tok, self.cfg.n_kv_heads), dtype=torch.float32, device=x.device)
        _check(lib().spkv_score(self._h, C.byref(pred), _ptr(x, torch.bfloat16), n_tok,
                                _ptr(logits, torch.float32), _ptr(flags, torch.uint8),
                                _stream(stream)), "spkv_score")
        return logits

    def spkv_append_evict(self, layer, seq_ids, k, v, logits, stream=None):
        _check(lib().spkv_append_evict(self._h, layer, _ptr(seq_ids, torch.int32), seq_ids.numel(),
                                       _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16),
                                       _ptr(logits, torch.float32), _stream(stream)),
               "spkv_append_evict")

    def spkv_score_append_evict(self, layer, pred, seq_ids, x, k, v, logits_out=None, stream=None):
        _check(lib().spkv_score_append_evict(
            self._h, layer, C.byref(pred), _ptr(seq_ids, torch.int32), seq_ids.numel(),
            _ptr(x, torch.bfloat16), _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16),
            _ptr(logits_out, torch.float32), _stream(stream)), "spkv_score_append_evict")

    def spkv_decode_attention(self, layer, seq_ids, q, out=None, lse=None, sm_scale=None,
                              stream=None):
        B = seq_ids.numel()
        if out is None:
            out = torch.empty_like(q)
        ws = self.decode_workspace(B)
        _check(lib().spkv_decode_attention(
            self._h, layer, _ptr(seq_ids, torch.int32), B, _ptr(q, torch.bfloat16),
            _ptr(out, torch.bfloat16), _ptr(lse, torch.float32),
            self.default_scale if sm_scale is None else sm_scale, _ptr(ws), ws.numel(),
            _stream(stream)), "spkv_decode_attention")
        return out

    def spkv_decode_attention_f32(self, layer, seq_ids, q, out=None, out_f32=None, lse=None, sm_scale=None,
                                  stream=None):
        """spkv_decode_attention that also returns the rows before their rounding to bf16;
        returns (out bf16, out float32)."""
        B = seq_ids.numel()
        if out is None:
            out = torch.empty_like(q)
        if out_f32 is None:
            out_f32 = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        ws = self.decode_workspace(B)
        _check(lib().spkv_decode_attention_f32(
            self._h, layer, _ptr(seq_ids, torch.int32), B, _ptr(q, torch.bfloat16),
            _ptr(out, torch.bfloat16), _ptr(out_f32, torch.float32), _ptr(lse, torch.float32),
            self.default_scale if sm_scale is None else sm_scale, _ptr(ws), ws.numel(),
            _stream(stream)), "spkv_decode_attention_f32")
        return out, out_f32

    def spkv_decode_attention_static(self, layer, seq_ids, q, out=None, lse=None, sm_scale=None,
                                     stream=None):
        """Same result as spkv_decode_attention, for callers that may not allocate device
        memory: the scratch is a fixed array inside the library (no workspace tensor)."""
        B = seq_ids.numel()
        if out is None:
            out = torch.empty_like(q)
        _check(lib().spkv_decode_attention_static(
            self._h, layer, _ptr(seq_ids, torch.int32), B, _ptr(q, torch.bfloat16),
            _ptr(out, torch.bfloat16), _ptr(lse, torch.float32),
            self.default_scale if sm_scale is None else sm_scale, _stream(stream)),
            "spkv_decode_attention_static")
        return out

    def spkv_prefill(self, layer, seq, k, v, logits, q=None, out=None, sm_scale=None, stream=None):
        Cn = k.shape[0]
        if q is not None and out is None:
            out = torch.empty_like(q)
        ws = self._workspace("prefill", lib().spkv_prefill_workspace_bytes(C.byref(self.cfg), Cn))
        _check(lib().spkv_prefill(
            self._h, layer, seq, Cn, _ptr(q, torch.bfloat16), _ptr(k, torch.bfloat16),
            _ptr(v, torch.bfloat16), _ptr(logits, torch.float32), _ptr(out, torch.bfloat16),
            self.default_scale if sm_scale is None else sm_scale, _ptr(ws), ws.numel(),
            _stream(stream)), "spkv_prefill")
        return out

    def spkv_decode_step_host(self, layer, pred, seq_ids, h_x, h_q, h_k, h_v, h_out, sm_scale=None,
                              stream=None):
        """Host (pinned) tensors in, host tensor out; enqueues the copies (on the cache's own
        copy streams) and the kernels.  h_out is complete after spkv_decode_step_host_flush()
        and a synchronisation of the stream."""
        B = seq_ids.numel()
        nbytes = lib().spkv_decode_step_staging_bytes(C.byref(self.cfg), B, pred.d_in)
        old = self._ws.get("staging")
        if old is not None and old.numel() < nbytes:   # growing: drain the pipeline that uses the old one
            self.spkv_decode_step_host_flush(stream)
            torch.cuda.synchronize(self.device)
        st = self._workspace("staging", nbytes)
        for t in (h_x, h_q, h_k, h_v, h_out):
            assert not t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16
        _check(lib().spkv_decode_step_host(
            self._h, layer, C.byref(pred), _ptr(seq_ids, torch.int32), B,
            C.c_void_p(h_x.data_ptr()), C.c_void_p(h_q.data_ptr()), C.c_void_p(h_k.data_ptr()),
            C.c_void_p(h_v.data_ptr()), C.c_void_p(h_out.data_ptr()),
            self.default_scale if sm_scale is None else sm_scale, _ptr(st), st.numel(),
            _stream(stream)), "spkv_decode_step_host")

    def spkv_decode_stack(self, preds, seq_ids, x, q, k, v, out=None, logits_out=None, lse=None, sm_scale=None,
                          stream=None):
        """One decode step of all layers from device tensors [L, B, ...]: the appends of every layer in
        one launch, decode attention of every layer in one persistent launch."""
        B, L = seq_ids.numel(), self.cfg.n_layers
        assert len(preds) == L and q.shape[0] == L
        arr = (Predictor * L)(*preds)
        if out is None:
            out = torch.empty_like(q)
        ws = self._workspace("decode_stack", lib().spkv_decode_stack_workspace_bytes(C.byref(self.cfg), B))
        _check(lib().spkv_decode_stack(
            self._h, C.cast(arr, C.c_void_p), _ptr(seq_ids, torch.int32), B, _ptr(x, torch.bfloat16),
            _ptr(q, torch.bfloat16), _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16), _ptr(out, torch.bfloat16),
            _ptr(logits_out, torch.float32), _ptr(lse, torch.float32),
            self.default_scale if sm_scale is None else sm_scale, _ptr(ws), ws.numel(), _stream(stream)),
            "spkv_decode_stack")
        return out

    def spkv_decode_stack_host(self, preds, seq_ids, h_x, h_q, h_k, h_v, h_out, sm_scale=None, stream=None):
        """One decode step of all layers from host (pinned) tensors [L, B, ...]; enqueues four
        copies in, the 2 L kernels and one copy out on the stream."""
        B, L = seq_ids.numel(), self.cfg.n_layers
        assert len(preds) == L
        arr = (Predictor * L)(*preds)
        nbytes = lib().spkv_decode_stack_staging_bytes(C.byref(self.cfg), B, preds[0].d_in)
        st = self._workspace("stack_staging", nbytes)
        for t in (h_x, h_q, h_k, h_v, h_out):
            assert not t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16 and t.shape[0] == L
        _check(lib().spkv_decode_stack_host(
            self._h, C.cast(arr, C.c_void_p), _ptr(seq_ids, torch.int32), B,
            C.c_void_p(h_x.data_ptr()), C.c_void_p(h_q.data_ptr()), C.c_void_p(h_k.data_ptr()),
            C.c_void_p(h_v.data_ptr()), C.c_void_p(h_out.data_ptr()),
            self.default_scale if sm_scale is None else sm_scale, _ptr(st), st.numel(),
            _stream(stream)), "spkv_decode_stack_host")

    def spkv_decode_step_host_flush(self, stream=None):
        """Makes the stream wait for the output copy of the last spkv_decode_step_host call."""
        _check(lib().spkv_decode_step_host_flush(self._h, _stream(stream)), "spkv_decode_step_host_flush")

    # -- maintenance / introspection ---------------------------------------------------
    def spkv_cache_reset_seq(self, seq, stream=None):
        _check(lib().spkv_cache_reset_seq(self._h, seq, _stream(stream)), "spkv_cache_reset_seq")

    def spkv_set_tau(self, tau):
        _check(lib().spkv_set_tau(self._h, tau), "spkv_set_tau")

    def spkv_set_head_tau(self, layer, kv_head, tau, stream=None):
        """Threshold of one (layer, KV head) (kv_head = -1: the whole layer); NaN clears it."""
        _check(lib().spkv_set_head_tau(self._h, layer, kv_head, tau, _stream(stream)), "spkv_set_head_tau")

    def spkv_tau_logit(self) -> float:
        return float(lib().spkv_tau_logit(self._h))

    def spkv_status(self, stream=None) -> int:
        return int(lib().spkv_status(self._h, _stream(stream)))

    def spkv_clear_status(self, stream=None):
        _check(lib().spkv_clear_status(self._h, _stream(stream)), "spkv_clear_status")

    def check(self):
        _check(self.spkv_status(), "device status")

    def spkv_cache_stats(self, stream=None) -> Stats:
        s = Stats()
        _check(lib().spkv_cache_stats(self._h, _stream(stream), C.byref(s)), "spkv_cache_stats")
        return s

    def spkv_read_lengths(self, layer, stream=None):
        import numpy as np
        shape = (self.cfg.max_seqs, self.cfg.n_kv_heads)
        ln, t = np.empty(shape, np.int32), np.empty(shape, np.int32)
        _check(lib().spkv_read_lengths(self._h, layer, ln.ctypes.data, t.ctypes.data,
                                       _stream(stream)), "spkv_read_lengths")
        return ln, t

    def spkv_read_kept(self, layer, seq, kvh, stream=None):
        """(positions int32 [n], K bits uint16 [n,128], V bits uint16 [n,128])"""
        import numpy as np
        n = C.c_int32()
        _check(lib().spkv_read_kept(self._h, layer, seq, kvh, None, None, None, 0, C.byref(n),
                                    _stream(stream)), "spkv_read_kept")
        cap = n.value
        pos = np.empty(cap, np.int32)
        k = np.empty((cap, 128), np.uint16)
        v = np.empty((cap, 128), np.uint16)
        _check(lib().spkv_read_kept(self._h, layer, seq, kvh, pos.ctypes.data, k.ctypes.data,
                                    v.ctypes.data, cap, C.byref(n), _stream(stream)),
               "spkv_read_kept")
        return pos, k, v

    def spkv_read_window(self, layer, seq, kvh, stream=None):
        """(positions [n], K bits [n,128], V bits [n,128], logits f32 [n]), ascending position"""
        import numpy as np
        w = self.cfg.window
        pos = np.empty(w, np.int32)
        k = np.empty((w, 128), np.uint16)
        v = np.empty((w, 128), np.uint16)
        lg = np.empty(w, np.float32)
        n = C.c_int32()
        _check(lib().spkv_read_window(self._h, layer, seq, kvh, pos.ctypes.data, k.ctypes.data,
                                      v.ctypes.data, lg.ctypes.data, C.byref(n), _stream(stream)),
               "spkv_read_window")
        n = n.value
        return pos[:n], k[:n], v[:n], lg[:n]


def spkv_stream_read(buf, passes=5, stream=None):
    """Read-only HBM rate in GB/s: streams the uint8 tensor `buf` through spkv_stream_read
    `passes` times (after one warm-up pass), timed with CUDA events on the launching stream."""
    sink = torch.zeros(2, dtype=torch.int64, device=buf.device)   # checksum, page counter
    status = torch.zeros(1, dtype=torch.int32, device=buf.device)
    nbytes = buf.numel() // 32768 * 32768
    call = lambda: _check(lib().spkv_stream_read(_ptr(buf), nbytes, _ptr(sink), _ptr(status), _stream(stream)),
                          "spkv_stream_read")
    call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(passes):
        call()
    e1.record()
    e1.synchronize()
    if int(status.item()) != 0:
        raise SpkvError(int(status.item()), "spkv_stream_read")
    return nbytes * passes / (e0.elapsed_time(e1) * 1e-3) / 1e9


_softgate_ws = {}


def spkv_softgate_forward(q, k, v, logits, window=128, alpha=0.0, tau=0.5, sm_scale=None, flags=0, out=None,
                          want_lse=False, stream=None, status=None):
    """Soft-gated whole-sequence forward (Eq. 6 / Eq. 7; see spkv.h).  q [T,Hq,128], k, v [T,Hkv,128]
    bf16, logits [T,Hkv] float32 on one device -> out [T,Hq,128] bf16 (and lse [T,Hq] float32).
    status: an int32 device tensor of one zero that receives the device-side verdict; when given,
    the call does not synchronise and the caller reads it; otherwise the call waits and raises."""
    T, Hq, Hkv = q.shape[0], q.shape[1], k.shape[1]
    if out is None:
        out = torch.empty_like(q)
    lse = torch.empty((T, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    nbytes = lib().spkv_softgate_workspace_bytes(T, Hq, Hkv)
    ws = _softgate_ws.get(q.device)
    if ws is None or ws.numel() < nbytes:
        ws = _softgate_ws[q.device] = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
    own_status = status is None
    if own_status:
        status = torch.zeros(1, dtype=torch.int32, device=q.device)
    _check(lib().spkv_softgate_forward(
        T, Hq, Hkv, window, _ptr(q, torch.bfloat16), _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16),
        _ptr(logits, torch.float32), alpha, tau, 1.0 / math.sqrt(q.shape[2]) if sm_scale is None else sm_scale,
        flags, _ptr(out, torch.bfloat16), _ptr(lse), _ptr(ws), ws.numel(), _ptr(status), _stream(stream)),
        "spkv_softgate_forward")
    if own_status:
        code = int(status.item())      # synchronises: the status word is the call's device-side verdict
        if code != 0:
            raise SpkvError(code, "spkv_softgate_forward (device)")
    return (out, lse) if want_lse else out


def spkv_wait_selftest(buf, limit_clocks, stream=None):
    """Runs the library's bounded-wait error path once (see spkv.h); returns the four status
    words [code, drained, clocks waited, data in place] as a list."""
    status = torch.zeros(4, dtype=torch.int32, device=buf.device)
    _check(lib().spkv_wait_selftest(_ptr(buf), int(limit_clocks), _ptr(status), _stream(stream)),
           "spkv_wait_selftest")
    return status.cpu().tolist()


def bf16_from_bits(bits, device):
    """numpy uint16 bit patterns -> torch.bfloat16 tensor on `device` (same bits)."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.view(torch.bfloat16).to(device)


def bits_from_bf16(t):
    """torch.bfloat16 tensor -> numpy uint16 bit patterns."""
    import numpy as np
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
