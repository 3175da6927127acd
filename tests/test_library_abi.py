"""The C-ABI library loads without a GPU and exports every symbol the header declares;
host-only entry points (layout sizing, validation, error strings) behave."""
import ctypes as C
import os
import re

import pytest

from paper_2605_14037_b200 import build as spkv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def spkv():
    spkv_build.build()
    from paper_2605_14037_b200 import spkv as mod
    mod.lib()
    return mod


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "spkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spkv_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(spkv):
    names = declared_symbols()
    assert len(names) >= 20 and "spkv_prefill" in names and "spkv_decode_attention" in names
    for name in names:
        assert hasattr(spkv.lib(), name), name


def test_binding_declares_every_symbol(spkv):
    l = spkv.lib()
    for name in declared_symbols():
        assert getattr(l, name).argtypes is not None, name


def cfg(spkv, **kw):
    base = dict(n_layers=2, max_seqs=3, n_q_heads=8, n_kv_heads=2, head_dim=128, window=128,
                page_tokens=64, max_context=4096, pool_pages=100, tau=0.5, flags=0)
    base.update(kw)
    return spkv.Config(**base)


def test_arena_bytes_accounts_for_every_region(spkv):
    n = C.c_size_t()
    c = cfg(spkv)
    assert spkv.lib().spkv_arena_bytes(C.byref(c), C.byref(n)) == 0
    units = 2 * 3 * 2
    pages = (units * 2 + 100) * 32768
    meta = units * 4 * 2 + units * 64 * 4 + 100 * 4 + 100 * 64 * 4 + units * 128 * 4
    assert pages + meta <= n.value <= pages + meta + 16 * 1024
    # more pool pages cost exactly one page + its position row + its stack slot each
    c2 = cfg(spkv, pool_pages=100 + 64)
    n2 = C.c_size_t()
    assert spkv.lib().spkv_arena_bytes(C.byref(c2), C.byref(n2)) == 0
    assert abs((n2.value - n.value) - 64 * (32768 + 256 + 4)) <= 2048  # region alignment slack
    # window 1 still needs one ring page per unit; window 129 needs three
    for w, rp in ((1, 1), (64, 1), (65, 2), (129, 3)):
        cw, nw = cfg(spkv, window=w, pool_pages=0), C.c_size_t()
        assert spkv.lib().spkv_arena_bytes(C.byref(cw), C.byref(nw)) == 0
        assert nw.value >= units * rp * 32768
        assert nw.value < units * rp * 32768 + 64 * 1024


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=64), -3), (dict(page_tokens=16), -3), (dict(n_q_heads=7), -1),
    (dict(window=0), -1), (dict(n_layers=0), -1), (dict(pool_pages=-1), -1),
    (dict(n_q_heads=64, n_kv_heads=2), -3), (dict(tau=float("nan")), -1),
])
def test_config_validation(spkv, kw, code):
    n = C.c_size_t()
    c = cfg(spkv, **kw)
    assert spkv.lib().spkv_arena_bytes(C.byref(c), C.byref(n)) == code


def test_workspace_sizes_and_error_strings(spkv):
    c = cfg(spkv)
    l = spkv.lib()
    a, b = l.spkv_decode_workspace_bytes(C.byref(c), 1), l.spkv_decode_workspace_bytes(C.byref(c), 3)
    assert 0 < a < b
    assert l.spkv_decode_step_staging_bytes(C.byref(c), 3, 512) > b
    assert l.spkv_prefill_workspace_bytes(C.byref(c), 8192) > 0
    assert l.spkv_error_string(0) == b"ok"
    seen = {l.spkv_error_string(code) for code in range(-10, 1)}
    assert len(seen) == 11 and b"unknown error" not in seen
    assert l.spkv_error_string(-99) == b"unknown error"
    # null handles are rejected, not dereferenced
    assert l.spkv_cache_destroy(None) == -1
    assert l.spkv_set_tau(None, 0.5) == -1
    assert l.spkv_status(None, None) == -1
