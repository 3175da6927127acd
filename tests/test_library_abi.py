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
    # the stack step keeps arrival counters and partial results per layer (one half of a per-layer
    # workspace each), one counter word, and a per-layer workspace for its fallback path
    per_layer = (b // 2 + 255) // 256 * 256
    assert l.spkv_decode_stack_workspace_bytes(C.byref(c), 3) == 256 + c.n_layers * per_layer + b
    assert l.spkv_decode_stack_workspace_bytes(None, 3) == 0
    assert l.spkv_error_string(0) == b"ok"
    seen = {l.spkv_error_string(code) for code in range(-10, 1)}
    assert len(seen) == 11 and b"unknown error" not in seen
    assert l.spkv_error_string(-99) == b"unknown error"
    # null handles are rejected, not dereferenced
    assert l.spkv_cache_destroy(None) == -1
    assert l.spkv_set_tau(None, 0.5) == -1
    assert l.spkv_status(None, None) == -1


def brute_force_safe_steps(w, max_context, lens, ts, pages_free, cap=5000):
    """Steps n = 1, 2, ... with every evicted pair kept, page by page, until a unit would need a
    page the pool no longer has or its table has no room for."""
    lens, ts, free = list(lens), list(ts), pages_free
    max_pages = (max_context + 63) // 64
    for n in range(cap):
        for u in range(len(lens)):
            if ts[u] >= w:                      # the pair of position t - w leaves the window and is kept
                if lens[u] % 64 == 0:
                    if lens[u] // 64 >= max_pages or free == 0:
                        return n
                    free -= 1
                lens[u] += 1
            ts[u] += 1
    return cap


@pytest.mark.parametrize("seed", range(6))
def test_safe_step_budget_equals_a_page_by_page_simulation(spkv, seed):
    """The safe-step budget of the paper's inference appendix: the closed-form count the library
    uses against a literal simulation of the worst case."""
    import numpy as np
    rng = np.random.default_rng(seed)
    w = int(rng.choice([1, 16, 128, 200]))
    n_units = int(rng.integers(1, 12))
    ts = rng.integers(0, 3 * w + 5, size=n_units).astype(np.int32)
    lens = np.array([rng.integers(0, max(t - w, 0) + 1) for t in ts], dtype=np.int32)
    free = int(rng.integers(0, 12))
    max_context = int(rng.choice([256, 1024, 1 << 20]))
    c = cfg(spkv, window=w, max_context=max_context)
    out = C.c_int64()
    rc = spkv.lib().spkv_safe_steps_from_lengths(C.byref(c), lens.ctypes.data, ts.ctypes.data, n_units, free,
                                                 C.byref(out))
    assert rc == 0
    assert out.value == brute_force_safe_steps(w, max_context, lens, ts, free), (w, lens, ts, free)


def test_safe_step_budget_special_cases(spkv):
    import numpy as np
    c = cfg(spkv, window=128, max_context=1 << 20)
    out = C.c_int64()
    f = spkv.lib().spkv_safe_steps_from_lengths

    def one(ln, t, free):
        a, b = np.array([ln], np.int32), np.array([t], np.int32)     # kept alive across the call
        return f(C.byref(c), a.ctypes.data, b.ctypes.data, 1, free, C.byref(out)), out.value

    assert one(0, 0, 0) == (0, 128)           # an empty unit evicts nothing for w steps
    assert one(0, 128, 0) == (0, 0)           # the next step may need a page and none is free
    assert one(1, 500, 0) == (0, 63)          # 63 rows left in the unit's last page
    assert one(64, 500, 1) == (0, 64)         # one page buys 64 steps
    assert one(0, 0, 3) == (0, 128 + 3 * 64)
    assert f(C.byref(c), None, None, 1, 0, C.byref(out)) == -1
    empty = np.zeros(1, np.int32)
    assert f(C.byref(c), empty.ctypes.data, empty.ctypes.data, 0, 0, C.byref(out)) == 0
    assert out.value == 1 << 31               # nothing to count: no limit


def test_canary_blocks_lie_between_the_metadata_regions(spkv):
    c = cfg(spkv)
    n, total = C.c_int32(), C.c_size_t()
    offs = (C.c_size_t * 16)()
    assert spkv.lib().spkv_arena_canaries(C.byref(c), offs, 16, C.byref(n)) == 0
    assert spkv.lib().spkv_arena_bytes(C.byref(c), C.byref(total)) == 0
    o = list(offs)[:n.value]
    assert n.value == 11 and o == sorted(o) and o[0] == 256 and all(x % 256 == 0 for x in o)
    units = 2 * 3 * 2
    assert o[-1] + 256 <= total.value - (units * 2 + 100) * 32768     # all before the pages


def test_local_only_heads_cost_no_page_table(spkv):
    """Static hybrid layout declared at creation: the arena shrinks by exactly the page tables of the
    local-only heads' units."""
    import numpy as np
    n_all, n_some, n_none = C.c_size_t(), C.c_size_t(), C.c_size_t()
    c = cfg(spkv, n_layers=3, max_seqs=5, n_q_heads=8, n_kv_heads=4, max_context=64 * 1024)
    assert spkv.lib().spkv_arena_bytes(C.byref(c), C.byref(n_all)) == 0
    flags = np.zeros((3, 4), np.uint8)
    flags[0, :] = 1
    flags[2, 1] = 1                       # 5 of the 12 heads
    c.h_local_only = flags.ctypes.data
    assert spkv.lib().spkv_arena_bytes(C.byref(c), C.byref(n_some)) == 0
    assert n_all.value - n_some.value == 5 * 5 * 1024 * 4          # heads x sequences x entries x 4 bytes
    flags[:] = 1
    assert spkv.lib().spkv_arena_bytes(C.byref(c), C.byref(n_none)) == 0
    assert n_all.value - n_none.value == 12 * 5 * 1024 * 4
    big = cfg(spkv, n_q_heads=130, n_kv_heads=65)
    big.h_local_only = flags.ctypes.data
    assert spkv.lib().spkv_arena_bytes(C.byref(big), C.byref(n_none)) == -3
