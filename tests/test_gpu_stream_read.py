"""The read-stream measurement aid: it must touch every 32 KB page of the buffer exactly once
(its checksum adds the first 32-bit word of each page), leave its page counter at zero for the
next call, and report no timed-out wait."""
import ctypes as C

import numpy as np
import pytest
import torch

from gpu_util import dev, load

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_pages,tail", [(1, 0), (5, 100), (6, 0), (7, 32767), (148 * 13 + 3, 16)])
def test_stream_read_visits_every_page_once(n_pages, tail):
    spkv = load()
    words = np.zeros((n_pages * 32768 + tail) // 4 + 1, dtype=np.uint32)
    first = np.random.default_rng(n_pages).integers(0, 2 ** 32, size=n_pages, dtype=np.uint64).astype(np.uint32)
    words[np.arange(n_pages) * 8192] = first
    buf = torch.from_numpy(words.view(np.uint8)[:n_pages * 32768 + tail].copy()).to(dev())
    sink = torch.zeros(2, dtype=torch.int64, device=dev())      # checksum, page counter
    status = torch.zeros(1, dtype=torch.int32, device=dev())
    for rep in range(3):
        rc = spkv.lib().spkv_stream_read(C.c_void_p(buf.data_ptr()), buf.numel(), C.c_void_p(sink.data_ptr()),
                                         C.c_void_p(status.data_ptr()), C.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert int(sink[0].item()) == 3 * int(first.astype(np.uint64).sum())
    assert int(sink[1].item()) == 0          # the last claim of every launch clears the counter


def test_stream_read_rejects_bad_arguments_and_ignores_less_than_a_page():
    spkv = load()
    buf = torch.zeros(40000, dtype=torch.uint8, device=dev())
    sink = torch.zeros(2, dtype=torch.int64, device=dev())
    status = torch.zeros(1, dtype=torch.int32, device=dev())
    s = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    f = spkv.lib().spkv_stream_read
    assert f(None, 40000, C.c_void_p(sink.data_ptr()), C.c_void_p(status.data_ptr()), s) != 0
    assert f(C.c_void_p(buf.data_ptr() + 4), 36000, C.c_void_p(sink.data_ptr()), C.c_void_p(status.data_ptr()), s) != 0
    assert f(C.c_void_p(buf.data_ptr()), 1000, C.c_void_p(sink.data_ptr()), C.c_void_p(status.data_ptr()), s) == 0
    assert spkv.spkv_stream_read(buf, passes=2) > 0


def test_a_bounded_wait_runs_out_and_the_context_stays_usable():
    """Failure path without a fault: a barrier armed for more bytes than its copy delivers.  The
    wait gives up after the limit it was given (about a millisecond here), the kernel reports
    SPKV_E_TIMEOUT, waits for the copy it has in flight and returns; the next calls on the same
    context work as if nothing had happened."""
    spkv = load()
    words = np.arange(8192 * 2, dtype=np.uint32) + 77
    buf = torch.from_numpy(words.view(np.uint8).copy()).to(dev())
    limit = 2_000_000                      # clocks: ~1 ms at ~2 GHz
    code, drained, waited, data_ok = spkv.spkv_wait_selftest(buf, limit)
    assert code == -8 and spkv.lib().spkv_error_string(code) == b"bounded device wait ran out"
    assert drained == 1 and data_ok == 1
    assert limit <= waited < 50 * limit, waited
    # a second run gives the same answer, and ordinary work follows without an error
    assert spkv.spkv_wait_selftest(buf, limit // 4)[:2] == [-8, 1]
    assert torch.cuda.current_stream().query() in (True, False)
    torch.cuda.synchronize()
    assert spkv.spkv_stream_read(buf, passes=1) > 0
    assert spkv.lib().spkv_wait_selftest(None, limit, None, None) == -1
