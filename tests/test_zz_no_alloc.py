"""sh_compress_static — the compression entry point for callers that cannot
allocate device memory (a server whose KV-block pool already owns all of HBM,
or code in a latency-critical loop that must not trigger cudaMalloc's implicit
synchronisation).  It keeps its selection scratch in a static device array
inside the library.  This test drives it through the C ABI next to the regular
sh_compress on identical caches and requires bit-identical results on two
compressions in a row (the second call sees the scratch the first one left
behind).  It is collected last so that a failure here cannot hide another test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2305_17118_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,unordered,shape", [
    ("f16", False, (37, 128, 100, 8, 24, 30)),        # stable compaction: the static array holds every survivor's source slot
    ("int4", False, (37, 128, 100, 8, 24, 30)),
    ("f16", False, (700, 64, 410, 64, 128, 64)),      # 287 000 entries of the array in use
    ("f16", True, (3, 64, 1000, 10, 700, 400)),       # hole filling with bit-planes too large for the one-kernel path:
                                                      # the static array carries the list of moves between two kernels
    ("f16", True, (37, 128, 100, 8, 24, 30)),         # one-kernel path: same entry point, the array stays untouched
])
def test_static_scratch_compress_matches_regular_compress_twice(dtype, unordered, shape):
    from paper_2305_17118_b200 import binding as sh
    U, d, B, r, w, m = shape
    T = B + m + 5     # fills once at step B, again at step B + m
    q, k, v = wl.random_stream(U, d, T, seed=21, dtype=dtype, peaked=3.0, device="cuda")
    a = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=unordered)
    b = sh.Handle(B, r, w, m, U, d, dtype, auto_compress=False, unordered=unordered)
    calls = 0
    for t in range(T):
        oa = a.decode_step(q[t], k[t], v[t])
        ob = b.decode_step(q[t], k[t], v[t])
        assert torch.equal(oa, ob)
        ea = C.c_int(-1)
        eb = C.c_int(-1)
        assert sh.lib.sh_compress(a._h, torch.cuda.current_stream().cuda_stream, C.byref(ea)) == sh.SH_OK
        assert sh.lib.sh_compress_static(b._h, torch.cuda.current_stream().cuda_stream, C.byref(eb)) == sh.SH_OK
        assert ea.value == eb.value
        if ea.value:
            calls += 1
            sa, sb = a.state(), b.state()
            assert sa[0] == sb[0] == B - m
            for x, y in zip(sa[2:], sb[2:]):
                assert (x == y).all()
            for u in (0, U // 2, U - 1):
                Ka, Va = a.export_unit(u)
                Kb, Vb = b.export_unit(u)
                n = sa[0]
                assert (Ka[:n] == Kb[:n]).all() and (Va[:n] == Vb[:n]).all()
    assert calls == 2


def test_static_scratch_rejects_problems_beyond_its_capacity():
    from paper_2305_17118_b200 import binding as sh
    B, U = 1024, 1025          # U * B just over the static array's capacity
    assert U * B > sh.SH_STATIC_SCRATCH_MAX_ENTRIES
    h = sh.Handle(B, 1, 2, 2, U, 64, "f16", auto_compress=False)
    ev = C.c_int(-1)
    assert sh.lib.sh_compress_static(h._h, None, C.byref(ev)) == sh.SH_ETOOBIG
    assert ev.value == 0
    assert b"capacity" in sh.lib.sh_strerror(sh.SH_ETOOBIG)
    assert sh.lib.sh_compress_static(None, None, None) == sh.SH_EINVAL
