"""The C-ABI library builds, loads and exports every symbol the header declares
(no compute calls: this runs without a GPU)."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "scissorhands.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sh_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2305_17118_b200 import build
    lib = C.CDLL(build.build())
    names = _declared()
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in scissorhands.h but not exported"


def test_bounds_checked_build_exports_the_same_symbols():
    from paper_2305_17118_b200 import build
    lib = C.CDLL(build.build(debug_bounds=True))
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_entry_points():
    from paper_2305_17118_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_host_only_calls_validate_arguments():
    from paper_2305_17118_b200 import binding as sh
    lib = sh.lib
    h = C.c_void_p()
    assert lib.sh_create(410, 64, 128, 64, 9216, 128, sh.SH_F16, C.byref(h)) == sh.SH_OK
    kv = 2 * 9216 * 410 * 128 * 2
    assert kv < lib.sh_workspace_bytes(h) < 1.1 * kv
    assert lib.sh_set_option(h, sh.SH_OPT_SPLIT, 3.0) == sh.SH_EINVAL
    assert lib.sh_set_option(h, sh.SH_OPT_SOFTMAX_SCALE, -1.0) == sh.SH_EINVAL
    assert lib.sh_set_option(h, 99, 1.0) == sh.SH_EINVAL
    assert lib.sh_compress(h, None, None) == sh.SH_ESTATE           # nothing bound yet
    assert lib.sh_bind(h, None, 0, None) == sh.SH_EINVAL
    assert lib.sh_strerror(sh.SH_EFULL).decode().startswith("cache is full")
    assert lib.sh_last_cuda_error(h) == b""
    lib.sh_destroy(h)
    assert lib.sh_create(410, 64, 128, 64, 9216, 128, sh.SH_F16, None) == sh.SH_EINVAL
    assert lib.sh_create(40000, 64, 128, 64, 1, 128, sh.SH_F16, C.byref(h)) == sh.SH_EINVAL
    assert lib.sh_select(None, 1, 10, 0, 1, None, None) == sh.SH_EINVAL
    one = C.c_void_p(16)          # never dereferenced: the size check comes first
    assert lib.sh_select(one, 1, sh.SH_SELECT_MAX_N + 1, 0, 1, one, None) == sh.SH_EINVAL
    h2 = C.c_void_p()
    assert lib.sh_create(16, 2, 8, 6, 4, 64, sh.SH_F16, C.byref(h2)) == sh.SH_OK
    assert lib.sh_restore(h2, 3, 3) == sh.SH_ESTATE                 # nothing bound
    assert lib.sh_set_option(h2, sh.SH_OPT_SELFTEST_SKIP_TILE, -2.0) == sh.SH_EINVAL
    assert lib.sh_set_option(h2, sh.SH_OPT_SELFTEST_SKIP_TILE, 3.0) == sh.SH_OK
    lib.sh_destroy(h2)


def _handle(sh, B, r, w, m, heads, d, dtype):
    h = C.c_void_p()
    assert sh.lib.sh_create(B, r, w, m, heads, d, sh.DTYPE_CODE[dtype], C.byref(h)) == sh.SH_OK
    return h


def test_option_values_and_the_shapes_they_need():
    """Host logic of sh_set_option: which values each option takes, and which shapes the chunk kernels
    and the recompute mode need (no device call is made)."""
    from paper_2305_17118_b200 import binding as sh
    lib = sh.lib
    h = _handle(sh, 410, 64, 128, 64, 16, 128, "f16")
    assert lib.sh_prefill_chunk_max(h) == 128          # the persistent tcgen05 kernel: up to 128 tokens, never more than w
    assert lib.sh_set_option(h, sh.SH_OPT_PREFILL_CHUNK, 3.0) == sh.SH_OK
    assert lib.sh_prefill_chunk_max(h) == 64           # one CTA per unit: 64
    for key, good, bad in ((sh.SH_OPT_COMPACTION, (0, 1), (2, -1)), (sh.SH_OPT_PREFILL_CHUNK, (0, 1, 2, 3, 4, 1), (5, -1)),
                           (sh.SH_OPT_DECODE_KERNEL, (0, 1, 2), (3,)), (sh.SH_OPT_SPLIT, (1, 2, 4, 8), (3, 16))):
        for v in good:
            assert lib.sh_set_option(h, key, float(v)) == sh.SH_OK, (key, v)
        for v in bad:
            assert lib.sh_set_option(h, key, float(v)) == sh.SH_EINVAL, (key, v)
    before = lib.sh_workspace_bytes(h)
    assert lib.sh_set_option(h, sh.SH_OPT_RECORD_MODE, 1.0) == sh.SH_OK
    assert lib.sh_workspace_bytes(h) >= before + 16 * 128 * 128 * 2          # the ring of the last w queries
    lib.sh_destroy(h)
    # a window shorter than a chunk bounds the chunk; every storage type and head size has a chunk kernel
    # and the recompute mode (fp32 rows and head_dim 64 on CUDA cores)
    h = _handle(sh, 150, 9, 37, 41, 3, 128, "bf16")
    assert lib.sh_prefill_chunk_max(h) == 37
    lib.sh_destroy(h)
    for dtype in ("f32", "f16", "bf16", "int4"):
        for d in (64, 128):
            h = _handle(sh, 410, 64, 128, 64, 3, d, dtype)
            assert lib.sh_prefill_chunk_max(h) == (128 if d == 128 and dtype in ("f16", "bf16") else 64), (dtype, d)
            assert lib.sh_set_option(h, sh.SH_OPT_PREFILL_CHUNK, 4.0) == sh.SH_OK
            assert lib.sh_prefill_chunk_max(h) == 64
            assert lib.sh_set_option(h, sh.SH_OPT_RECORD_MODE, 1.0) == sh.SH_OK, (dtype, d)
            lib.sh_destroy(h)
    # the int4 store with head_dim 128 has a chunk kernel and a recompute mode, on the tcgen05 kernel only
    h = _handle(sh, 150, 9, 37, 41, 3, 128, "int4")
    assert lib.sh_prefill_chunk_max(h) == 37
    assert lib.sh_set_option(h, sh.SH_OPT_PREFILL_CHUNK, 2.0) == sh.SH_OK
    assert lib.sh_prefill_chunk_max(h) == 0
    assert lib.sh_set_option(h, sh.SH_OPT_RECORD_MODE, 1.0) == sh.SH_EINVAL
    assert lib.sh_set_option(h, sh.SH_OPT_PREFILL_CHUNK, 1.0) == sh.SH_OK
    assert lib.sh_set_option(h, sh.SH_OPT_RECORD_MODE, 1.0) == sh.SH_OK
    lib.sh_destroy(h)
    # the warp-level chunk kernel keeps a row of logits in shared memory: it stops at budgets of about 700,
    # the tcgen05 kernel does not; the recompute mode follows the kernel that is chosen
    h = _handle(sh, 4000, 10, 400, 2000, 2, 128, "f16")
    assert lib.sh_prefill_chunk_max(h) == 128
    assert lib.sh_set_option(h, sh.SH_OPT_PREFILL_CHUNK, 2.0) == sh.SH_OK
    assert lib.sh_prefill_chunk_max(h) == 0
    assert lib.sh_set_option(h, sh.SH_OPT_RECORD_MODE, 1.0) == sh.SH_EINVAL
    assert lib.sh_set_option(h, sh.SH_OPT_PREFILL_CHUNK, 1.0) == sh.SH_OK
    assert lib.sh_set_option(h, sh.SH_OPT_RECORD_MODE, 1.0) == sh.SH_OK
    assert lib.sh_set_option(h, sh.SH_OPT_PREFILL_CHUNK, 2.0) == sh.SH_EINVAL      # would strand the recount
    lib.sh_destroy(h)


def test_create_rejects_shapes_outside_the_documented_range():
    from paper_2305_17118_b200 import binding as sh
    lib = sh.lib
    h = C.c_void_p()
    ok = (410, 64, 128, 64, 16, 128, sh.SH_F16)
    assert lib.sh_create(*ok, C.byref(h)) == sh.SH_OK
    lib.sh_destroy(h)
    for bad in ((0, 0, 1, 1, 1, 128, sh.SH_F16), (32769, 1, 1, 1, 1, 128, sh.SH_F16), (410, 64, 16385, 64, 1, 128, sh.SH_F16),
                (410, 64, 0, 64, 1, 128, sh.SH_F16), (410, 64, 128, 0, 1, 128, sh.SH_F16), (410, 64, 128, 347, 1, 128, sh.SH_F16),
                (410, -1, 128, 64, 1, 128, sh.SH_F16), (410, 64, 128, 64, 0, 128, sh.SH_F16), (410, 64, 128, 64, 1, 96, sh.SH_F16),
                (410, 64, 128, 64, 1, 128, 17)):
        assert lib.sh_create(*bad, C.byref(h)) == sh.SH_EINVAL, bad
    assert lib.sh_create(*ok, None) == sh.SH_EINVAL
    for code in (sh.SH_OK, sh.SH_EINVAL, sh.SH_ESTATE, sh.SH_EFULL, sh.SH_ECUDA, sh.SH_ETOOBIG):
        assert len(lib.sh_strerror(code)) >= 2
