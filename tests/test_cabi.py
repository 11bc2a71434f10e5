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
