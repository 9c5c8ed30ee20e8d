"""The C-ABI library loads without a GPU and exports every function include/hbf.h declares."""
import ctypes
import os
import re

import pytest

from paper_2609_09800_b200 import build as hbf_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def so_path():
    return hbf_build.build()


def declared_functions():
    with open(os.path.join(ROOT, "include", "hbf.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(hbf_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ("hbf_create", "hbf_register_range", "hbf_submit_batch", "hbf_thermal_step", "hbf_last_result",
                 "hbf_workspace_bytes", "hbf_destroy"):
        assert must in names


def test_library_exports_every_declared_symbol(so_path):
    lib = ctypes.CDLL(so_path)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_functions(so_path):
    from paper_2609_09800_b200 import hbf
    assert sorted(hbf.EXPORTS) == [n for n in declared_functions() if not n.endswith("_t")]
    lib = hbf.lib()
    assert lib.hbf_strerror(-7).decode().startswith("batch refused")
    assert lib.hbf_strerror(0) == b"ok"


def test_host_side_argument_checks_need_no_gpu(so_path):
    from paper_2609_09800_b200 import hbf
    lib = hbf.lib()
    assert lib.hbf_create(None, None, None) == hbf.E_INVAL
    assert lib.hbf_destroy(None) == hbf.E_INVAL
    assert lib.hbf_workspace_bytes(None, 10) == 0
    assert lib.hbf_submit_host(None, None, 0, None, None, None, 0, None) == hbf.E_INVAL
    cfg = hbf.hbf_config_t()                       # all zero: rejected before any CUDA call
    h = ctypes.c_void_p()
    assert lib.hbf_create(ctypes.byref(cfg), None, ctypes.byref(h)) == hbf.E_INVAL


def test_struct_layouts_match_the_header(tmp_path):
    """Compiles the header with gcc and compares sizes and field offsets with the ctypes mirror."""
    import subprocess
    from paper_2609_09800_b200 import hbf
    fields = [n for n, _ in hbf.hbf_config_t._fields_]
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "hbf.h"\nint main(void){\n'
                   'printf("%zu %zu %zu %zu\\n", sizeof(hbf_config_t), sizeof(hbf_batch_result_t), sizeof(hbf_access_t), sizeof(hbf_die_stats_t));\n'
                   + "".join('printf("%%zu\\n", offsetof(hbf_config_t, %s));\n' % f for f in fields) + "return 0;}\n")
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    out = subprocess.check_output([str(exe)]).decode().split()
    assert [int(x) for x in out[:4]] == [ctypes.sizeof(hbf.hbf_config_t), ctypes.sizeof(hbf.hbf_batch_result_t),
                                         hbf.ACCESS_DTYPE.itemsize, hbf.DIE_STATS_DTYPE.itemsize]
    assert [int(x) for x in out[4:]] == [getattr(hbf.hbf_config_t, f).offset for f in fields]
