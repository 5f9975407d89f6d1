"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments
on the host without launching anything (no GPU needed)."""
import ctypes as C
import os
import re
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "diffqkv.h")
HEADERS = [HEADER, os.path.join(ROOT, "include", "diffqkv_debug.h")]


@pytest.fixture(scope="module")
def api():
    from paper_2501_13629_b200 import build
    build.build()
    from paper_2501_13629_b200 import api as _api
    return _api


def _declared_functions():
    text = "".join(open(h).read() for h in HEADERS)
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:diffqkv|gqa)_[a-z0-9_]+)\s*\(", text)))


def test_header_compiles_as_plain_c(tmp_path):
    src = tmp_path / "t.c"
    src.write_text('#include "diffqkv.h"\n#include "diffqkv_debug.h"\n'
                   'int main(void){diffqkv_shape s; (void)s; return DIFFQKV_OK;}\n')
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.dirname(HEADER), "-c", str(src),
                           "-o", str(tmp_path / "t.o")])


def test_every_declared_symbol_is_exported(api):
    names = _declared_functions()
    assert "diffqkv_decode" in names and "gqa_decode" in names and "diffqkv_combine" in names
    assert "diffqkv_prefill" in names and "diffqkv_debug_decode_timeout" in names and "diffqkv_fold_k_up" in names
    lib = C.CDLL(api.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert set(api.EXPORTS) <= set(names)


def test_status_strings(api):
    assert api.status_string(api.OK) == "ok"
    assert len({api.status_string(i) for i in range(8)}) == 8


def test_planning_functions(api):
    import torch
    sh = api.make_shape(4, 32, 4, 8, 128, 128, torch.bfloat16, torch.float32, 0.088)
    s = api.diffqkv_decode_num_splits(sh, 32768)
    assert s >= 1
    need = api.diffqkv_decode_workspace_bytes(sh, 32768, 0)
    assert need >= 4 * 32 * s * (128 + 1) * 4
    assert api.diffqkv_decode_workspace_bytes(sh, 32768, 1) >= 4 * 32 * 129 * 4
    bad = api.make_shape(4, 32, 5, 8, 128, 128, torch.bfloat16, torch.float32, 0.088)
    assert api.diffqkv_decode_workspace_bytes(bad, 32768, 0) == 0


def test_host_side_argument_errors(api):
    """Null pointers and non-dividing head counts are refused before anything is launched."""
    import torch
    lib = api._lib
    sh = api.make_shape(1, 6, 4, 3, 64, 64, torch.bfloat16, torch.float32, 1.0)
    cs = api.CacheStruct()
    st = lib.diffqkv_decode(None, C.byref(cs), C.byref(sh), 0, None, 0, None, None, None, None)
    assert st == api.ERR_INVALID_ARG
    sh = api.make_shape(1, 8, 4, 2, 64, 64, torch.bfloat16, torch.float32, 1.0)
    st = lib.diffqkv_decode(None, C.byref(cs), C.byref(sh), 0, None, 0, None, None, None, None)
    assert st == api.ERR_INVALID_ARG  # null q / out
    st = lib.gqa_decode(C.c_void_p(256), C.byref(cs), C.byref(sh), 0, None, 0, C.c_void_p(256), None, None, None)
    assert st == api.ERR_INVALID_ARG  # n_k != n_v
    sh = api.make_shape(1, 8, 4, 2, 60, 64, torch.bfloat16, torch.float32, 1.0)
    st = lib.diffqkv_decode(C.c_void_p(256), C.byref(cs), C.byref(sh), 0, None, 0, C.c_void_p(256), None, None, None)
    assert st == api.ERR_UNSUPPORTED  # d_qk not a multiple of the 16-byte vector
    st = lib.diffqkv_combine(None, None, 1, 1, 64, 1, 0, None, None, None)
    assert st == api.ERR_INVALID_ARG
