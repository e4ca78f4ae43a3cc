"""The C boundary without a GPU: the library loads, exports what include/ersd.h declares,
and rejects bad arguments on the host before anything is launched."""
import ctypes as C
import os
import re

import pytest

from paper_2504_15475_b200 import build as ersd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    ersd_build.build()
    from paper_2504_15475_b200 import binding
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ersd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ersd_[a-z_]+)\s*\(", text)))


def test_every_declared_entry_point_is_exported(L):
    names = declared_functions()
    assert {"ersd_race_sample", "ersd_verify", "ersd_verify_tree"} <= set(names)
    for n in names:
        assert hasattr(L, n), n
    from paper_2504_15475_b200 import binding
    assert set(binding.EXPORTS) == set(names)
    for n in names:                       # the Python binding carries the same names
        assert hasattr(binding, n) or n in ("ersd_status_string", "ersd_last_cuda_error"), n


def test_opts_struct_layout_matches_header():
    from paper_2504_15475_b200 import binding
    text = open(os.path.join(ROOT, "include", "ersd.h")).read()
    body = re.search(r"typedef struct ersd_opts \{(.*?)\} ersd_opts;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [re.search(r"(\w+)\s*$", d.strip()).group(1) for d in body.split(";") if d.strip()]
    assert fields == [f[0] for f in binding.ErsdOpts._fields_]
    # sizes and offsets as a C compiler sees the header
    import subprocess, tempfile
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "t.c")
        open(src, "w").write(
            '#include <stdio.h>\n#include <stddef.h>\n#include "ersd.h"\n'
            'int main(void){printf("%zu %zu %zu %zu", sizeof(ersd_opts), offsetof(ersd_opts, temps),'
            ' offsetof(ersd_opts, out_key), offsetof(ersd_opts, workspace_bytes));return 0;}\n')
        exe = os.path.join(d, "t")
        subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), src, "-o", exe])
        got = [int(v) for v in subprocess.check_output([exe]).split()]
    O = binding.ErsdOpts
    assert got == [C.sizeof(O), O.temps.offset, O.out_key.offset, O.workspace_bytes.offset]


def test_status_strings_and_version(L):
    assert L.ersd_version() >= 100
    assert L.ersd_status_string(0) == b"ok"
    for s in (-1, -2, -3, -4, -5):
        assert len(L.ersd_status_string(s)) > 3
    assert L.ersd_workspace_bytes(0, 4) == 0
    assert L.ersd_workspace_bytes(8, 5) >= 8 * 5 * (4 + 2 * 64 * 16)


def test_argument_errors_are_found_on_the_host(L):
    """None of these reaches a CUDA call (there is no GPU here)."""
    p = C.c_void_p(0x1000)          # plausible aligned non-null address; never dereferenced
    odd = C.c_void_p(0x1001)
    EINVAL, EALIGN, EUNSUP = -1, -2, -3
    f = L.ersd_race_sample
    assert f(None, 1, p, 1, 1, 8, 1.0, p, None, None) == EINVAL
    assert f(p, 1, None, 1, 1, 8, 1.0, p, None, None) == EINVAL
    assert f(p, 1, p, 1, 1, 8, 1.0, None, None, None) == EINVAL
    assert f(p, 1, p, 0, 1, 8, 1.0, p, None, None) == EINVAL
    assert f(p, 1, p, 1, 1, 0, 1.0, p, None, None) == EINVAL
    assert f(p, 7, p, 1, 1, 8, 1.0, p, None, None) == EINVAL
    assert f(p, 1, p, 1, 1, 8, -0.5, p, None, None) == EINVAL
    assert f(p, 1, p, 1, 1, 8, float("nan"), p, None, None) == EINVAL
    assert f(p, 1, p, 1, 1, 8, float("inf"), p, None, None) == EINVAL
    assert f(odd, 1, p, 1, 1, 8, 1.0, p, None, None) == EALIGN
    assert f(p, 1, p, 1, 1, 0x7FFF0001, 1.0, p, None, None) == EUNSUP
    from paper_2504_15475_b200.binding import ErsdOpts
    o = ErsdOpts()
    o.struct_size = C.sizeof(ErsdOpts)
    o.top_c = 65
    assert f(p, 1, p, 1, 1, 8, 1.0, p, C.byref(o), None) == EUNSUP
    v = L.ersd_verify
    assert v(p, None, 1, p, 1, 2, 8, 1.0, p, p, None, None) == EINVAL      # k > 0 needs draft rows
    assert v(p, p, 1, p, 1, -1, 8, 1.0, p, p, None, None) == EINVAL
    assert v(p, p, 1, p, 1, 256, 8, 1.0, p, p, None, None) == EUNSUP
    assert v(p, p, 1, p, 1, 2, 8, 1.0, None, p, None, None) == EINVAL
    assert v(p, odd, 1, p, 1, 2, 8, 1.0, p, p, None, None) == EALIGN
    t = L.ersd_verify_tree
    good = (C.c_int32 * 3)(-1, 0, 0)
    bad_root = (C.c_int32 * 3)(0, 0, 0)
    forward = (C.c_int32 * 3)(-1, 2, 0)
    assert t(p, p, 1, None, p, 1, 2, 8, 1.0, p, p, None, None) == EINVAL
    assert t(p, p, 1, bad_root, p, 1, 2, 8, 1.0, p, p, None, None) == EINVAL
    assert t(p, p, 1, forward, p, 1, 2, 8, 1.0, p, p, None, None) == EINVAL
    assert t(p, p, 1, good, p, 1, 2, 8, -1.0, p, p, None, None) == EINVAL
    wide = (C.c_int32 * 67)(-1, *([0] * 66))                                 # 66 children: beyond ERSD_MAX_TOP_C
    assert t(p, p, 1, wide, p, 1, 66, 8, 1.0, p, p, None, None) == EUNSUP
    o = ErsdOpts()
    o.struct_size = C.sizeof(ErsdOpts)
    o.ld_target = 4                                                          # stride below V
    assert v(p, p, 1, p, 1, 2, 8, 1.0, p, p, C.byref(o), None) == EINVAL
    o = ErsdOpts()
    o.struct_size = C.sizeof(ErsdOpts)
    o.kernel_path = 3                                                        # 0, 1, 2 are the choices
    assert v(p, p, 1, p, 1, 2, 8, 1.0, p, p, C.byref(o), None) == EINVAL
    assert f(p, 1, p, 1, 1, 8, 1.0, p, C.byref(o), None) == EINVAL
    o.kernel_path = 2                                                        # the cluster kernel where it cannot run
    assert v(p, p, 1, p, 1, 32, 8, 1.0, p, p, C.byref(o), None) == EUNSUP    # more than 32 positions
    assert v(p, C.c_void_p(0x1002), 1, p, 1, 2, 8, 1.0, p, p, C.byref(o), None) == EUNSUP  # draft rows not 16-byte aligned
    star33 = (C.c_int32 * 34)(-1, *([0] * 33))
    assert t(p, p, 1, star33, p, 1, 33, 8, 1.0, p, p, C.byref(o), None) == EUNSUP  # more than 32 arrivals per race
    o.top_c = 33
    assert f(p, 1, p, 1, 1, 8, 1.0, p, C.byref(o), None) == EUNSUP
    assert L.ersd_verify_tokens(p, None, 1, p, 1, 2, 8, 1.0, p, p, None, None) == EINVAL      # k > 0 needs tokens
    assert L.ersd_verify_tokens(p, C.c_void_p(4098), 1, p, 1, 2, 8, 1.0, p, p, None, None) == -2  # misaligned int32
    assert L.ersd_row_keys(None, 1, 8, 1.0, 0, 0, 0, 0, p, None) == EINVAL
    assert L.ersd_row_keys(p, 1, 8, 1.0, 0, 0, 0, 3, p, None) == EINVAL     # modes are 0, 1, 2
    assert L.ersd_workspace_init(None, 16, None) == EINVAL


def test_tree_depth_helper(L):
    from paper_2504_15475_b200 import binding, workloads as wl
    assert binding.ersd_tree_depth(wl.TREE_4x4) == 4
    assert binding.ersd_tree_depth(wl.TREE_SPECINFER) == 4
    assert binding.ersd_tree_depth(wl.chain_parent(7)) == 7
    assert binding.ersd_tree_depth(wl.star_parent(5)) == 1
    assert binding.ersd_tree_depth([-1]) == 0
    assert binding.ersd_tree_depth([-1, 1]) == -1
    assert binding.ersd_tree_depth([0, 0]) == -1


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2504_15475_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libersd.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
