"""CPU-side checks of the boundary: the shared library builds, loads and exports every symbol
the header declares (no compute calls: there is no GPU here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "elitekv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(elitekv_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_hot_path_calls():
    names = _declared_symbols()
    for must in ("elitekv_append", "elitekv_absorb_query", "elitekv_decode"):
        assert must in names


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2503_01586_b200 import build
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    for name in _declared_symbols():
        assert hasattr(lib, name), name
    lib.elitekv_strerror.restype = ctypes.c_char_p
    assert lib.elitekv_strerror(0) == b"ok"
    assert b"page" in lib.elitekv_strerror(-6)


def test_binding_exposes_the_same_names():
    from paper_2503_01586_b200 import binding
    for name in _declared_symbols():
        if name in ("elitekv_layer_create", "elitekv_layer_destroy", "elitekv_strerror"):
            continue   # wrapped by binding.Layer / binding.strerror
        assert hasattr(binding, name), name


def test_struct_layouts_match_the_header(tmp_path):
    """sizeof/offsetof as the C compiler sees the header vs. the ctypes mirror."""
    import subprocess
    from paper_2503_01586_b200 import binding
    src = tmp_path / "layout.c"
    fields_p = [f[0] for f in binding.Params._fields_]
    fields_c = [f[0] for f in binding.CacheDesc._fields_]
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "elitekv.h"', 'int main(void){',
             'printf("%zu\\n", sizeof(elitekv_params));']
    lines += [f'printf("%zu\\n", offsetof(elitekv_params, {f}));' for f in fields_p]
    lines += ['printf("%zu\\n", sizeof(elitekv_cache));']
    lines += [f'printf("%zu\\n", offsetof(elitekv_cache, {f}));' for f in fields_c]
    lines += ['return 0;}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = [int(x) for x in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    want = [ctypes.sizeof(binding.Params)] + [getattr(binding.Params, f).offset for f in fields_p]
    want += [ctypes.sizeof(binding.CacheDesc)] + [getattr(binding.CacheDesc, f).offset for f in fields_c]
    assert got == want
