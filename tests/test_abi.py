"""The C-ABI library loads without a GPU and exports every symbol the header
declares; argument errors are reported as codes (no compute is attempted)."""
import ctypes
import os
import re
import subprocess

import pytest

from paper_2504_05295_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        for mt in re.finditer(r"\b(dion_[a-z_0-9]+)\s*\(", text):
            names.add(mt.group(1))
    return sorted(names)


def test_header_symbols_are_exported(lib):
    names = declared_functions()
    assert set(binding.EXPORTS) <= set(names)
    raw = ctypes.CDLL(binding.LIB_PATH)
    for nm in names:
        assert hasattr(raw, nm), f"{nm} declared in include/ but not exported"


def test_struct_layout_matches_header(tmp_path):
    # the C compiler's view of include/dion.h against the ctypes structures, field by field
    fields_m = [f for f, _ in binding.DionMatrix._fields_]
    fields_c = [f for f, _ in binding.DionConfig._fields_]
    src = tmp_path / "layout.c"
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "dion.h"', 'int main(void) {',
             '  printf("%zu %zu\\n", sizeof(dion_matrix), sizeof(dion_config));']
    lines += [f'  printf("%zu\\n", offsetof(dion_matrix, {f}));' for f in fields_m]
    lines += [f'  printf("%zu\\n", offsetof(dion_config, {f}));' for f in fields_c]
    lines += ['  return 0;', '}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    subprocess.run(["gcc", "-I", inc, str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    vals = [int(v) for v in out]
    assert vals[0] == ctypes.sizeof(binding.DionMatrix) and vals[1] == ctypes.sizeof(binding.DionConfig)
    got = vals[2:]
    want = [getattr(binding.DionMatrix, f).offset for f in fields_m] + \
           [getattr(binding.DionConfig, f).offset for f in fields_c]
    assert got == want


def test_error_codes_and_strings(lib):
    assert lib.dion_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert lib.dion_strerror(code) not in (b"", b"unknown error")
    assert lib.dion_strerror(-99) == b"unknown error"
    # NULL arguments are rejected before any CUDA call
    assert lib.dion_init(None, None) == -1
    ctx = ctypes.c_void_p()
    assert lib.dion_init(ctypes.byref(ctx), None) == -1
    assert lib.dion_step(None, None, 0.0, None) == -1
    assert lib.dion_step_grouped(None, None, 0, 0.0, None) == -1
    assert lib.dion_workspace_bytes(None, 4, 4, 2) == 0
    assert lib.dion_launch_count(None) == 0
    lib.dion_destroy(None)


def test_default_config_and_bad_enums(lib):
    cfg = binding.DionConfig()
    lib.dion_default_config(ctypes.byref(cfg))
    assert abs(cfg.mu - 0.95) < 1e-7 and abs(cfg.eps - 1e-8) < 1e-12
    assert (cfg.precision, cfg.orth, cfg.engine, cfg.device, cfg.workspace_bytes) == (0, 0, 0, 0, 0)
    ctx = ctypes.c_void_p()
    cfg.orth = 17
    assert lib.dion_init(ctypes.byref(ctx), ctypes.byref(cfg)) == -1 and not ctx.value


def test_init_without_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    cfg = binding.DionConfig()
    lib.dion_default_config(ctypes.byref(cfg))
    ctx = ctypes.c_void_p()
    assert lib.dion_init(ctypes.byref(ctx), ctypes.byref(cfg)) == -6   # DION_ERR_CUDA, no fallback
    assert not ctx.value
