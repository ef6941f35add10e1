"""The C-ABI library builds, loads and exports what include/fb4.h declares; host-side argument
checks that need no device.  No kernel runs here."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2603_02883_b200 import fb4, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fb4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fb4_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = fb4.lib()
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(L, n), f"{n} declared in fb4.h but not exported"
    assert sorted(fb4.EXPORTS) == names


def test_default_config():
    cfg = fb4.Fb4Config()
    fb4.lib().fb4_default_config(ctypes.byref(cfg))
    assert (cfg.block_size, cfg.num_groups, cfg.exp_min, cfg.exp_max, cfg.select_mode) == (32, 8, -124, 127, 0)


def test_strerror_names_every_code():
    L = fb4.lib()
    seen = {L.fb4_strerror(c).decode() for c in range(0, -7, -1)}
    assert len(seen) == 7 and "unknown error" not in seen
    assert L.fb4_strerror(-99).decode() == "unknown error"


def test_init_rejects_bad_arguments_before_touching_a_device():
    L = fb4.lib()
    h = ctypes.c_void_p()
    assert L.fb4_init(None, 0, None, None, None) == fb4.ERR_INVALID_ARG
    bad = synth.STANDIN_FORMATBOOK.copy()
    bad[3, 4] = bad[3, 3]                       # not strictly ascending
    assert L.fb4_init(ctypes.byref(h), 0, bad.ctypes.data_as(ctypes.c_void_p), None, None) == fb4.ERR_FORMATBOOK
    bad = synth.STANDIN_FORMATBOOK.copy()
    bad[0, 0] = 1                               # index 0 must be the value 0
    assert L.fb4_init(ctypes.byref(h), 0, bad.ctypes.data_as(ctypes.c_void_p), None, None) == fb4.ERR_FORMATBOOK
    for cfg in (fb4.Fb4Config(24, 8, -124, 127, 0), fb4.Fb4Config(32, 4, -124, 127, 0),
                fb4.Fb4Config(32, 8, -130, 127, 0), fb4.Fb4Config(32, 8, 5, 4, 0), fb4.Fb4Config(32, 8, -124, 127, 2)):
        assert L.fb4_init(ctypes.byref(h), 0, None, None, ctypes.byref(cfg)) == fb4.ERR_INVALID_ARG
    assert h.value is None


def test_null_context_is_rejected():
    L = fb4.lib()
    assert L.fb4_quantize(None, None, 1, 32, 32, None, None, None) == fb4.ERR_INVALID_ARG
    assert L.fb4_dequantize(None, None, None, 1, 32, None, 0, None, None, None, 0, None) == fb4.ERR_INVALID_ARG
    assert L.fb4_destroy(None) == fb4.OK
    assert L.fb4_launch_count(None) == 0


def test_no_device_is_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = ctypes.c_void_p()
    assert fb4.lib().fb4_init(ctypes.byref(h), 0, None, None, None) == fb4.ERR_NO_DEVICE
    with pytest.raises(RuntimeError):
        fb4.Fb4()


def test_header_is_plain_c(tmp_path):
    """include/fb4.h is a C header: it must compile as C99 on its own, and a C caller must link."""
    import subprocess
    src = tmp_path / "use_fb4.c"
    src.write_text('#include "fb4.h"\n'
                   "int main(void) {\n"
                   "  fb4_config cfg;\n"
                   "  fb4_default_config(&cfg);\n"
                   "  return (cfg.block_size == 32 && fb4_mxfp8_scale_bytes(128, 128, 1) == 512 &&\n"
                   "          fb4_quantize(0, 0, 1, 32, 32, 0, 0, 0) == FB4_ERR_INVALID_ARG) ? 0 : 1;\n"
                   "}\n")
    exe = tmp_path / "use_fb4"
    libdir = os.path.dirname(fb4.library_path())
    fb4.lib()
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe), "-L", libdir, "-lfb4", f"-Wl,-rpath,{libdir}"])
    assert subprocess.call([str(exe)]) == 0
