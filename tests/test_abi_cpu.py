"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, and turns bad arguments / a missing device into error codes."""
import ctypes as C
import os
import re

import pytest

from paper_2604_09244_b200 import build, mvla

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return mvla.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "mvla_prune.h")).read()
    declared = set(re.findall(r"^\s*(?:int32_t|void)\s+(mvla_\w+)\s*\(", header, flags=re.M))
    assert set(mvla.EXPORTS) <= declared
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_sizes_match_the_header_layout():
    assert C.sizeof(mvla.Config) == 14 * 4 + 6 * 8 + 6 * 4      # five int32 and a reserved one after the doubles
    assert C.sizeof(mvla.CSample) == 8 * 4 + 3 * 8
    assert C.sizeof(mvla.CDiag) == 64
    assert C.sizeof(mvla.CTensors) == 7 * 8
    assert C.sizeof(mvla.COutputs) == 14 * 8
    assert C.sizeof(mvla.CPatchDiag) == 64


def test_bad_arguments_are_error_codes(lib):
    h = C.c_void_p()
    assert lib.mvla_prune_create(None, C.byref(h)) == mvla.ERR_INVALID_ARG
    cfg = mvla.Config(0, mvla.DTYPE_BF16, 32, 128, 4096, 1, 32, 256, 512, 1, 0, 7, 1, 0, 0.08, 0.2, 0.85, 0.02, 0.1)
    assert lib.mvla_prune_create(C.byref(cfg), None) == mvla.ERR_INVALID_ARG
    bad = mvla.Config.from_buffer_copy(cfg); bad.head_dim = 48
    assert lib.mvla_prune_create(C.byref(bad), C.byref(h)) == mvla.ERR_UNSUPPORTED
    bad = mvla.Config.from_buffer_copy(cfg); bad.max_text = 65
    assert lib.mvla_prune_create(C.byref(bad), C.byref(h)) == mvla.ERR_UNSUPPORTED
    bad = mvla.Config.from_buffer_copy(cfg); bad.n_heads = 0
    assert lib.mvla_prune_create(C.byref(bad), C.byref(h)) == mvla.ERR_INVALID_ARG
    bad = mvla.Config.from_buffer_copy(cfg); bad.beta = 1.5
    assert lib.mvla_prune_create(C.byref(bad), C.byref(h)) == mvla.ERR_INVALID_ARG
    # null context
    assert lib.mvla_salience(None, 1, None, None, None, None, 1, None, None, None) == mvla.ERR_INVALID_ARG
    assert lib.mvla_select(None, 0, 1, None, 0, 0, None, None, None, None, None, None, None, None, None) == mvla.ERR_INVALID_ARG
    assert lib.mvla_compact(None, 1, None, None, None, 0, None, None, None, None, None, None, None) == mvla.ERR_INVALID_ARG
    assert lib.mvla_prune_step(None, 0, 1, None, 0, 0, None, None, None, None) == mvla.ERR_INVALID_ARG
    assert lib.mvla_patch_indicators(None, 1, None, None, None, None, 1, None, None, None) == mvla.ERR_INVALID_ARG
    assert lib.mvla_patch_select(None, 0, 1, None, 0, None, None, None, None, None, None, None, None, None, None) == mvla.ERR_INVALID_ARG
    lib.mvla_prune_destroy(None)           # accepted


def test_no_device_is_an_error_not_a_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    h = C.c_void_p()
    cfg = mvla.Config(0, mvla.DTYPE_BF16, 32, 128, 4096, 1, 32, 256, 512, 1, 0, 7, 1, 0, 0.08, 0.2, 0.85, 0.02, 0.1)
    assert lib.mvla_prune_create(C.byref(cfg), C.byref(h)) == mvla.ERR_CUDA
    assert not h


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(OSError):
        mvla.load_library(str(tmp_path / "libmvla_prune.so"))


def test_mvla_log_prints_one_line_per_call():
    """MVLA_LOG=1: every public call reports its arguments and its result on stderr (host side only); without the
    variable nothing is printed.  Runs in a child process: the variable is read once per process."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import ctypes as C, sys\n"
            f"sys.path.insert(0, {root!r})\n"
            "from paper_2604_09244_b200 import mvla\n"
            "lib = mvla.load_library()\n"
            "h = C.c_void_p()\n"
            "cfg = mvla.Config(0, mvla.DTYPE_BF16, 32, 128, 4096, 1, 32, 256, 512, 1, 0, 7, 1, 0, 0.08, 0.2, 0.85, 0.02, 0.1)\n"
            "rc = lib.mvla_prune_create(C.byref(cfg), C.byref(h))\n"
            "rc2 = lib.mvla_salience(None, 1, None, None, None, None, 0, None, None, None)\n"
            "print(rc, rc2)\n")
    for on in (True, False):
        env = dict(os.environ)
        env.pop("MVLA_LOG", None)
        if on:
            env["MVLA_LOG"] = "1"
        r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr
        rc, rc2 = (int(x) for x in r.stdout.split())
        lines = [ln for ln in r.stderr.splitlines() if ln.startswith("[mvla] ")]
        if on:
            assert len(lines) == 2
            assert lines[0].startswith("[mvla] mvla_prune_create(heads 32 x 128, d_model 4096") and lines[0].endswith(f"-> {rc}")
            assert lines[1].startswith("[mvla] mvla_salience(batch 1") and lines[1].endswith(f"-> {rc2}")
        else:
            assert not lines
