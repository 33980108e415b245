"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, its host-side
calibration helpers agree with the oracle, and argument validation answers without touching a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import build as libbuild
from paper_2603_24840_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return B.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "arrol.h")).read()
    declared = set(re.findall(r"\b(arrol_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert B.arrol_version() >= 100
    assert B.status_string(0) == "ok" and "argument" in B.status_string(-1)


def test_calibration_helpers_match_the_oracle():
    for name in ("tiny", "qwen3-4b"):
        w = synth.WORKLOADS[name]
        s, y = synth.calib_history(w)
        cpos, cneg = B.arrol_calib_counts(s, y, w.B)
        ocpos, ocneg = oracle.calib_counts(s, y, w.B)
        assert np.array_equal(cpos, ocpos) and np.array_equal(cneg, ocneg)
        for alpha in (1.0, 0.5):
            lut = B.arrol_build_q_lut(cpos, cneg, alpha)
            _, o32 = oracle.build_q_lut(ocpos, ocneg, alpha)
            assert lut.dtype == np.float32 and np.array_equal(lut, o32)      # same doubles, rounded once
    lut = B.arrol_build_q_lut([0, 1, 2, 5], [6, 3, 2, 1], 1.0)
    assert np.allclose(lut, [8 / 71, 4 / 13, 8 / 17, 8 / 11], atol=1e-7)
    cpos, cneg = B.arrol_calib_counts(np.array([1.0, 0.0, 0.999999]), np.array([1, 0, 1], np.uint8), 4)
    assert list(cpos) == [0, 0, 0, 2] and list(cneg) == [1, 0, 0, 0]


def test_host_side_argument_errors_need_no_gpu(lib):
    null = C.c_void_p()
    assert lib.arrol_create(None, 0) == -1
    assert lib.arrol_build_q_lut(None, None, 4, 1.0, None) == -1
    assert lib.arrol_calib_counts(None, None, 5, 0, None, None) == -1
    # every compute call rejects a NULL context before anything else
    assert lib.arrol_select(null, None, 1, 8, 4, 0.5, 0, None, None) == -1
    assert lib.arrol_score_partial(null, None, 0, None, 1, None, None, None, None, None, None, None) == -1
    assert lib.arrol_token_logprob(null, None, None, None, 1, None, 64, 64, 1.0, None, None, None, 0, None) == -1
    assert lib.arrol_token_logprob_workspace(null, 10, 64, 64) == 0
    assert lib.arrol_poll_status(null, None, None) == -1
    assert lib.arrol_destroy(null) == 0


def test_create_without_a_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = C.c_void_p()
    rc = lib.arrol_create(C.byref(h), 0)
    assert rc in (-7, -5) and not h.value          # no CPU fallback: the context cannot be made
    with pytest.raises(B.ArrolError):
        B.Context(0)


def test_header_is_plain_c_and_links_against_the_library(tmp_path, lib):
    """The boundary is a C ABI: the header compiles as strict C99 and a C program links against the library and
    calls an entry point that needs no GPU."""
    import os
    import shutil
    import subprocess
    from paper_2603_24840_b200 import binding as B
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "c_abi.c"
    src.write_text('#include <stdio.h>\n#include "arrol.h"\n'
                   'int main(void) { printf("%d %s\\n", arrol_version(), arrol_status_string(ARROL_ERR_WORKSPACE));\n'
                   '  return arrol_create(NULL, 0) == ARROL_ERR_INVALID_ARG ? 0 : 1; }\n')
    exe = tmp_path / "c_abi"
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.check_call([gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(root, "include"),
                           str(src), "-o", str(exe), "-L", libdir, "-l:libarrol.so", "-Wl,-rpath," + libdir])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0
    assert out.stdout.split()[0] == str(B.arrol_version())
