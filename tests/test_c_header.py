"""include/psd.h is a C header and libpsd_b200.so a C library: a C99 program compiled with gcc -pedantic
includes the one, links the other and exercises the host-side calls (no GPU needed)."""
import os
import shutil
import subprocess

import pytest

import paper_2605_15609_b200 as psd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c99_program_against_the_library(tmp_path):
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("gcc not found")
    lib_dir = os.path.dirname(psd.LIB_PATH)
    lib_name = os.path.basename(psd.LIB_PATH)[3:-3]          # libNAME.so -> NAME
    exe = tmp_path / "c_abi_check"
    build = subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"),
                            os.path.join(ROOT, "tests", "c_abi_check.c"), "-o", str(exe), "-L", lib_dir, "-l" + lib_name,
                            "-Wl,-rpath," + lib_dir], capture_output=True, text=True)
    assert build.returncode == 0, build.stderr[-3000:]
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and run.stdout.strip().startswith("ok"), run.stdout + run.stderr[-2000:]
