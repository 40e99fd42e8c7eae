"""The C boundary from a C program: include/kvrebuild.h compiles as C99 with warnings as errors, and a
program that links only libkvrebuild.so calls the host-only entry points (no GPU is touched)."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("gcc") is None, reason="no C compiler")
def test_header_is_c_and_host_entry_points_run_from_c(tmp_path):
    from paper_2608_14635_b200 import binding as kb
    lib_dir, lib_file = os.path.split(kb.LIB_PATH)
    exe = str(tmp_path / "host_calls")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
           os.path.join(ROOT, "tests", "c_abi", "host_calls.c"), "-o", exe, "-L", lib_dir, "-l:" + lib_file,
           "-Wl,-rpath," + lib_dir]
    built = subprocess.run(cmd, capture_output=True, text=True)
    assert built.returncode == 0, built.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0, run.stdout + run.stderr
    assert "c abi host calls ok" in run.stdout
