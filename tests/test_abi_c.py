"""include/drk.h is valid C99, and the library is usable from C without Python or torch in the process."""
import os
import shutil
import subprocess

import pytest

from paper_2602_05885_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_header_compiles_as_c_and_host_entry_points_work(tmp_path):
    exe = str(tmp_path / "abi_check")
    src = os.path.join(ROOT, "tests", "c", "abi_check.c")
    # the header by itself, strictly
    hdr = subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-fsyntax-only", "-x", "c",
                          os.path.join(ROOT, "include", "drk.h")], capture_output=True, text=True)
    assert hdr.returncode == 0, hdr.stderr
    # (dlsym's object-to-function pointer conversion is outside ISO C, hence no -pedantic for the program)
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"), src,
           "-o", exe, "-ldl", "-lm"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    run = subprocess.run([exe, build.build_library()], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0, (run.returncode, run.stdout, run.stderr)
    assert "abi ok" in run.stdout
