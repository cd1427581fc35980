"""Host logic of the launchers: what they remember about a kernel is looked up by device (a process that
uses two GPUs must not launch on the second with what it learned about the first).  The cache is plain
C++ (csrc/launch_cache.hpp); this test compiles a small program against it and runs it with made-up
device numbers."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs a host C++ compiler")
def test_launch_cache_is_indexed_by_device(tmp_path):
    exe = tmp_path / "launch_cache_check"
    src = os.path.join(ROOT, "tests", "cpp", "launch_cache_check.cpp")
    inc = os.path.join(ROOT, "paper_2507_07149_b200", "csrc")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-pthread", "-I", inc, src, "-o", str(exe)])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr


def test_no_environment_flags_on_the_call_path():
    """The library reads no environment variable: launch policy is part of daf_params.flags."""
    csrc = os.path.join(ROOT, "paper_2507_07149_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name)) as f:
            assert "getenv" not in f.read(), name
