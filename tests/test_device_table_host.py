"""The launchers cache per-device CUDA state (a kernel's raised shared-memory limit, the SM count)
in mq::PerDeviceTable.  Its logic is plain C++, so it is compiled with the host compiler and run
here: one initialisation per device, none shared between devices, failures not cached."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_per_device_table_logic(tmp_path):
    gxx = shutil.which("g++")
    if gxx is None:
        pytest.skip("no host C++ compiler")
    exe = str(tmp_path / "device_table_check")
    src = os.path.join(ROOT, "tests", "device_table_check.cpp")
    inc = os.path.join(ROOT, "paper_2502_00425_b200", "csrc")
    subprocess.run([gxx, "-std=c++17", "-O1", "-pthread", "-I", inc, src, "-o", exe], check=True)
    res = subprocess.run([exe], capture_output=True, text=True)
    assert res.returncode == 0 and res.stdout.strip() == "ok", res.stdout + res.stderr
