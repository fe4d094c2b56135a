"""The scheduler's ordering ledger (host-side vector clocks over streams and events) on hand-made
schedules: compiled with the host compiler and run, no GPU involved."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_ledger_accepts_correct_schedules_and_reports_missing_waits(tmp_path):
    cxx = shutil.which("g++") or shutil.which("c++")
    if cxx is None:
        pytest.skip("no host C++ compiler")
    exe = str(tmp_path / "order_ledger_test")
    subprocess.run([cxx, "-std=c++17", "-O1", "-Wall", "-I", os.path.join(ROOT, "paper_2605_27081_b200", "csrc"),
                    os.path.join(ROOT, "tests", "native", "order_ledger_test.cc"), "-o", exe], check=True)
    res = subprocess.run([exe], capture_output=True, text=True)
    assert res.returncode == 0 and res.stdout.strip() == "ok", res.stdout + res.stderr
