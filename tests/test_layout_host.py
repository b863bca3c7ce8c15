"""Packed-code positions of the cache layout, checked on the host (no GPU): `host_layout_check.cpp` includes the
library's layout header, and verifies that every position function is a bijection and that the decode kernel's
mask arithmetic on byte-ordered rows / chunks yields code x weight for the promised (token, channel)."""
import os
import shutil
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "..", "paper_2602_23200_b200", "csrc")


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs a host C++ compiler")
def test_positions_are_bijections_and_operand_bytes_are_code_times_weight(tmp_path):
    exe = str(tmp_path / "host_layout_check")
    subprocess.run(["g++", "-std=c++17", "-O1", "-I", CSRC, "-o", exe, os.path.join(HERE, "host_layout_check.cpp")],
                   check=True)
    r = subprocess.run([exe], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout
    assert r.stdout.strip().endswith("0 failure(s)")
