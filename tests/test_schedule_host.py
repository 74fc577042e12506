"""The attention kernel's static schedule is plain C++ shared by host and device: compile it for the host and
sweep it (every query tile exactly once, even load, at most one pair across two heads per CTA at the model shapes)."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs a host C++ compiler")
def test_every_tile_once_even_load_straddling_pairs_spread(tmp_path):
    exe = str(tmp_path / "schedule_check")
    subprocess.run(["g++", "-O2", "-std=c++17", "-I", os.path.join(ROOT, "paper_2604_17397_b200", "csrc"),
                    os.path.join(ROOT, "tests", "schedule_check.cpp"), "-o", exe], check=True)
    r = subprocess.run([exe], capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.startswith("ok "), r.stdout + r.stderr
