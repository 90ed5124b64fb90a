"""Host-side logic of the launchers that needs neither a GPU nor the CUDA toolkit: compiled with g++ and run."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_per_device_setup_bookkeeping(tmp_path):
    exe = str(tmp_path / "device_once_check")
    src = os.path.join(ROOT, "tests", "host", "device_once_check.cpp")
    inc = os.path.join(ROOT, "paper_2503_02495_b200", "csrc")
    subprocess.run(["g++", "-std=c++17", "-O1", "-Wall", "-Werror", "-I", inc, src, "-o", exe], check=True)
    r = subprocess.run([exe], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.strip() == "ok"
