"""Host logic of the scratch-buffer pool behind gemm_s4 (CPU only): compiled with g++ against
a fake backend, so the policy -- one buffer per stream, reuse after completion, stream-ordered
growth, no allocation during capture, no buffer held by two threads at once -- is checked
without a GPU."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_workspace_pool_policy(tmp_path):
    src = os.path.join(ROOT, "tests", "cpp", "workspace_pool_test.cpp")
    exe = str(tmp_path / "workspace_pool_test")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-pthread", "-o", exe, src])
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr
