"""Host logic of the overlapped INT4 pre-pass (CPU only): the order in which the chunks of the
int8 operand images are produced is compiled with g++ and checked to be a bijection onto the
chunks that puts the first wave's rows first, k-chunk by k-chunk."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_work_list_is_a_bijection_in_need_order(tmp_path):
    src = os.path.join(ROOT, "tests", "cpp", "s4_ahead_test.cpp")
    exe = str(tmp_path / "s4_ahead_test")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-o", exe, src])
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr
