"""A plain C program against include/zipmoe.h and libzipmoe.so: encode, validate and plan a launch without any
Python in the path (host entry points only, so it runs without a GPU)."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_program_encodes_validates_and_plans(tmp_path):
    from paper_2601_21198_b200 import build
    build.build()
    pkg = os.path.join(ROOT, "paper_2601_21198_b200")
    exe = str(tmp_path / "launch_plan_check")
    subprocess.check_call(["gcc", "-std=c99", "-O1", "-Wall", "-I", os.path.join(ROOT, "include"),
                           os.path.join(ROOT, "tests", "csrc", "launch_plan_check.c"), "-o", exe,
                           "-L", pkg, "-l:libzipmoe.so", "-Wl,-rpath," + pkg, "-Wl,-rpath,/usr/local/cuda/lib64"])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr
