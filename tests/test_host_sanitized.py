"""The host half of the library under -fsanitize=address,undefined: encoder, validator (on damaged and truncated
blobs), launch planner, cache-pool planner and scheduler, driven by a small C++ program."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_host_code_is_clean_under_the_sanitizers(tmp_path):
    csrc = os.path.join(ROOT, "paper_2601_21198_b200", "csrc")
    exe = str(tmp_path / "host_sanitized")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
                           "-Wall", "-I", os.path.join(ROOT, "include"), "-I", csrc,
                           os.path.join(ROOT, "tests", "csrc", "host_sanitized.cpp"),
                           os.path.join(csrc, "zipmoe_host.cpp"), os.path.join(csrc, "planner.cpp"),
                           os.path.join(csrc, "scheduler.cpp"), "-lpthread", "-o", exe])
    out = subprocess.run([exe], capture_output=True, text=True, env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1"))
    assert out.returncode == 0 and out.stdout.strip().endswith("ok"), out.stdout[-2000:] + out.stderr[-4000:]
