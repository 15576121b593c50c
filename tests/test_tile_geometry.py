"""The piece arithmetic of the decode kernels (how many bytes of a tile's sign+mantissa section each bulk copy
moves) is plain C++ shared by host and device; this compiles it with g++ and checks it for every tile size, so a
copy that would read past a short last tile shows up without a GPU."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_sign_mantissa_pieces_cover_the_tile_and_nothing_else(tmp_path):
    exe = str(tmp_path / "tile_geometry_check")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-Wall", "-I", os.path.join(ROOT, "paper_2601_21198_b200", "csrc"),
                           os.path.join(ROOT, "tests", "csrc", "tile_geometry_check.cpp"), "-o", exe])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout
