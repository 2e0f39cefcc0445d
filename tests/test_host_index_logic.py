"""The index arithmetic shared by the host entry points and the kernels (block order, spill block
numbering, tiles of a group; csrc/s2a_params.h), checked exhaustively on small shapes by a host-only C++
program: the persistent kernels take their work items and their spill addresses from these functions."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "host", "index_logic.cpp")
CSRC = os.path.join(ROOT, "paper_2309_12307_b200", "csrc")
CUDA_INC = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "include")


@pytest.mark.skipif(shutil.which("g++") is None or not os.path.isdir(CUDA_INC), reason="needs g++ and the CUDA headers")
def test_block_order_spill_blocks_and_group_tiles(tmp_path):
    exe = str(tmp_path / "index_logic")
    subprocess.run(["g++", "-std=c++17", "-O1", "-I", CSRC, "-I", CUDA_INC, SRC, "-o", exe], check=True)
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr
