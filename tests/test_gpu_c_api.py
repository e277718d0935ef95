"""The library from plain C: compile the single-chunk example against include/kdn.h with a C99 compiler, run it on the
GPU (it checks the scattered bytes itself), and read the host cost of one call."""
import os
import re
import shutil
import subprocess

import pytest

from paper_2409_13761_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_single_chunk_example_in_c(tmp_path):
    exe = build.build_example("single_chunk", str(tmp_path))
    out = subprocess.run([exe], capture_output=True, text=True, timeout=600, env=build.example_env())
    assert out.returncode == 0, out.stdout + out.stderr
    m = re.search(r"ok host_us=([0-9.]+) device_us=([0-9.]+) gbs=([0-9.]+)", out.stdout)
    assert m, out.stdout
    host_us, device_us = float(m.group(1)), float(m.group(2))
    print("one 512-token 8B chunk per call from C: host %.2f us, device %.2f us" % (host_us, device_us))
    assert host_us < 25.0                                   # a generous bound: the call is a validation and one launch
    assert device_us < 60.0
