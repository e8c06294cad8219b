"""The boundary is a C ABI: a plain-C program (gcc, no CUDA, no Python types) includes include/isv.h, loads the
library and drives a plan-only handle.  Its figures are compared with the reference cache model."""
import os
import re
import subprocess

import pytest

from oracle import kv_model as km
from paper_2504_11816_b200 import binding as B
from paper_2504_11816_b200 import build as isv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_plain_c_program_uses_the_header_and_the_library(tmp_path):
    isv_build.build()
    exe = str(tmp_path / "abi_plan_only")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "c", "abi_plan_only.c"), "-o", exe, "-ldl"], check=True)
    out = subprocess.run([exe, B.LIB_PATH], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    m = re.search(r"block_bytes=(\d+) kappa=(\d+) max_blocks=(\d+) res=(\d+) off=(\d+) chunks=(\d+) decode_rc=(-?\d+) "
                  r'err="([^"]*)"', out.stdout)
    assert m, out.stdout
    block_bytes, kappa, max_blocks, res, off, chunks, rc = (int(x) for x in m.groups()[:7])
    assert kappa == km.kv_bytes_per_token(4, 128, 2) and block_bytes == 16 * kappa and max_blocks == 7
    assert (res, off) == km.layer_step_bytes([34, 65, 2], 0.5, 16, kappa)
    assert chunks == (1 if off else 0)
    assert rc == B.ISV_ENODEVICE and "plan-only" in m.group(8)
    assert "bad_rc=-1 bad_handle=null" in out.stdout
