"""The boundary used the way a C program uses it: tests/c_abi/smoke.c is compiled with gcc
against include/oilbird.h and liboilbird.so (plus the CUDA runtime for its buffers) and run
as a process of its own; no Python object touches the library."""
import os
import shutil
import subprocess

import pytest

from paper_2608_03839_b200 import build as libbuild

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_program_through_the_c_abi(tmp_path):
    lib = libbuild.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = str(tmp_path / "smoke")
    cc = shutil.which("gcc")
    assert cc, "gcc not found"
    subprocess.run([cc, "-O1", "-std=c11", "-o", exe, os.path.join(ROOT, "tests", "c_abi", "smoke.c"),
                    "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                    "-L", os.path.dirname(lib), "-loilbird", "-L", os.path.join(cuda, "lib64"),
                    "-lcudart", "-lm", f"-Wl,-rpath,{os.path.dirname(lib)}",
                    f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"], check=True)
    r = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == "ok", (r.returncode, r.stdout, r.stderr)
