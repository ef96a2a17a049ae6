"""Builds tests/c_abi_client.c as strict C99 against include/gms.h, links it with libgms.so and runs it
(no GPU needed: it only makes host-only calls).  A header that is not valid C, a declared function
the library does not export, or a host-side regression visible from C fails here."""
import os
import shutil
import subprocess

import pytest

from paper_2609_25451_b200 import build as gms_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_c99_client_links_every_declared_symbol_and_runs(tmp_path):
    lib = gms_build.build()
    exe = tmp_path / "c_abi_client"
    cmd = ["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror",
           "-I", os.path.join(ROOT, "include"), os.path.join(ROOT, "tests", "c_abi_client.c"),
           "-o", str(exe), "-L", os.path.dirname(lib), "-lgms", "-Wl,-rpath," + os.path.dirname(lib)]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "c abi client: ok" in r.stdout


@pytest.mark.gpu
@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_c_program_restore_digest_verify_parity_without_python_or_torch(tmp_path, oracle):
    """tests/c_abi_gpu_parity.c: device memory from the CUDA runtime, the library through gms.h, the oracle
    through its C functions; destination bytes, digests and the mismatch list compared bit for bit."""
    from oracle import gms_oracle

    lib = gms_build.build()
    olib = gms_oracle.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = tmp_path / "c_abi_gpu_parity"
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-O1",
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
           os.path.join(ROOT, "tests", "c_abi_gpu_parity.c"), "-o", str(exe),
           "-L", os.path.dirname(lib), "-lgms", "-Wl,-rpath," + os.path.dirname(lib),
           olib, "-Wl,-rpath," + os.path.dirname(olib),
           "-L", os.path.join(cuda, "lib64"), "-lcudart", "-Wl,-rpath," + os.path.join(cuda, "lib64")]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "c abi gpu parity: ok" in r.stdout
