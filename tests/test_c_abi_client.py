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
