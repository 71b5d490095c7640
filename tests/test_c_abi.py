"""The library used from plain C: compiles tests/c_abi_smoke.c against include/iso.h with gcc
(-std=c99 -pedantic) and runs it; no Python binding and no GPU involved."""
import os
import subprocess

from paper_1606_07676_b200 import binding as iso

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_header_is_c_and_host_entry_points_work(tmp_path):
    iso.load_library()
    exe = tmp_path / "c_abi_smoke"
    libdir = os.path.dirname(iso.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           os.path.join(ROOT, "tests", "c_abi_smoke.c"), "-o", str(exe),
                           "-L", libdir, "-l:" + iso.LIB_NAME, "-Wl,-rpath," + libdir])
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and "c abi ok" in out.stdout, out.stdout + out.stderr
