"""The CPU oracle under AddressSanitizer and UndefinedBehaviorSanitizer: every entry point on small, odd shapes
with exactly sized buffers (tests/oracle_sanitize_driver.cpp).  The oracle is what every GPU parity test
trusts; an out-of-bounds read in it would go unnoticed otherwise."""
import os
import shutil
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_is_clean_under_asan_and_ubsan(tmp_path):
    gxx = shutil.which("g++")
    if gxx is None:
        pytest.skip("no g++")
    exe = str(tmp_path / "oracle_san")
    build = subprocess.run([gxx, "-std=c++17", "-O1", "-g", "-ffp-contract=off", "-fsanitize=address,undefined",
                            "-fno-sanitize-recover=all", "-o", exe, os.path.join(HERE, "oracle_sanitize_driver.cpp")],
                           capture_output=True, text=True, timeout=300)
    if build.returncode != 0 and ("asan" in build.stderr.lower() or "ubsan" in build.stderr.lower()):
        pytest.skip("sanitizer runtime not installed: " + build.stderr[-200:])
    assert build.returncode == 0, build.stderr[-2000:]
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300,
                         env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1", UBSAN_OPTIONS="print_stacktrace=1"))
    assert run.returncode == 0 and "oracle sanitizer run ok" in run.stdout, (run.stdout[-1000:], run.stderr[-3000:])
