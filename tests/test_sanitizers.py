"""The host-only scheduler of the library and the CPU oracle under AddressSanitizer and
UndefinedBehaviorSanitizer (compute-sanitizer is not available for the kernels; their guard is the
canary and parity tests on the GPU)."""
import os
import subprocess
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_scheduler_and_oracle_are_clean_under_asan_and_ubsan():
    srcs = [os.path.join(ROOT, "tests", "sanitizer_driver.cpp"),
            os.path.join(ROOT, "paper_1509_04210_b200", "csrc", "sched.cpp"),
            os.path.join(ROOT, "oracle", "rudra_oracle.cpp")]
    with tempfile.TemporaryDirectory() as d:
        exe = os.path.join(d, "driver")
        cmd = ["g++", "-std=c++17", "-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
               "-ffp-contract=off", "-I", os.path.join(ROOT, "include"), "-o", exe] + srcs
        built = subprocess.run(cmd, capture_output=True, text=True)
        if built.returncode != 0 and "sanitize" in built.stderr:
            pytest.skip("sanitizer runtime not installed")
        assert built.returncode == 0, built.stderr
        run = subprocess.run([exe], capture_output=True, text=True, timeout=600,
                             env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1", LD_PRELOAD=""))
        assert run.returncode == 0, (run.returncode, run.stdout, run.stderr[-3000:])
        assert "sanitizer driver ok" in run.stdout
