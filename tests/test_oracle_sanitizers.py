"""The oracle under AddressSanitizer and UndefinedBehaviorSanitizer (host code only, no GPU)."""
import os
import subprocess
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_oracle_under_asan_ubsan():
    with tempfile.TemporaryDirectory() as d:
        exe = os.path.join(d, "selftest")
        cmd = ["gcc", "-O1", "-g", "-std=c99", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
               "-o", exe, os.path.join(ROOT, "oracle", "selftest.c"), os.path.join(ROOT, "oracle", "avsg_oracle.c")]
        built = subprocess.run(cmd, capture_output=True, text=True)
        if built.returncode != 0 and "sanitize" in built.stderr:
            pytest.skip("this toolchain has no sanitizer runtime")
        assert built.returncode == 0, built.stderr
        env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0")
        run = subprocess.run([exe], capture_output=True, text=True, env=env, timeout=300)
        assert run.returncode == 0, (run.returncode, run.stdout[-500:], run.stderr[-2000:])
        assert "oracle selftest ok" in run.stdout
