"""The oracle under AddressSanitizer and UndefinedBehaviorSanitizer (gcc): exact-size
buffers, ragged lengths, all result codes.  Skipped if gcc has no sanitizer runtime."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_oracle_is_clean_under_asan_and_ubsan(tmp_path):
    exe = tmp_path / "oracle_san"
    cmd = ["gcc", "-std=c11", "-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
           os.path.join(ROOT, "tests", "c", "oracle_sanitizer_driver.c"), os.path.join(ROOT, "oracle", "gk_oracle.c"),
           os.path.join(ROOT, "oracle", "gk_sha256_oracle.c"),
           "-o", str(exe)]
    build = subprocess.run(cmd, capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr:
        pytest.skip("gcc without sanitizer runtime")
    assert build.returncode == 0, build.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120,
                         env={**os.environ, "ASAN_OPTIONS": "detect_leaks=1"})
    assert run.returncode == 0, run.stdout + run.stderr
    assert "clean" in run.stdout
