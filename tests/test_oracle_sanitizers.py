"""The CPU oracle under AddressSanitizer and UndefinedBehaviorSanitizer.

The oracle is what every parity claim rests on, so its own memory and arithmetic hygiene is
checked too: oracle/sbc_oracle.c is compiled together with a small C driver with
``-fsanitize=address,undefined -fno-sanitize-recover=all`` and run over a few dozen seeded cases
(tiny and ragged sizes, all-zero and tie-heavy tensors, a carried residual).  Any out-of-bounds
access, use of uninitialised stack memory the sanitizers see, signed overflow or invalid shift
ends the run with a non-zero exit code."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_oracle_runs_clean_under_asan_and_ubsan(tmp_path):
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc")
    exe = tmp_path / "oracle_sanitize"
    build = subprocess.run(
        [gcc, "-O1", "-g", "-std=c11", "-Wall", "-Wextra", "-ffp-contract=off", "-fno-fast-math",
         "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
         "-o", str(exe), os.path.join(ROOT, "tests", "sanitize", "oracle_sanitize_driver.c"),
         os.path.join(ROOT, "oracle", "sbc_oracle.c"), "-lm"],
        capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr and "cannot find" in build.stderr:
        pytest.skip("the sanitizer runtimes are not installed")
    assert build.returncode == 0, build.stderr
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")
    run = subprocess.run([str(exe)], capture_output=True, text=True, env=env, timeout=600)
    assert run.returncode == 0, run.stdout + run.stderr
    assert "clean" in run.stdout
