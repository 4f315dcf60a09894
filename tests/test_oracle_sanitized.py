"""The oracle's pins once more, over a build of ``oracle/dodo_oracle.c`` instrumented with
AddressSanitizer and UndefinedBehaviorSanitizer (gcc): every array access and every arithmetic step the
pins drive through the oracle is checked for out-of-bounds reads and writes, signed overflow, bad shifts
and misaligned or null pointer use.  This stands in, on the CPU side, for the device-side memory checker
that cannot be run on the shared GPUs.  Runs in a child process because the sanitizer runtime has to be
loaded before the interpreter starts.
"""
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def _runtime(name):
    out = subprocess.run(["gcc", f"-print-file-name={name}"], capture_output=True, text=True).stdout.strip()
    return out if os.path.isabs(out) and os.path.exists(out) else None


def test_oracle_pins_pass_under_address_and_ub_sanitizers():
    asan = _runtime("libasan.so")
    if asan is None:
        pytest.skip("gcc's sanitizer runtime is not installed")
    env = dict(os.environ, LD_PRELOAD=asan, ASAN_OPTIONS="detect_leaks=0:abort_on_error=0",
               UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1", DODO_ORACLE_SANITIZE="1")
    cmd = [sys.executable, "-m", "pytest", str(ROOT / "tests" / "test_oracle_pins.py"), "-x", "-q",
           "-p", "no:cacheprovider"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=900, cwd=str(ROOT), env=env)
    tail = (r.stdout + r.stderr)[-3000:]
    assert r.returncode == 0, tail
    assert "passed" in r.stdout and "runtime error" not in r.stderr and "AddressSanitizer" not in r.stderr, tail
