"""The C oracle under AddressSanitizer and UndefinedBehaviorSanitizer (host only): a harness with
exactly-sized heap buffers runs every oracle routine on small ragged shapes; any access outside a
buffer or undefined arithmetic makes the sanitized build exit non-zero.  The same harness built
without sanitizers must print the same checksum."""
import os
import shutil
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = [os.path.join(HERE, "oracle_sanitize_main.c"), os.path.join(ROOT, "oracle", "mustdrop_oracle.c")]
FLAGS = ["-O1", "-g", "-std=c11", "-ffp-contract=off", "-fno-fast-math"]


def _build(tmp_path, name, extra):
    exe = str(tmp_path / name)
    subprocess.check_call(["gcc"] + FLAGS + extra + ["-o", exe] + SRC + ["-lm"])
    return exe


@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_oracle_is_clean_under_address_and_undefined_behaviour_sanitizers(tmp_path):
    plain = _build(tmp_path, "plain", [])
    try:
        san = _build(tmp_path, "san", ["-fsanitize=address,undefined", "-fno-sanitize-recover=all"])
    except subprocess.CalledProcessError:
        pytest.skip("this gcc has no sanitizer runtime")
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")
    a = subprocess.run([plain], capture_output=True, text=True)
    b = subprocess.run([san], capture_output=True, text=True, env=env)
    assert a.returncode == 0, a.stderr
    assert b.returncode == 0, b.stdout + b.stderr
    assert a.stdout == b.stdout and a.stdout.startswith("checksum ")
