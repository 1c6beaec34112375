"""The oracle under AddressSanitizer and UndefinedBehaviorSanitizer (host code only): every
routine on exactly-sized heap buffers at awkward sizes.  The device has no sanitizer here, so the
checker at least is shown to stay inside its buffers and free of undefined behaviour."""
import os
import shutil
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
FLAGS = ["-O1", "-g", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fno-omit-frame-pointer",
         "-fsanitize=address,undefined", "-fno-sanitize-recover=all"]


def build(tmp_path, name, extra=()):
    exe = os.path.join(tmp_path, name)
    done = subprocess.run(["gcc", *FLAGS, *extra, os.path.join(HERE, "oracle_sanitize_driver.c"), "-o", exe, "-lm"],
                          capture_output=True, text=True)
    if done.returncode != 0 and ("asan" in done.stderr or "ubsan" in done.stderr):
        pytest.skip("this gcc has no sanitizer runtime: " + done.stderr.strip().splitlines()[-1])
    assert done.returncode == 0, done.stderr
    return exe


@pytest.mark.skipif(shutil.which("gcc") is None, reason="no gcc")
def test_oracle_is_clean_under_asan_and_ubsan(tmp_path):
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")
    env.pop("LD_PRELOAD", None)
    # the harness notices an overrun when there is one ...
    bad = subprocess.run([build(str(tmp_path), "selfcheck", ["-DKBO_SAN_SELFCHECK"])], capture_output=True,
                         text=True, env=env, timeout=120)
    assert bad.returncode != 0 and "heap-buffer-overflow" in bad.stderr and "ok" not in bad.stdout
    # ... and reports nothing on the oracle as it stands
    good = subprocess.run([build(str(tmp_path), "driver")], capture_output=True, text=True, env=env, timeout=300)
    assert good.returncode == 0, good.stderr[-2000:]
    assert "oracle_sanitize_driver: ok" in good.stdout and "runtime error" not in good.stderr
