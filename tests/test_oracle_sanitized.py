"""The oracle's own pins once more, with the oracle compiled under AddressSanitizer and
UndefinedBehaviorSanitizer: an out-of-range read or a signed overflow in the program every
parity claim rests on would pass the value checks by luck and show here."""
import glob
import os
import subprocess
import sys

import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_pins_under_sanitizers():
    asan = subprocess.check_output(["g++", "-print-file-name=libasan.so"], text=True).strip()
    if not os.path.isabs(asan) or not os.path.exists(asan):
        pytest.skip("this toolchain has no libasan")
    oracle.build(sanitized=True)
    files = sorted(f for f in glob.glob(os.path.join(HERE, "test_oracle_*.py")) if not f.endswith("test_oracle_sanitized.py"))
    assert len(files) >= 6
    env = dict(os.environ, LD_PRELOAD=os.path.realpath(asan), AASD_ORACLE_SANITIZED="1",
               ASAN_OPTIONS="detect_leaks=0:halt_on_error=1", UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider"] + files,
                       env=env, capture_output=True, text=True, cwd=os.path.dirname(HERE))
    out = r.stdout + r.stderr
    assert r.returncode == 0, out[-4000:]
    assert "AddressSanitizer" not in out and "runtime error" not in out, out[-4000:]
    assert " passed" in out


def test_the_sanitizers_see_the_oracles_reads():
    # the check above means something only if a stray read inside the oracle is reported: a
    # call (made here, on purpose, from a process of its own) that tells the oracle a row is
    # 64 logits longer than its buffer must end that process with AddressSanitizer's report
    asan = subprocess.check_output(["g++", "-print-file-name=libasan.so"], text=True).strip()
    if not os.path.isabs(asan) or not os.path.exists(asan):
        pytest.skip("this toolchain has no libasan")
    oracle.build(sanitized=True)
    code = ("import ctypes as C, numpy as np, oracle\n"
            "x = np.zeros(1000, np.float32); p = np.zeros(1064)\n"
            "oracle.lib().oracle_softmax_row(x.ctypes.data_as(C.c_void_p), 0, C.c_int64(0), C.c_int64(1064),\n"
            "                                C.c_int64(1064), C.c_double(1.0), p.ctypes.data_as(C.c_void_p))\n"
            "print('returned')\n")
    env = dict(os.environ, LD_PRELOAD=os.path.realpath(asan), AASD_ORACLE_SANITIZED="1",
               ASAN_OPTIONS="detect_leaks=0:halt_on_error=1")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, cwd=os.path.dirname(HERE))
    assert r.returncode != 0 and "AddressSanitizer" in r.stderr and "returned" not in r.stdout, (r.stdout + r.stderr)[-2000:]
