"""Host-side memory and undefined-behaviour checks. The CPU reference engine is rebuilt with AddressSanitizer and
UndefinedBehaviorSanitizer and the scenario, error-code and random-stream tests are run against it in a child
process (the ASan runtime has to be loaded before Python). The CUDA library's checked build (-DKVT_DEBUG: device
side index checks, another launch shape) must compile and export the same symbols; it runs in the GPU tests."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_oracle_under_asan_and_ubsan():
    asan = subprocess.run(["g++", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    if not os.path.isabs(asan) or not os.path.exists(asan):
        pytest.skip("no ASan runtime on this machine")
    env = dict(os.environ, KVT_ORACLE_SANITIZE="1", LD_PRELOAD=asan,
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=1", UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_oracle_engine.py"), os.path.join(ROOT, "tests", "test_oracle_hash.py"),
           "-k", "scenario or error_codes or mixed_pool or hash_matches or parallel or pinned"]
    r = subprocess.run(cmd, env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-3000:])
    assert "passed" in r.stdout


def test_checked_build_of_the_cuda_library_exports_the_same_symbols():
    import ctypes
    from paper_2609_39819_b200 import binding, build
    lib = ctypes.CDLL(build.build_debug_lib())
    for name in binding.EXPORTS:
        assert hasattr(lib, name), name
