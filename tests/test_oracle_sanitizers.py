"""The CPU oracle under AddressSanitizer and UndefinedBehaviorSanitizer: a small C driver links
the oracle's source with -fsanitize=address,undefined and runs 40 random problems (both wire
orders, windowed layers, empty requests). Any out-of-bounds access, overflow or misaligned
access in the oracle's loops ends the run with a non-zero exit code."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_oracle_runs_clean_under_asan_and_ubsan(tmp_path):
    if shutil.which("gcc") is None:
        pytest.skip("gcc not available")
    exe = tmp_path / "oracle_sanitized"
    cmd = ["gcc", "-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
           "-I", os.path.join(ROOT, "oracle"), "-o", str(exe),
           os.path.join(ROOT, "tests", "native", "oracle_sanitize_driver.c"),
           os.path.join(ROOT, "oracle", "topkv_oracle.c"), "-lpthread"]
    build = subprocess.run(cmd, capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr:
        pytest.skip("sanitizer runtime not installed: " + build.stderr[-200:])
    assert build.returncode == 0, build.stderr[-2000:]
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0")
    run = subprocess.run([str(exe)], capture_output=True, text=True, env=env, timeout=300)
    assert run.returncode == 0, (run.stdout[-1000:], run.stderr[-3000:])
    assert "sanitized oracle ok" in run.stdout


def test_host_shims_run_clean_under_asan_and_ubsan(tmp_path):
    """The CUDA-free part of the library (validator, size bookkeeping, header, host CRC-64,
    retry, analytic helpers) built from its own source with the sanitizers and driven with 200
    random layouts and tables."""
    if shutil.which("g++") is None or shutil.which("gcc") is None:
        pytest.skip("gcc / g++ not available")
    flags = ["-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
             "-I", os.path.join(ROOT, "include")]
    obj_c, obj_cpp, exe = tmp_path / "driver.o", tmp_path / "host.o", tmp_path / "host_sanitized"
    steps = [["gcc", "-std=c99", *flags, "-c", os.path.join(ROOT, "tests", "native",
                                                          "host_shims_sanitize_driver.c"), "-o", str(obj_c)],
             ["g++", "-std=c++17", *flags, "-c", os.path.join(ROOT, "paper_2607_28633_b200", "csrc",
                                                            "topkv_host.cpp"), "-o", str(obj_cpp)],
             ["g++", "-fsanitize=address,undefined", str(obj_c), str(obj_cpp), "-o", str(exe), "-lpthread"]]
    for cmd in steps:
        build = subprocess.run(cmd, capture_output=True, text=True)
        if build.returncode != 0 and "sanitize" in build.stderr:
            pytest.skip("sanitizer runtime not installed: " + build.stderr[-200:])
        assert build.returncode == 0, build.stderr[-2000:]
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0")
    run = subprocess.run([str(exe)], capture_output=True, text=True, env=env, timeout=300)
    assert run.returncode == 0, (run.returncode, run.stdout[-1000:], run.stderr[-3000:])
    assert "sanitized host shims ok" in run.stdout

