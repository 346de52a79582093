"""The library's host-only code (tables from a gate map, plan building, append-token, drop-evicted,
suffix-prefill tables) compiled with AddressSanitizer and UndefinedBehaviorSanitizer and run on 400
random inputs, valid and corrupted (tests/host_sanitizer_driver.cpp).  The device-side sanitizer is not
available to this project, so bounds are checked on the host before anything reaches a kernel; this
test checks that the checking code itself is clean."""
import os
import shutil
import subprocess

import pytest


def test_host_code_is_clean_under_asan_and_ubsan(repo_root, tmp_path):
    gxx = shutil.which("g++")
    if gxx is None:
        pytest.skip("no g++")
    cuda_inc = "/usr/local/cuda/include"
    exe = tmp_path / "san_driver"
    cmd = [gxx, "-O1", "-g", "-std=c++17", "-fsanitize=address,undefined", "-fno-omit-frame-pointer", "-DRKSC_BUILD",
           "-I", os.path.join(repo_root, "include"), "-I", os.path.join(repo_root, "paper_2606_09937_b200", "csrc"),
           "-I", cuda_inc, os.path.join(repo_root, "paper_2606_09937_b200", "csrc", "plan.cpp"),
           os.path.join(repo_root, "tests", "host_sanitizer_driver.cpp"), "-o", str(exe)]
    build = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    if build.returncode != 0 and "sanitize" in build.stderr.lower() and "cannot find" in build.stderr.lower():
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr[-2000:]
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=300, env=env)
    assert run.returncode == 0, (run.stdout[-1000:], run.stderr[-3000:])
    assert "plans built" in run.stdout and "runtime error" not in run.stderr and "AddressSanitizer" not in run.stderr
