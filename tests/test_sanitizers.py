"""AddressSanitizer and UndefinedBehaviorSanitizer builds (CPU only): the
oracle, with every function driven by a small C program on empty,
single-element, ragged and multi-bucket inputs in allocations exactly as large
as the ranges; and the host side of the CUDA library (layout arithmetic, slot
map, state machine, argument checks), walked at random in dry-run mode."""
from __future__ import annotations

import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_oracle_is_clean_under_asan_and_ubsan(tmp_path):
    exe = tmp_path / "sanitize_driver"
    cmd = ["gcc", "-O1", "-g", "-std=c99", "-ffp-contract=off", "-fsanitize=address,undefined",
           "-fno-sanitize-recover=all", "-fno-omit-frame-pointer",
           os.path.join(ROOT, "tests", "sanitize_driver.c"), os.path.join(ROOT, "oracle", "so_oracle.c"),
           "-o", str(exe), "-lm"]
    build = subprocess.run(cmd, capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr.lower() and "cannot find" in build.stderr.lower():
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")
    env.pop("LD_PRELOAD", None)
    run = subprocess.run([str(exe)], capture_output=True, text=True, env=env, timeout=300)
    assert run.returncode == 0, run.stdout + run.stderr
    assert run.stdout.strip().endswith("sanitized ok"), run.stdout + run.stderr


@pytest.mark.skipif(shutil.which("gcc") is None or shutil.which("nvcc") is None
                    and not os.path.exists("/usr/local/cuda/bin/nvcc"), reason="needs gcc and nvcc")
def test_library_host_code_is_clean_under_asan_and_ubsan(tmp_path):
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    inc = os.path.join(ROOT, "include")
    csrc = os.path.join(ROOT, "paper_2509_21271_b200", "csrc")
    lib = tmp_path / "libso_sanitized.so"
    san = "-fPIC,-fsanitize=address,-fsanitize=undefined,-fno-sanitize-recover=all,-fno-omit-frame-pointer"
    build = subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O1", "-g", "-std=c++17",
                            "--fmad=false", "-Xcompiler", san, "-shared", "-I", inc, "-I", csrc,
                            "-o", str(lib), os.path.join(csrc, "superoffload.cu"),
                            os.path.join(csrc, "so_static_check.cu"), "-lasan", "-lubsan"],
                           capture_output=True, text=True)
    if build.returncode != 0 and "cannot find -lasan" in build.stderr:
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr[-3000:]
    exe = tmp_path / "sanitize_host_driver"
    subprocess.run(["gcc", "-std=c99", "-O1", "-g", "-fsanitize=address,undefined",
                    "-fno-sanitize-recover=all", "-I", inc,
                    os.path.join(ROOT, "tests", "sanitize_host_driver.c"), "-o", str(exe),
                    "-L", str(tmp_path), "-lso_sanitized", f"-Wl,-rpath,{tmp_path}"], check=True)
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:protect_shadow_gap=0", UBSAN_OPTIONS="print_stacktrace=1")
    env.pop("LD_PRELOAD", None)
    run = subprocess.run([str(exe)], capture_output=True, text=True, env=env, timeout=600)
    assert run.returncode == 0, run.stdout[-2000:] + run.stderr[-4000:]
    assert run.stdout.strip().endswith("sanitized ok"), run.stdout + run.stderr
