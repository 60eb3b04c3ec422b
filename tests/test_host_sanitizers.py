"""AddressSanitizer + UndefinedBehaviorSanitizer over the CPU oracle.

The device-side memory checker is not available for the kernels, so the kernels are guarded by canary
words, odd sizes and the comparison with the oracle; the oracle that all of that leans on is itself
run here under the host sanitizers, on tiny problems with buffers of exactly the documented sizes.
"""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SAN = ["-fsanitize=address,undefined", "-fno-sanitize-recover=all", "-fno-omit-frame-pointer"]


def build_and_run(tmp_path, extra_flags=()):
    exe = str(tmp_path / "oracle_sanitized")
    cmd = ["g++", "-std=c++17", "-O1", "-g", "-ffp-contract=off", *SAN, *extra_flags,
           os.path.join(ROOT, "tests", "sanitizer_driver.cpp"), os.path.join(ROOT, "oracle", "signsgd_ref.cpp"),
           "-o", exe]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    if res.returncode != 0 and "sanitize" in res.stderr and "cannot find" in res.stderr:
        pytest.skip("the sanitizer runtime libraries are not installed")
    assert res.returncode == 0, res.stderr
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")
    return subprocess.run([exe], capture_output=True, text=True, timeout=600, env=env)


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs g++")
def test_oracle_is_clean_under_asan_and_ubsan(tmp_path):
    run = build_and_run(tmp_path)
    assert run.returncode == 0, run.stdout + run.stderr
    assert "all cases ran" in run.stdout
    assert "runtime error" not in run.stderr and "AddressSanitizer" not in run.stderr


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs g++")
def test_the_sanitizer_run_does_catch_a_planted_overrun(tmp_path):
    # the same driver with the gradient buffer one element short at d = 33: the run must now fail, which shows
    # that a clean run above means something
    src = open(os.path.join(ROOT, "tests", "sanitizer_driver.cpp")).read()
    planted = src.replace("Tight<float> g(M * ld)", "Tight<float> g(M * ld - (d == 33 ? 1 : 0))")
    assert planted != src
    drv = tmp_path / "planted.cpp"
    drv.write_text(planted)
    exe = str(tmp_path / "planted")
    res = subprocess.run(["g++", "-std=c++17", "-O1", "-g", *SAN, str(drv),
                          os.path.join(ROOT, "oracle", "signsgd_ref.cpp"), "-o", exe],
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=600)
    assert run.returncode != 0 and "AddressSanitizer" in run.stderr


@pytest.mark.skipif(shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"), reason="needs nvcc")
def test_host_argument_checks_are_clean_under_asan_and_ubsan(tmp_path):
    """The CUDA library's host layer (argument checks, size arithmetic, the warm-up length scan) built with the
    host sanitizers and driven through every entry point's rejection and empty-input paths; runs without a GPU
    because none of these calls may reach a launch."""
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    csrc = os.path.join(ROOT, "paper_1802_04434_b200", "csrc")
    exe = str(tmp_path / "abi_sanitized")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O1", "-std=c++17", "--fmad=false",
           "-I", os.path.join(ROOT, "include"),
           "-Xcompiler", "-fsanitize=address", "-Xcompiler", "-fsanitize=undefined",
           "-Xcompiler", "-fno-sanitize-recover=all",
           *[os.path.join(csrc, n) for n in ("signsgd.cu", "variants.cu", "stats.cu", "exchange.cu", "vote_staged.cu")],
           os.path.join(ROOT, "tests", "sanitizer_abi_driver.cpp"), "-o", exe]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    # the CUDA runtime reserves address ranges that ASan's shadow-gap protection would refuse
    env = dict(os.environ, ASAN_OPTIONS="protect_shadow_gap=0:detect_leaks=0", UBSAN_OPTIONS="print_stacktrace=1")
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300, env=env)
    assert run.returncode == 0, run.stdout + run.stderr[-2000:]
    assert "all checks passed" in run.stdout
    assert "runtime error" not in run.stderr and "AddressSanitizer" not in run.stderr
