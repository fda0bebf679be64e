"""Sanitizer and self-check runs (the stand-in for a device memory checker, which cannot run on the test machines).

CPU: the oracle's pins and the host-side ABI tests again, in a child python that has AddressSanitizer's runtime
preloaded, against builds of the oracle and of the library's host code with -fsanitize=address,undefined.
GPU: the small parity suite against the -DREKV_CHECKS build, whose kernels test their own index and address
arithmetic and report through the status word (any violation fails rekv_check_status in those tests), and the
Tiny configuration through the sanitized host code.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _child(env_extra, args, timeout=1500):
    from oracle import build as oracle_build
    env = dict(os.environ, **env_extra)
    if env_extra.get("ORACLE_SANITIZE") == "1" or env_extra.get("REKV_SANITIZE") == "1":
        env["LD_PRELOAD"] = oracle_build.sanitizer_runtime()
        # leaks: python itself never frees everything; shadow gap: the CUDA driver maps memory there
        env["ASAN_OPTIONS"] = "detect_leaks=0:protect_shadow_gap=0"
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider"] + args, cwd=ROOT, env=env,
                       capture_output=True, text=True, timeout=timeout)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-3000:])
    assert "AddressSanitizer" not in r.stderr and "runtime error" not in r.stderr, r.stderr[-3000:]
    return r.stdout


def test_oracle_pins_under_address_and_undefined_behaviour_sanitizers():
    out = _child({"ORACLE_SANITIZE": "1"}, ["tests/test_oracle_pins.py"])
    assert " passed" in out


def test_host_side_abi_under_address_and_undefined_behaviour_sanitizers():
    out = _child({"REKV_SANITIZE": "1"}, ["tests/test_abi.py", "-m", "not gpu"])
    assert " passed" in out


@pytest.mark.gpu
def test_small_parity_suite_on_the_self_checking_build():
    out = _child({"REKV_CHECKS": "1"}, ["tests/test_parity_gpu.py", "tests/test_random_shapes_gpu.py",
                                        "tests/test_attend_full_gpu.py", "tests/test_layer_mode_gpu.py", "-m", "gpu"])
    assert " passed" in out


@pytest.mark.gpu
def test_tiny_configuration_through_sanitized_host_code():
    out = _child({"REKV_SANITIZE": "1"}, ["tests/test_parity_gpu.py", "-k", "tiny or error or host_tier_small", "-m", "gpu"])
    assert " passed" in out
