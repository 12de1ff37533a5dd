"""The oracle's own pins once more, with the oracle compiled under AddressSanitizer and
UndefinedBehaviorSanitizer (any report aborts the run): a plain C program that indexes arenas,
bitmaps and caller buffers by hand is exactly what these two are for.  Likewise the host half
of the CUDA library (argument checks, workspace layout, the volume model), as far as it runs
without a device."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _runtime(name: str) -> str:
    path = subprocess.run(["gcc", f"-print-file-name={name}"], capture_output=True, text=True).stdout.strip()
    if not os.path.isabs(path) or not os.path.exists(path):
        pytest.skip(f"{name} not found")
    return path


def _env():
    env = dict(os.environ)
    env["LD_PRELOAD"] = _runtime("libasan.so") + ":" + _runtime("libubsan.so")
    env["ASAN_OPTIONS"] = "detect_leaks=0:abort_on_error=1"          # the interpreter itself is not leak-clean
    env["UBSAN_OPTIONS"] = "halt_on_error=1:print_stacktrace=1"
    return env


def test_oracle_pins_pass_under_asan_and_ubsan():
    from oracle import td_oracle
    td_oracle.build(sanitize=True)
    env = _env()
    env[td_oracle.SANITIZED_ENV] = "1"
    res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                          os.path.join(ROOT, "tests", "test_oracle_dock.py"),
                          os.path.join(ROOT, "tests", "test_oracle_model.py")],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert "passed" in res.stdout and "ERROR: AddressSanitizer" not in tail and "runtime error" not in tail, tail


def test_library_host_side_passes_under_asan_and_ubsan(tmp_path):
    """libtd.so built with the host compiler's sanitizers; the ABI tests that need no device
    (layout, argument checks, Eq. 1 / 2 / 4) run against it."""
    from paper_2507_19017_b200 import build as b
    out = str(tmp_path / "libtd_san.so")
    san = []
    for flag in ("-fsanitize=address", "-fsanitize=undefined", "-fno-sanitize-recover=all", "-fno-omit-frame-pointer"):
        san += ["-Xcompiler", flag]
    cmd = [b._nvcc()] + b.NVCC_FLAGS + san + ["-o", out] + [os.path.join(b.CSRC, s) for s in b.SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    env = _env()
    env["TD_LIB_PATH"] = out
    env["ASAN_OPTIONS"] += ":protect_shadow_gap=0"                    # the CUDA runtime reserves address space of its own
    res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                          os.path.join(ROOT, "tests", "test_abi.py"), os.path.join(ROOT, "tests", "test_model_bytes.py")],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert "passed" in res.stdout and "ERROR: AddressSanitizer" not in tail and "runtime error" not in tail, tail
