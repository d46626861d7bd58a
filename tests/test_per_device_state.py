"""The library keeps launch state that belongs to a device (a kernel's dynamic shared-memory limit, the
multiprocessor count) per device ordinal.  The cache logic is plain C++ and is checked here behind fake
device ordinals, compiled with the host compiler: no GPU and no CUDA runtime involved."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_per_device_cache_logic(tmp_path):
    exe = tmp_path / "per_device_check"
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-Wall", "-Wextra", "-Werror", "-pthread",
                           "-I", os.path.join(ROOT, "paper_2505_19115_b200", "csrc"),
                           os.path.join(ROOT, "tests", "native", "per_device_check.cpp"), "-o", str(exe)])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr


def test_no_process_wide_launch_flags_left_in_the_sources():
    # every cudaFuncSetAttribute goes through the per-device helper
    csrc = os.path.join(ROOT, "paper_2505_19115_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        text = open(os.path.join(csrc, name)).read()
        assert "static bool attr_set" not in text, name
        if name != "common.cuh":
            assert "cudaFuncSetAttribute" not in text, name
