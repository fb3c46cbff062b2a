"""The transform core of the CUDA library, compiled for the CPU and run thread by thread
against the definition of the negacyclic transform (no GPU, no oracle): index arithmetic,
both limb arithmetics and the range bounds the double-precision arithmetic relies on."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_transform_core_on_the_host(tmp_path):
    exe = str(tmp_path / "host_transform_check")
    csrc = os.path.join(ROOT, "paper_2303_10837_b200", "csrc")
    cmd = ["g++", "-O2", "-std=gnu++17", "-ffp-contract=off", "-o", exe,
           os.path.join(ROOT, "tests", "host_transform_check.cpp"), os.path.join(csrc, "fedhe_host.cpp"),
           "-lquadmath"]
    build = subprocess.run(cmd, capture_output=True, text=True)
    assert build.returncode == 0, build.stderr[-4000:]
    run = subprocess.run([exe], capture_output=True, text=True, timeout=600)
    assert run.returncode == 0 and run.stdout.strip().endswith("ok"), run.stdout[-2000:] + run.stderr[-2000:]
