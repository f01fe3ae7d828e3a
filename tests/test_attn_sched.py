"""Host logic of the attention kernel: the slice / segment / scratch-slot arithmetic of
csrc/attn_sched.h, compiled for the host and checked by brute force (coverage of every tile exactly
once, balance, at most two partial segments per CTA, slot and part-count consistency)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))


def test_attention_work_partition(tmp_path):
    exe = tmp_path / "attn_sched_check"
    subprocess.run(["g++", "-O1", "-std=c++17", "-o", str(exe), os.path.join(HERE, "native", "attn_sched_check.cpp")],
                   check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr
