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


def test_wide_window_parts_hold_whole_tokens_and_fit_a_tile():
    """A verification window of more than 128 rows is cut into parts of whole query tokens: for every
    supported (heads per KV head, window tokens) a part has at most 128 rows, no part is empty, the
    parts cover the window, and no cut is made when the window fits one part."""
    import ctypes

    from paper_2508_16201_b200 import specvlm
    L = specvlm.lib()
    for group in range(1, 17):
        for n_q in range(1, 65):
            n_parts, q_per = ctypes.c_int32(), ctypes.c_int32()
            assert L.specvlm_debug_window_parts(n_q, group, ctypes.byref(n_parts), ctypes.byref(q_per)) == 0
            n, q = n_parts.value, q_per.value
            assert q * group <= 128, (group, n_q, n, q)
            assert (n - 1) * q < n_q <= n * q, (group, n_q, n, q)
            assert (n == 1) == (n_q * group <= 128 or n_q <= 128 // group)
            assert n == -(-n_q // (128 // group))
    assert L.specvlm_debug_window_parts(0, 8, None, None) == specvlm.ERR_INVALID_ARG
