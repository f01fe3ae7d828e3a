"""The N > 1 part of bench.py on CPU: two gloo ranks run the benchmark's rank-reduction (each rank
is an independent replica of the path; step time = the slowest rank's; value = all replicas' bytes
over that time) and its reference arm's rule that only rank 0 prints."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_ranks(code, world=2):
    procs, port = [], _free_port()
    for r in range(world):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE=str(world), LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), PYTHONPATH=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    return [o for o, _ in outs]


def test_max_over_ranks_and_whole_job_value_gloo():
    code = textwrap.dedent("""
        import os, json, torch, torch.distributed as dist
        import bench
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo", rank=rank, world_size=world)
        mine = [10.0 + rank, 2.0 - rank]              # rank 1 is slower on the first, faster on the second
        dist.barrier()
        total, attn = bench.max_over_ranks(mine, world, torch.device("cpu"))
        print(json.dumps({"rank": rank, "total": total, "attn": attn,
                          "value": bench.replicas_value(4.0e9, attn, world)}))
        dist.barrier()
        dist.destroy_process_group()
    """)
    outs = [json.loads(o.strip().splitlines()[-1]) for o in _run_ranks(code)]
    for o in outs:
        assert o["total"] == 11.0 and o["attn"] == 2.0          # the same maxima on every rank
        assert abs(o["value"] - 2 * 4.0e9 / 2.0e-3 / 1e9) < 1e-6  # two replicas' bytes over the slowest time


def test_reference_arm_prints_on_rank_0_only():
    base = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
            "--warmup", "0"]
    env1 = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r1 = subprocess.run(base, env=env1, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    r0 = subprocess.run(base, env=env0, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r0.returncode == 0, r0.stderr[-2000:]
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
