#!/usr/bin/env python
"""Benchmark of the SpecVLM pruned-draft speculative-decoding hot path on B200.

One step = one pass of the whole hot path over the LLaVA-OneVision-72B / 7B shaped workload
(6272 video + 128 text tokens, batch 1):
    token-rating row LSE -> token rating -> select -> gather -> gamma x draft decode attention
    -> verify attention -> accept.
The headline value is the K/V bandwidth of the memory-bound attention calls (draft decode over the
pruned cache + verification over the full cache): K/V bytes they must read once / their device
time.  Prune time (rating + select, gather listed apart) and every call's time are reported too.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

`--impl reference` times the CPU oracle (the plain fp64 restatement of the method) on the host
cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "draft-decode + verify attention KV GB/s"
UNIT = "GB/s"
HBM_NOMINAL_GBS = 8000.0
EX2_PER_CLK_PER_SM = 16                   # special-function units: base-2 exponentials per clock per SM


def ex2_peak_gops(n_sms, sm_max_mhz):
    """Exponentials per ns of the whole GPU at its maximum SM clock."""
    return EX2_PER_CLK_PER_SM * n_sms * sm_max_mhz * 1e-3


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d["bf16_tflops_sustained"]),
                "sm_max_mhz": float(d.get("sm_max_mhz", 0) or 0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 0.0,
            "source": "fallback"}


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures
# summarised under profiles/; None where no capture of that launch exists.  Each capture ran a
# subset of the layers (a many-pass capture has to stay small) and is scaled to the layers one
# launch processes: traffic is proportional to the layers streamed.  verify: 216.0 MB for 8 of 80 layers; rating
# passes: 155.8 MB and 153.3 MB for 10 of 80 layers; decode: 43.5 MB, captured whole.
NCU_TRAFFIC_BYTES = {"verify": 216.0e6 * 10, "decode": 43.5e6, "scores_colsum": 153.3e6 * 8, "scores_lse": 155.8e6 * 8}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs.  Every sample carries
    nvidia-smi's own timestamp; `stop(t0, t1)` keeps the samples taken between the two host wall-clock
    times that bracket the timed region (all samples if none fell inside: a region of a few tens of
    milliseconds can slip between two samples; the samples within 50 ms of it are tried first)."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    @staticmethod
    def _when(stamp):
        import datetime
        try:
            return datetime.datetime.strptime(stamp, "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, t0=None, t1=None):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        parsed = []
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                parsed.append((self._when(r[0]), float(r[1]), float(r[2]), r[4:8]))
            except ValueError:
                continue
        inside = [x for x in parsed if t0 is not None and x[0] is not None and t0 <= x[0] <= t1]
        if not inside and t0 is not None:       # nearest neighbours of a region shorter than the sampling interval
            inside = [x for x in parsed if x[0] is not None and t0 - 0.05 <= x[0] <= t1 + 0.05]
        use = inside or parsed
        sm, mx, reasons = [x[1] for x in use], [x[2] for x in use], set()
        for x in use:
            for name, val in zip(names, x[3]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "samples_inside_timed_region": len(inside), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
def ctypes_byref(cache):
    return ctypes.byref(cache.struct)


def max_over_ranks(times_ms, world, device):
    """Each rank runs an independent replica of the path (it does not shard: no data-path
    collective); the job's time for a step is the slowest rank's."""
    if world <= 1:
        return [float(t) for t in times_ms]
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def replicas_value(bytes_per_replica, ms, world):
    """Whole-job K/V GB/s: every replica moved `bytes_per_replica` in the slowest rank's time."""
    return world * bytes_per_replica / (ms * 1e-3) / 1e9


class GraphTimer:
    """Times a call the way the headline is timed: the call (its C-ABI entry point with every
    launch and memset it makes) is captured once into a CUDA graph and the graph is replayed;
    CUDA events bracket each replay on the replaying stream.  With `flush`, a buffer larger than
    the L2 cache is overwritten and then read back before every replay (outside the event pair), so
    that a call whose inputs would fit in L2 still reads them from HBM.  The read-back matters: after
    a write alone the L2 is full of dirty lines whose write-back then competes with the timed call's
    own reads (a 367 MB decode call measured 67 us behind a write-only flush, 55 us behind this one)."""

    def __init__(self, device, eager=False, flush_mb=512):
        import torch
        self.torch, self.eager = torch, eager
        self.side = torch.cuda.Stream()
        self.flush_buf = torch.empty(flush_mb << 20, dtype=torch.uint8, device=device)

    def flush(self):
        self.flush_buf.zero_()
        self.flush_buf.view(self.torch.int32).sum()

    def prepare(self, fn, warm=3):
        torch = self.torch
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        if self.eager:
            return fn
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(self.side):
            with torch.cuda.graph(g, stream=self.side):
                fn()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        return g.replay

    def time(self, fn, reps=20, warm=3, flush=True, prepared=False):
        """Median and minimum device time of `fn` in microseconds."""
        torch = self.torch
        run = fn if prepared else self.prepare(fn, warm)
        ts = []
        for _ in range(reps):
            if flush:
                self.flush()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            run()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3)
        return statistics.median(ts), min(ts)


def sd_projection(tau, gamma, t_draft, t_target, t_verify):
    """Speed-up of speculative decoding over plain target decoding by the paper's latency model
    (Section 3.1, Eq. 1-3): tau / (gamma * T_d / T_t + T_t^gamma / T_t)."""
    return tau / (gamma * t_draft / t_target + t_verify / t_target)


def build_inputs(w, device, n_copies):
    """Synthetic tensors of the workload, resident on the device."""
    import torch
    from paper_2508_16201_b200 import specvlm, synth
    D, nv, nt, g1 = w.head_dim, w.n_video(), w.n_text[0], w.gamma + 1
    n_t = nv + nt + g1                      # verifier cache incl. the gamma+1 new tokens
    inp = {}
    tk = synth.randn_bf16((w.t_layers, 1, w.t_kv_heads, n_t, D), device, 0, "tK")
    tv = synth.randn_bf16((w.t_layers, 1, w.t_kv_heads, n_t, D), device, 0, "tV")
    q_text = synth.randn_bf16((w.t_layers, nt, w.t_q_heads, D), device, 0, "Qtext")
    synth.plant_salient_(tk[:, 0, :, :nv, :], q_text, synth.salient_set(nv, w.planted_permille, 0))
    lens_t = torch.tensor([n_t], dtype=torch.int32, device=device)
    inp["tcache"] = specvlm.KvCache(tk, tv, lens_t, n_t)
    # rating reads the prompt part only (the same memory, shorter length bound)
    inp["tcache_prompt"] = specvlm.KvCache(tk, tv, torch.tensor([nv + nt], dtype=torch.int32, device=device),
                                           nv + nt)
    inp["q_text"] = q_text
    # draft: full-length cache (gather source) and gamma+1 pruned copies (copy 0 = gather target)
    n_d = nv + nt
    sk = synth.randn_bf16((w.d_layers, 1, w.d_kv_heads, n_d, D), device, 0, "dK")
    sv = synth.randn_bf16((w.d_layers, 1, w.d_kv_heads, n_d, D), device, 0, "dV")
    inp["dsrc"] = specvlm.KvCache(sk, sv, torch.tensor([n_d], dtype=torch.int32, device=device), n_d)
    n_p = w.k_total() + nt
    lens_p = torch.tensor([n_p], dtype=torch.int32, device=device)
    inp["dpruned"] = []
    for c in range(n_copies + 1):
        pk = torch.zeros((w.d_layers, 1, w.d_kv_heads, n_p, D), dtype=torch.bfloat16, device=device)
        pv = torch.zeros_like(pk)
        inp["dpruned"].append(specvlm.KvCache(pk, pv, lens_p, n_p))
    inp["q_dec"] = [synth.randn_bf16((w.d_layers, 1, w.d_q_heads, D), device, 0, "Qd", c) for c in range(w.gamma)]
    inp["q_ver"] = synth.randn_bf16((w.t_layers, 1, g1, w.t_q_heads, D), device, 0, "Qv")
    inp["logits"], inp["drafts"] = synth.logits_and_drafts(1, w.gamma, w.vocab, device, 0)
    return inp


class Path:
    """Pre-allocated outputs / workspaces and the sequence of C-ABI calls of one step."""

    def __init__(self, w, inp, device):
        import torch
        from paper_2508_16201_b200 import specvlm
        self.w, self.inp, self.sv, self.torch = w, inp, specvlm, torch
        D, nv, nt = w.head_dim, w.n_video(), w.n_text[0]
        self.scale = 1.0 / math.sqrt(D)
        self.kt, self.k1 = w.k_total(), w.k_stage1()
        self.row_lse = torch.empty((w.t_layers, nt, w.t_q_heads), dtype=torch.float32, device=device)
        self.scores = torch.empty(nv, dtype=torch.float32, device=device)
        self.ws_scores = torch.empty(specvlm.stage1_scores_workspace_bytes(inp["tcache_prompt"], [0, nt], [nv],
                                                                           w.t_q_heads),
                                     dtype=torch.uint8, device=device)
        self.kept = torch.empty(self.kt, dtype=torch.int32, device=device)
        self.o_dec = [torch.empty_like(q) for q in inp["q_dec"]]
        self.ws_dec = torch.empty(max(256, specvlm.attn_workspace_bytes(inp["dpruned"][0], 1, w.d_q_heads, 0)),
                                  dtype=torch.uint8, device=device)
        self.o_ver = torch.empty_like(inp["q_ver"])
        self.ws_ver = torch.empty(max(256, specvlm.attn_workspace_bytes(inp["tcache"], 1, w.t_q_heads, w.gamma)),
                                  dtype=torch.uint8, device=device)
        self.acc = (torch.empty(1, dtype=torch.int32, device=device),
                    torch.empty(1, dtype=torch.int32, device=device), None)
        self.ws_acc = torch.empty(specvlm.accept_workspace_bytes(1, w.gamma, w.vocab), dtype=torch.uint8,
                                  device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        # launches of our kernels per step: row LSE 1, rating 2 (column sums + finish), select 1,
        # gather 1, one per draft decode step, verify 1, accept 2 (split merges run inside the
        # attention kernels; the counter resets before them are memsets, not counted)
        self.launches_per_step = 1 + 2 + 1 + 1 + w.gamma + 1 + 2

    # the calls, in path order ------------------------------------------------------------------
    def row_lse_call(self):
        w, nv, nt = self.w, self.w.n_video(), self.w.n_text[0]
        self.sv.stage1_row_lse(self.inp["tcache_prompt"], self.inp["q_text"], [0, nt], [nv], self.scale,
                               row_lse=self.row_lse, d_status=self.status)

    def scores_call(self):
        nv, nt = self.w.n_video(), self.w.n_text[0]
        self.sv.stage1_scores(self.inp["tcache_prompt"], self.inp["q_text"], [0, nt], [nv], [0], [nv], [0, nv],
                              self.scale, scores=self.scores, ws=self.ws_scores, d_status=self.status,
                              row_lse=self.row_lse)

    def select_call(self):
        w, nv = self.w, self.w.n_video()
        self.sv.select(self.scores, [0, nv], [w.n_frames[0]], w.tokens_per_frame, [self.k1], [self.kt],
                       [0, self.kt], kept_idx=self.kept, d_status=self.status)

    def gather_call(self, dst):
        nv, nt = self.w.n_video(), self.w.n_text[0]
        self.sv.gather_kv(self.inp["dsrc"], self.kept, [0, self.kt], [0], [nv], [nv + nt], dst,
                          d_status=self.status)

    def decode_call(self, c, cache):
        self.sv.draft_decode_attn(cache, self.inp["q_dec"][c], self.scale, out=self.o_dec[c], ws=self.ws_dec,
                                  d_status=self.status)

    def verify_call(self):
        self.sv.verify_attn(self.inp["tcache"], self.inp["q_ver"], self.w.gamma, self.scale, out=self.o_ver,
                            ws=self.ws_ver, d_status=self.status)

    def accept_call(self):
        self.sv.accept(self.inp["logits"], self.inp["drafts"], ws=self.ws_acc, out=self.acc)


SEGMENTS = ["row_lse", "scores", "select", "gather", "decode", "verify", "accept"]


def run_ours(args, rank, world):
    import torch
    import torch.distributed as dist
    from paper_2508_16201_b200 import specvlm, synth

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    specvlm.lib()
    w = synth.workload(2)
    D, nv, nt, gamma = w.head_dim, w.n_video(), w.n_text[0], w.gamma
    inp = build_inputs(w, device, n_copies=gamma)
    path = Path(w, inp, device)
    E = lambda: torch.cuda.Event(enable_timing=True)

    # one-time: fill every pruned copy with real gathered data (copies 1.. are the decode inputs)
    path.row_lse_call(); path.scores_call(); path.select_call()
    for c in inp["dpruned"]:
        path.gather_call(c)
    torch.cuda.synchronize()

    def all_decodes():
        for c in range(gamma):
            # each draft step reads its own copy of the pruned cache: nothing is L2-resident
            path.decode_call(c, inp["dpruned"][1 + c])

    # the calls of a step, in path order; "decode" is the gamma draft steps together
    calls = {"row_lse": path.row_lse_call, "scores": path.scores_call, "select": path.select_call,
             "gather": lambda: path.gather_call(inp["dpruned"][0]), "decode": all_decodes,
             "verify": path.verify_call, "accept": path.accept_call}
    for _ in range(args.warmup):
        for fn in calls.values():
            fn()
    torch.cuda.synchronize()
    if not args.eager:
        # Each call (its C-ABI entry point, launches and memsets) is captured once into a CUDA graph
        # and replayed: a serving loop would do the same, and the short calls (a 10 us decode step)
        # are otherwise timed by the host's launch path, not by the GPU.
        side = torch.cuda.Stream()
        graphs = {}
        with torch.cuda.stream(side):
            for name, fn in calls.items():
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    fn()
                graphs[name] = g
        torch.cuda.synchronize()
        calls = {name: g.replay for name, g in graphs.items()}
        for _ in range(3):
            for fn in calls.values():
                fn()
        torch.cuda.synchronize()

    def step(ev):
        """ev: dict name -> list of (start, stop) event pairs appended for this step."""
        for name, fn in calls.items():
            a, b = E(), E()
            a.record()
            fn()
            b.record()
            ev[name].append((a, b))

    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev = {k: [] for k in SEGMENTS}
    t0, t1 = E(), E()
    torch.cuda.synchronize()
    wall0 = time.time()
    t0.record()
    for _ in range(args.steps):
        step(ev)
    t1.record()
    torch.cuda.synchronize()
    wall1 = time.time()
    if world > 1:
        dist.barrier()
    total_ms = t0.elapsed_time(t1)
    if rank == 0:
        time.sleep(0.2)
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    assert int(path.status.item()) == 0, "a device-side wait timed out"
    seg_ms = {k: [a.elapsed_time(b) / (gamma if k == "decode" else 1) for a, b in v] for k, v in ev.items()}
    mean = {k: sum(v) / len(v) for k, v in seg_ms.items()}          # per call (decode: per draft step)
    med = {k: statistics.median(v) for k, v in seg_ms.items()}

    # algorithmic K/V bytes (read once): 2 (K,V) * tokens * kv_heads * d * 2 B * layers
    n_p = w.k_total() + nt
    n_t = nv + nt + gamma + 1
    bytes_dec = 2 * n_p * w.d_kv_heads * D * 2 * w.d_layers
    bytes_ver = 2 * n_t * w.t_kv_heads * D * 2 * w.t_layers
    attn_ms = mean["decode"] * gamma + mean["verify"]
    attn_bytes = bytes_dec * gamma + bytes_ver

    # ---------------- end-to-end leg: inputs from pinned host memory, results read back
    e2e = run_e2e(args, path, inp, w, device, attn_bytes)

    # ---------------- extras outside the timed region, each timed like the headline calls: captured
    # once into its own CUDA graph, replayed 20 times behind an L2 flush, median of the event times
    extra = {}
    gt = GraphTimer(device, eager=args.eager)
    dsrc = inp["dsrc"]
    ws_u = torch.empty(max(256, specvlm.attn_workspace_bytes(dsrc, 1, w.d_q_heads, 0)), dtype=torch.uint8,
                       device=device)
    # the unpruned draft cache: the draft of plain speculative decoding (the paper's SD baseline)
    us_unpruned, _ = gt.time(lambda: specvlm.draft_decode_attn(dsrc, inp["q_dec"][0], path.scale, out=path.o_dec[0],
                                                               ws=ws_u, d_status=path.status))
    bytes_unpruned = 2 * (nv + nt) * w.d_kv_heads * D * 2 * w.d_layers
    extra["decode_unpruned_us"] = us_unpruned
    extra["decode_unpruned_kv_gbs"] = bytes_unpruned / (us_unpruned * 1e-6) / 1e9
    # the same pruned copy at every draft step, replayed back to back without a flush: what a draft
    # loop does.  The 43 MB stay in the L2 cache, so the step is no longer an HBM stream (the
    # headline never reuses a copy and counts HBM bytes only)
    run_l2 = gt.prepare(lambda: path.decode_call(0, inp["dpruned"][1]))
    a, b = E(), E()
    a.record()
    for i in range(20):
        run_l2()
    b.record()
    torch.cuda.synchronize()
    extra["decode_pruned_l2_resident_us"] = a.elapsed_time(b) * 1e3 / 20
    # T_t: the target's own single-token decode attention over the full cache (verification with
    # gamma = 0), against T_t^gamma (the verification call of the step) and T_d (a draft step): the
    # terms of the paper's latency model (Section 3.1, Eq. 1-3), attention only
    q_t = inp["q_ver"][:, :, :1].contiguous()
    o_t = torch.empty_like(q_t)
    ws_t0 = torch.empty(max(256, specvlm.attn_workspace_bytes(inp["tcache"], 1, w.t_q_heads, 0)), dtype=torch.uint8,
                        device=device)
    us_tt, _ = gt.time(lambda: specvlm.verify_attn(inp["tcache"], q_t, 0, path.scale, out=o_t, ws=ws_t0,
                                                   d_status=path.status))
    extra["target_decode_T_t_us"] = us_tt
    extra["target_decode_T_t_kv_gbs"] = bytes_ver / (us_tt * 1e-6) / 1e9
    extra["verify_over_target_decode_ratio"] = mean["verify"] * 1e3 / us_tt
    # illustrative only: attention times stand in for whole-model times, tau is the paper's printed
    # average accept length for chain drafting on the 72B/7B pair (2.79 pruned draft, 3.12 unpruned)
    extra["eq3_projection_pruned_draft_tau_2.79"] = sd_projection(2.79, gamma, mean["decode"] * 1e3, us_tt,
                                                                  mean["verify"] * 1e3)
    extra["eq3_projection_unpruned_draft_tau_3.12"] = sd_projection(3.12, gamma, us_unpruned, us_tt,
                                                                    mean["verify"] * 1e3)

    kept_tp = torch.empty(path.kt, dtype=torch.int32, device=device)
    k1_tp = torch.empty(1, dtype=torch.int32, device=device)
    extra["select_top_p_us"], _ = gt.time(lambda: specvlm.select_top_p(
        path.scores, [0, nv], [w.n_frames[0]], w.tokens_per_frame, [400], [path.kt], [0, path.kt], kept_idx=kept_tp,
        k_stage1_out=k1_tp))
    extra["select_random_us"], _ = gt.time(lambda: specvlm.select_baseline(
        specvlm.SEL_RANDOM, [w.n_frames[0]], w.tokens_per_frame, [path.kt], [0, path.kt], seed=1, device=device,
        kept_idx=kept_tp, want_counts=False))
    # tree drafting: the widest tree one 128-row launch holds (16 nodes at 8 query heads per KV head),
    # and a 26-node static tree (root + 25 candidates, the size of the static draft tree the paper
    # adopts; its shape here is a binary heap, the paper's figure being unavailable): 208 rows, two parts of 13 nodes in one launch
    for n_nodes in (128 // (w.t_q_heads // w.t_kv_heads), 26):
        n_tree = nv + nt + n_nodes
        tk = synth.randn_bf16((w.t_layers, 1, w.t_kv_heads, n_tree, D), device, 1, "treeK")
        tv = synth.randn_bf16((w.t_layers, 1, w.t_kv_heads, n_tree, D), device, 1, "treeV")
        tcache = specvlm.KvCache(tk, tv, torch.tensor([n_tree], dtype=torch.int32, device=device), n_tree)
        q_tree = synth.randn_bf16((w.t_layers, 1, n_nodes, w.t_q_heads, D), device, 1, "treeQ")
        parents = torch.tensor([[-1] + [(t - 1) // 2 for t in range(1, n_nodes)]], dtype=torch.int32, device=device)
        o_tree = torch.empty_like(q_tree)
        ws_t = torch.empty(specvlm.lib().specvlm_verify_tree_workspace_bytes(ctypes_byref(tcache), 1, w.t_q_heads, n_nodes),
                           dtype=torch.uint8, device=device)
        us, _ = gt.time(lambda: specvlm.verify_tree_attn(tcache, q_tree, parents, path.scale, out=o_tree, ws=ws_t,
                                                         d_status=path.status), reps=10)
        extra["verify_tree_%d_nodes_us" % n_nodes] = us
        extra["verify_tree_%d_nodes_kv_gbs_per_pass" % n_nodes] = (
            2 * n_tree * w.t_kv_heads * D * 2 * w.t_layers * ((n_nodes * (w.t_q_heads // w.t_kv_heads) + 127) // 128)
            / (us * 1e-6) / 1e9)
        lg = torch.randn((1, n_nodes, w.vocab), device=device)
        toks = torch.zeros((1, n_nodes), dtype=torch.int32, device=device)
        t_out = specvlm.accept_tree_buffers(1, n_nodes, w.vocab, device)
        extra["accept_tree_%d_nodes_us" % n_nodes], _ = gt.time(lambda: specvlm.accept_tree(lg, toks, parents, out=t_out))
        del tk, tv, tcache, q_tree, o_tree, lg, ws_t
    new_kv = synth.randn_bf16((w.t_layers, 1, gamma + 1, w.t_kv_heads, D), device, 2, "newKV")
    lens_keep = inp["tcache"].seq_lens.clone()
    lens_base = torch.tensor([nv + nt], dtype=torch.int32, device=device)

    def append_once():
        inp["tcache"].seq_lens.copy_(lens_base)                  # room for the gamma+1 new rows again
        specvlm.append_kv(inp["tcache"], new_kv, new_kv, d_status=path.status)
    extra["append_kv_us_incl_len_reset"], _ = gt.time(append_once)
    inp["tcache"].seq_lens.copy_(lens_keep)
    assert int(path.status.item()) == 0

    # max over ranks
    total_ms, attn_ms = max_over_ranks([total_ms, attn_ms], world, device)
    if rank != 0:
        return
    peaks = measured_peaks()
    value = replicas_value(attn_bytes, attn_ms, world)

    def hbm(name, nbytes, ms, traffic):
        ach = nbytes / (ms * 1e-3) / 1e9
        return {"kernel": name, "bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": round(ach / peaks["hbm_gbs"], 4), "frac_of_nominal_8000": round(ach / HBM_NOMINAL_GBS, 4),
                "traffic": traffic, "peak_source": peaks["source"], "launch_ms": round(ms, 5)}

    n_sms = torch.cuda.get_device_properties(device).multi_processor_count
    sm_max_mhz = peaks["sm_max_mhz"] or (clocks or {}).get("sm_max_mhz") or 1965.0
    ex2_peak = ex2_peak_gops(n_sms, sm_max_mhz)

    def rating(name, n_exp, flops, ms, traffic):
        # The rating passes evaluate one base-2 exponential per (query row, key) logit on the
        # special-function units: 16 per clock per SM x the device's SM count x its maximum SM clock
        # (148 x 1.965 GHz: 4653 G/s).  That bound (0.89 ms per pass here) is tighter than the
        # tensor-core one (1.05 TFLOP at the measured dense bf16 rate: 0.75 ms), so it is the
        # roofline; the tensor view is reported beside it.
        ach = n_exp / (ms * 1e-3) / 1e9
        tf = flops / (ms * 1e-3) / 1e12
        return {"kernel": name, "bound": "alu", "achieved": round(ach, 1), "peak": round(ex2_peak, 1), "unit": "Gex2/s",
                "frac": round(ach / ex2_peak, 4), "traffic": traffic,
                "peak_source": "derived: %d ex2/clk/SM x %d SMs x %.0f MHz" % (EX2_PER_CLK_PER_SM, n_sms, sm_max_mhz),
                "launch_ms": round(ms, 5),
                "tensor_tflops": round(tf, 1), "tensor_frac_of_measured_sustained": round(tf / peaks["bf16_tflops_sustained"], 4)}

    rows = w.t_layers * w.t_q_heads * nt
    flops_colsum = 2.0 * rows * nv * D
    flops_lse = 2.0 * w.t_layers * w.t_q_heads * D * sum(nv + i + 1 for i in range(nt))
    roofs = {
        "verify": hbm("attn_tc_kernel (verify, tcgen05)", bytes_ver, mean["verify"], NCU_TRAFFIC_BYTES["verify"]),
        "decode": hbm("attn_rows16_kernel (draft decode, pruned cache)", bytes_dec, mean["decode"],
                      NCU_TRAFFIC_BYTES["decode"]),
        "scores_colsum": rating("scores_colsum_tc_kernel", float(rows) * nv, flops_colsum, mean["scores"],
                                NCU_TRAFFIC_BYTES["scores_colsum"]),
        "scores_lse": rating("scores_lse_tc_kernel", flops_lse / (2.0 * D), flops_lse, mean["row_lse"],
                             NCU_TRAFFIC_BYTES["scores_lse"]),
    }
    dominant = max(("scores_colsum", "scores_lse", "verify", "decode"),
                   key=lambda k: {"scores_colsum": mean["scores"], "scores_lse": mean["row_lse"],
                                  "verify": mean["verify"], "decode": mean["decode"] * gamma}[k])
    out = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(total_ms / args.steps, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name + ": verifier 80L 64q/8kv d128, draft 28L 28q/4kv, 6272 video + 128 text "
                               "tokens, retention 10%, gamma 5, vocab 152064, batch 1, contiguous caches",
                   "l2": "verify cache 2.1 GB and rating K 1.05 GB exceed L2; each of the gamma draft steps reads "
                         "its own copy of the 43 MB pruned cache (6 copies, 260 MB), so no call finds its K/V in L2",
                   "replicas": world,
                   "launch": "eager launches" if args.eager else "one CUDA graph per call, replayed"},
        "pct_of_hbm_peak": {"of_measured_%d" % int(peaks["hbm_gbs"]): round(100 * value / world / peaks["hbm_gbs"], 2),
                            "of_nominal_8000": round(100 * value / world / HBM_NOMINAL_GBS, 2)},
        "per_call_us": {k: round(mean[k] * 1e3, 2) for k in SEGMENTS},
        "per_call_us_median": {k: round(med[k] * 1e3, 2) for k in SEGMENTS},
        "prune_us_per_call": round((mean["row_lse"] + mean["scores"] + mean["select"]) * 1e3, 2),
        "prune_us_with_caller_lse": round((mean["scores"] + mean["select"]) * 1e3, 2),
        "prune_total_us_with_gather": round((mean["row_lse"] + mean["scores"] + mean["select"] + mean["gather"]) * 1e3, 2),
        "kv_gbs": {"decode_pruned": round(bytes_dec / (mean["decode"] * 1e-3) / 1e9, 1),
                   "verify": round(bytes_ver / (mean["verify"] * 1e-3) / 1e9, 1),
                   "gather_rw": round(2 * bytes_dec / (mean["gather"] * 1e-3) / 1e9, 1),
                   "accept_logits": round((gamma + 1) * w.vocab * 4 / (mean["accept"] * 1e-3) / 1e9, 1)},
        "extra": {k: round(v, 2) for k, v in extra.items()},
        "roofline": roofs[dominant], "roofline_all": roofs,
        "e2e": e2e, "gpu_launches": path.launches_per_step * args.steps,
        "clocks": clocks,
    }
    if args.cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w)
    print(json.dumps(out))


def run_e2e(args, path, inp, w, device, attn_bytes):
    """Same step, but every call's inputs start in pinned host memory and its result is read back;
    the copies sit inside the timed regions.  The K/V caches are the serving state and stay on the
    device."""
    import torch
    gamma = w.gamma
    pin = lambda t: t.detach().cpu().pin_memory()
    h_qtext, h_qver = pin(inp["q_text"]), pin(inp["q_ver"])
    h_qdec = [pin(q) for q in inp["q_dec"]]
    h_logits, h_drafts = pin(inp["logits"]), pin(inp["drafts"])
    h_kept = torch.empty(path.kt, dtype=torch.int32).pin_memory()
    h_odec = [torch.empty_like(h) for h in h_qdec]
    h_odec = [h.pin_memory() for h in h_odec]
    h_over = torch.empty_like(h_qver).pin_memory()
    h_acc = torch.empty(2, dtype=torch.int32).pin_memory()
    h2d = (h_qtext.numel() * 2 + h_qver.numel() * 2 + sum(h.numel() * 2 for h in h_qdec) + h_logits.numel() * 4 +
           h_drafts.numel() * 4)
    d2h = h_kept.numel() * 4 + sum(h.numel() * 2 for h in h_odec) + h_over.numel() * 2 + 8
    E = lambda: torch.cuda.Event(enable_timing=True)
    copy_stream = torch.cuda.Stream()
    n_chunks = min(8, w.t_layers)
    bounds = [c * w.t_layers // n_chunks for c in range(n_chunks + 1)]
    attn_ms, step_ms = [], []
    for it in range(args.warmup + args.steps):
        s0, s1 = E(), E()
        s0.record()
        main = torch.cuda.current_stream()
        # Every host->device copy goes through a copy stream, in the order the path needs the data;
        # the main stream waits for each input's event right before the call that reads it, and the
        # results go back on the copy stream behind an event of the call that wrote them.  The text
        # queries arrive a range of layers at a time and each range is rated as soon as it has landed
        # (specvlm_stage1_scores_layers): the 168 MB copy hides the rating.
        copy_stream.wait_stream(main)
        up = {}

        def upload(name, dst, src):
            with torch.cuda.stream(copy_stream):
                dst.copy_(src, non_blocking=True)
                up[name] = torch.cuda.Event()
                up[name].record(copy_stream)

        def download(dst, src):
            done = torch.cuda.Event()
            done.record(main)
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(done)
                dst.copy_(src, non_blocking=True)

        for c in range(n_chunks):
            upload(("qt", c), inp["q_text"][bounds[c]:bounds[c + 1]], h_qtext[bounds[c]:bounds[c + 1]])
        for c in range(gamma):
            upload(("qd", c), inp["q_dec"][c], h_qdec[c])
        upload("qv", inp["q_ver"], h_qver)
        upload("lg", inp["logits"], h_logits)
        upload("dr", inp["drafts"], h_drafts)
        nv_, nt_ = w.n_video(), w.n_text[0]
        for c in range(n_chunks):
            main.wait_event(up[("qt", c)])
            path.sv.stage1_scores_layers(inp["tcache_prompt"], inp["q_text"], [0, nt_], [nv_], [0], [nv_], [0, nv_],
                                         path.scale, path.scores, path.ws_scores, bounds[c], bounds[c + 1],
                                         finish=(c == n_chunks - 1), d_status=path.status)
        path.select_call()
        download(h_kept, path.kept)
        path.gather_call(inp["dpruned"][0])
        a0, a1 = E(), E()
        a0.record()
        for c in range(gamma):
            main.wait_event(up[("qd", c)])
            path.decode_call(c, inp["dpruned"][1 + c])
            download(h_odec[c], path.o_dec[c])
        main.wait_event(up["qv"])
        path.verify_call()
        download(h_over, path.o_ver)
        main.wait_stream(copy_stream)          # the attention results have reached the host
        a1.record()
        main.wait_event(up["lg"])
        main.wait_event(up["dr"])
        path.accept_call()
        download(h_acc[0:1], path.acc[0])
        download(h_acc[1:2], path.acc[1])
        main.wait_stream(copy_stream)
        s1.record()
        torch.cuda.synchronize()
        if it >= args.warmup:
            attn_ms.append(a0.elapsed_time(a1))
            step_ms.append(s0.elapsed_time(s1))
    am = sum(attn_ms) / len(attn_ms)
    return {"value": round(attn_bytes / (am * 1e-3) / 1e9, 1), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "ms_per_step": round(sum(step_ms) / len(step_ms), 4),
            "attention_ms_per_step": round(am, 4),
            "note": "pinned host q / logits in, outputs out, inside the timed region; K/V caches resident; the text "
                    "queries are copied and rated a range of layers at a time; all copies run on a copy stream beside the kernels"}


# ------------------------------------------------------------------------------------------------
def oracle_sample(w, n_verify_layers):
    """Times the CPU oracle on a bounded sample: gamma draft decode steps over the pruned cache (all
    draft layers) + verification over n_verify_layers verifier layers.  Returns (KV bytes, seconds)."""
    import numpy as np
    import oracle
    rng = np.random.default_rng(0)
    D, nv, nt, gamma = w.head_dim, w.n_video(), w.n_text[0], w.gamma
    n_p, n_t = w.k_total() + nt, nv + nt + gamma + 1
    scale = 1.0 / math.sqrt(D)

    def bf16(shape):
        return (rng.standard_normal(shape).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    kd, vd = bf16((w.d_kv_heads, n_p, D)), bf16((w.d_kv_heads, n_p, D))
    qd = bf16((1, w.d_q_heads, D))
    kt_, vt_ = bf16((w.t_kv_heads, n_t, D)), bf16((w.t_kv_heads, n_t, D))
    qv = bf16((gamma + 1, w.t_q_heads, D))
    t0 = time.perf_counter()
    for _ in range(gamma):
        for _l in range(w.d_layers):
            oracle.attention(qd, kd, vd, n_p, scale)
    for _l in range(n_verify_layers):
        oracle.attention(qv, kt_, vt_, n_t, scale)
    dt = time.perf_counter() - t0
    nbytes = gamma * w.d_layers * 2 * n_p * w.d_kv_heads * D * 2 + n_verify_layers * 2 * n_t * w.t_kv_heads * D * 2
    return nbytes, dt


def cpu_baseline(w):
    import oracle
    n_layers, reps = w.t_layers, 4
    oracle_sample(w, 1)                       # loads / builds the oracle before the clock starts
    nbytes, dt = 0, 0.0
    for _ in range(reps):
        b, t = oracle_sample(w, n_layers)
        nbytes += b
        dt += t
    out = {"value": round(nbytes / dt / 1e9, 4), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "seconds": round(dt, 2),
           "sample": f"fp64 oracle attention, {reps} steps: each {w.gamma} draft decode steps over the pruned cache "
                     f"(all {w.d_layers} draft layers) + verification over all {n_layers} verifier layers"}
    out["prune"] = oracle_prune_sample(w, 2)
    return out


def oracle_prune_sample(w, n_layers):
    """Times the oracle's prune stage once: token rating on n_layers verifier layers (every layer is
    the same amount of work, so the whole rating is extrapolated by the layer count), selection,
    and the K/V gather of all draft layers."""
    import numpy as np
    import oracle
    rng = np.random.default_rng(1)
    D, nv, nt = w.head_dim, w.n_video(), w.n_text[0]

    def bf16(shape):
        return (rng.standard_normal(shape).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    q = bf16((n_layers, nt, w.t_q_heads, D))
    k = bf16((n_layers, w.t_kv_heads, nv + nt, D))
    t0 = time.perf_counter()
    a = oracle.stage1_scores(q, k, 0, nv, nv, 1.0 / math.sqrt(D))
    t_rate = time.perf_counter() - t0
    a32 = a.astype(np.float32)
    t0 = time.perf_counter()
    kept = oracle.select(a32, w.n_frames[0], w.tokens_per_frame, w.k_stage1(), w.k_total())
    t_sel = time.perf_counter() - t0
    src = bf16((w.d_layers, w.d_kv_heads, nv + nt, D))
    t0 = time.perf_counter()
    for _ in range(2):                                       # K and V
        oracle.gather_kv(src, np.asarray(kept), 0, nv, nv + nt)
    t_gat = time.perf_counter() - t0
    rate_all = t_rate * w.t_layers / n_layers
    return {"rating_s_extrapolated": round(rate_all, 2), "rating_layers_timed": n_layers, "select_s": round(t_sel, 4),
            "gather_s": round(t_gat, 4), "prune_s_extrapolated": round(rate_all + t_sel, 2),
            "note": f"fp64 oracle: rating timed on {n_layers} of {w.t_layers} verifier layers and scaled by the layer "
                    f"count (extrapolated), selection and the gather of all {w.d_layers} draft layers timed whole"}


def run_reference(args, rank):
    if rank != 0:
        return
    from paper_2508_16201_b200 import synth
    import oracle
    w = synth.workload(2)
    n_layers = 16                           # bounded sample per step
    for _ in range(args.warmup):
        oracle_sample(w, 1)
    tot_b, tot_t = 0, 0.0
    for _ in range(args.steps):
        b, t = oracle_sample(w, n_layers)
        tot_b += b
        tot_t += t
    v = round(tot_b / tot_t / 1e9, 4)
    sample = (f"fp64 oracle attention per step: {w.gamma} draft decode steps over the pruned cache (all "
              f"{w.d_layers} draft layers) + verification over {n_layers} of {w.t_layers} verifier layers")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(tot_t / args.steps * 1e3, 2), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name + " (bounded sample, see cpu_baseline.sample)"},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_case(args):
    """One call of the path on a reduced number of layers (a small case for `ncu`, or a sweep):
    prints the median device time of `--iters` launches.  Not the benchmark line."""
    import dataclasses
    import torch
    from paper_2508_16201_b200 import specvlm, synth
    w = synth.workload(args.workload, gamma=args.gamma)
    if args.layers:
        w = dataclasses.replace(w, t_layers=args.layers, d_layers=args.layers)
    if args.frames:
        w = dataclasses.replace(w, n_frames=(args.frames,))
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    if w.batch > 1:
        run_case_batched(args, w, device)
        return
    inp = build_inputs(w, device, n_copies=1)
    path = Path(w, inp, device)
    path.row_lse_call(); path.scores_call(); path.select_call()
    for c in inp["dpruned"]:
        path.gather_call(c)
    D, nv, nt, gamma = w.head_dim, w.n_video(), w.n_text[0], w.gamma
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    dsrc = inp["dsrc"]
    ws_u = torch.empty(max(256, specvlm.attn_workspace_bytes(dsrc, 1, w.d_q_heads, 0)), dtype=torch.uint8,
                       device=device)
    calls = {
        "verify": (path.verify_call, 2 * (nv + nt + gamma + 1) * w.t_kv_heads * D * 2 * w.t_layers),
        "decode": (lambda: path.decode_call(0, inp["dpruned"][1]), 2 * (w.k_total() + nt) * w.d_kv_heads * D * 2 * w.d_layers),
        "decode_unpruned": (lambda: specvlm.draft_decode_attn(dsrc, inp["q_dec"][0], path.scale, out=path.o_dec[0], ws=ws_u),
                            2 * (nv + nt) * w.d_kv_heads * D * 2 * w.d_layers),
        "row_lse": (path.row_lse_call, 0), "scores": (path.scores_call, 0), "select": (path.select_call, 0),
        "gather": (lambda: path.gather_call(inp["dpruned"][0]), 4 * (w.k_total() + nt) * w.d_kv_heads * D * 2 * w.d_layers),
        "accept": (path.accept_call, (gamma + 1) * w.vocab * 4),
    }
    if args.case == "verify_tree":
        # a heap-shaped draft tree of --nodes nodes behind the prompt (128 rows per launch at most)
        n_nodes = args.nodes
        n_tree = nv + nt + n_nodes
        tk = synth.randn_bf16((w.t_layers, 1, w.t_kv_heads, n_tree, D), device, 1, "treeK")
        tv = synth.randn_bf16((w.t_layers, 1, w.t_kv_heads, n_tree, D), device, 1, "treeV")
        tcache = specvlm.KvCache(tk, tv, torch.tensor([n_tree], dtype=torch.int32, device=device), n_tree)
        q_tree = synth.randn_bf16((w.t_layers, 1, n_nodes, w.t_q_heads, D), device, 1, "treeQ")
        parents = torch.tensor([[-1] + [(t - 1) // 2 for t in range(1, n_nodes)]], dtype=torch.int32, device=device)
        o_tree = torch.empty_like(q_tree)
        ws_t = torch.empty(specvlm.lib().specvlm_verify_tree_workspace_bytes(ctypes_byref(tcache), 1, w.t_q_heads, n_nodes),
                           dtype=torch.uint8, device=device)
        passes = (n_nodes * (w.t_q_heads // w.t_kv_heads) + 127) // 128
        calls["verify_tree"] = (lambda: specvlm.verify_tree_attn(tcache, q_tree, parents, path.scale, out=o_tree, ws=ws_t),
                                passes * 2 * n_tree * w.t_kv_heads * D * 2 * w.t_layers)
    fn, nbytes = calls[args.case]
    ts = []
    for i in range(args.warmup + args.iters):
        if args.flush:
            flush.zero_()
            flush.view(torch.int32).sum()       # read back: leaves the L2 clean (no write-back under the timed call)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        if i >= args.warmup:
            ts.append(a.elapsed_time(b))
    assert int(path.status.item()) == 0
    med = statistics.median(ts)
    print(json.dumps({"case": args.case, "workload": w.name, "layers": args.layers, "gamma": gamma,
                      "median_us": round(med * 1e3, 2), "min_us": round(min(ts) * 1e3, 2),
                      "gbs": round(nbytes / (med * 1e-3) / 1e9, 1) if nbytes else None,
                      "env": {k: v for k, v in os.environ.items() if k.startswith("SPECVLM_")}}))


def run_case_batched(args, w, device):
    """The attention calls on a batched workload: ragged sequences in 64-token pages scattered over a
    pool (the rating / selection / gather cases time one sequence at a time and are not offered here)."""
    import torch
    from paper_2508_16201_b200 import specvlm, synth
    D, B, gamma = w.head_dim, w.batch, w.gamma
    scale = 1.0 / math.sqrt(D)

    def paged(n_layers, n_kv_heads, lens, tag):
        need = [(n + 63) // 64 for n in lens]
        pool, max_blocks = sum(need) + 3, max(need) + 1
        table = synth.page_table(B, max_blocks, pool, need, 0, device)
        k = synth.randn_bf16((n_layers, pool, n_kv_heads, 64, D), device, 0, tag + "K")
        v = synth.randn_bf16((n_layers, pool, n_kv_heads, 64, D), device, 0, tag + "V")
        cache = specvlm.KvCache(k, v, torch.tensor(lens, dtype=torch.int32, device=device), max(lens), table)
        return cache, 2 * sum(lens) * n_kv_heads * D * 2 * n_layers

    if args.case == "verify":
        cache, nbytes = paged(w.t_layers, w.t_kv_heads, [w.seq_len(b) + gamma + 1 for b in range(B)], "t")
        q = synth.randn_bf16((w.t_layers, B, gamma + 1, w.t_q_heads, D), device, 0, "Qv")
        out = torch.empty_like(q)
        ws = torch.empty(max(256, specvlm.attn_workspace_bytes(cache, B, w.t_q_heads, gamma)), dtype=torch.uint8, device=device)
        fn = lambda: specvlm.verify_attn(cache, q, gamma, scale, out=out, ws=ws)
    elif args.case in ("decode", "decode_unpruned"):
        lens = [(w.k_total(b) + w.n_text[b]) if args.case == "decode" else w.seq_len(b) for b in range(B)]
        cache, nbytes = paged(w.d_layers, w.d_kv_heads, lens, "d")
        q = synth.randn_bf16((w.d_layers, B, w.d_q_heads, D), device, 0, "Qd")
        out = torch.empty_like(q)
        ws = torch.empty(max(256, specvlm.attn_workspace_bytes(cache, B, w.d_q_heads, 0)), dtype=torch.uint8, device=device)
        fn = lambda: specvlm.draft_decode_attn(cache, q, scale, out=out, ws=ws)
    else:
        raise SystemExit("--case %s is timed one sequence at a time: use a batch-1 workload" % args.case)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    ts = []
    for i in range(args.warmup + args.iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        if i >= args.warmup:
            ts.append(a.elapsed_time(b))
    med = statistics.median(ts)
    print(json.dumps({"case": args.case, "workload": w.name, "batch": B, "paged": True, "gamma": gamma,
                      "median_us": round(med * 1e3, 2), "min_us": round(min(ts) * 1e3, 2),
                      "gbs": round(nbytes / (med * 1e-3) / 1e9, 1)}))


# ------------------------------------------------------------------------------------------------
# --workloads: every call of the path on every synthetic workload, with the sweeps
# ------------------------------------------------------------------------------------------------
class WorkloadCase:
    """Device-resident synthetic tensors of one workload shape (any batch; contiguous caches for a
    single sequence, 64-token pages scattered over a pool for a batch) and its calls.  The verifier
    side may hold fewer layers than the workload names when device memory is short: every layer is
    an independent, equally sized problem for every call, so a call's time is the sum over layer
    chunks; the chunks being alike, one is timed and multiplied by their number."""

    def __init__(self, w, device, gamma_max, retention_max_permille, t_layers=None):
        import torch
        from paper_2508_16201_b200 import specvlm, synth
        self.w, self.device, self.sv, self.torch, self.synth = w, device, specvlm, torch, synth
        self.B, self.D = w.batch, w.head_dim
        B, D = self.B, self.D
        self.scale = 1.0 / math.sqrt(D)
        self.t_layers = t_layers or w.t_layers
        self.t_chunks = -(-w.t_layers // self.t_layers)
        self.nv = [w.n_video(b) for b in range(B)]
        self.nt = [w.n_text[b] for b in range(B)]
        self.text_cu = [0] + [sum(self.nt[:b + 1]) for b in range(B)]
        self.video_cu = [0] + [sum(self.nv[:b + 1]) for b in range(B)]
        self.gamma_max = gamma_max
        cap_t = [self.nv[b] + self.nt[b] + gamma_max + 1 for b in range(B)]
        self.tk, self.tv, self.t_table = self._alloc(self.t_layers, w.t_kv_heads, cap_t, "t")
        self.q_text = synth.randn_bf16((self.t_layers, self.text_cu[-1], w.t_q_heads, D), device, 0, "Qtext")
        for b in range(B):
            sal = synth.salient_set(self.nv[b], w.planted_permille, 0, b)
            qb = self.q_text[:, self.text_cu[b]:self.text_cu[b + 1]]
            if self.t_table is None:
                synth.plant_salient_(self.tk[:, 0, :, :self.nv[b], :], qb, sal)
            else:
                synth.plant_salient_paged_(self.tk, self.t_table[b], 0, self.nv[b], qb, sal)
        self.prompt = self.cache(self.tk, self.tv, [self.nv[b] + self.nt[b] for b in range(B)], self.t_table)
        cap_d = [self.nv[b] + self.nt[b] for b in range(B)]
        self.sk, self.svv, self.s_table = self._alloc(w.d_layers, w.d_kv_heads, cap_d, "d")
        self.dsrc = self.cache(self.sk, self.svv, cap_d, self.s_table)
        cap_p = [self.nv[b] * retention_max_permille // 1000 + self.nt[b] for b in range(B)]
        # five copies of the pruned cache: a draft step is timed as five calls in one graph, each on
        # its own copy (as the headline does), so that no call finds its K/V in the L2 cache
        self.pcopies = [self._alloc(w.d_layers, w.d_kv_heads, cap_p, "p%d" % c) for c in range(5)]
        self.pk, self.pv, self.p_table = self.pcopies[0]
        self.q_dec = synth.randn_bf16((w.d_layers, B, w.d_q_heads, D), device, 0, "Qd")
        self.o_dec = torch.empty_like(self.q_dec)
        self.logits, self.drafts = synth.logits_and_drafts(B, gamma_max, w.vocab, device, 0)
        self.row_lse = torch.empty((self.t_layers, self.text_cu[-1], w.t_q_heads), dtype=torch.float32, device=device)
        self.scores = torch.empty(self.video_cu[-1], dtype=torch.float32, device=device)
        self.ws_scores = torch.empty(specvlm.stage1_scores_workspace_bytes(self.prompt, self.text_cu, self.nv,
                                                                           w.t_q_heads), dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def _alloc(self, n_layers, n_kv_heads, caps, tag):
        torch, synth, B, D = self.torch, self.synth, self.B, self.D
        if B == 1 and not self.w.paged:
            shape, table = (n_layers, 1, n_kv_heads, caps[0], D), None
        else:
            need = [(n + 63) // 64 for n in caps]
            pool = sum(need) + 3
            table = synth.page_table(B, max(need) + 1, pool, need, 0, self.device)
            shape = (n_layers, pool, n_kv_heads, 64, D)
        return (synth.randn_bf16(shape, self.device, 0, tag + "K"), synth.randn_bf16(shape, self.device, 0, tag + "V"),
                table)

    def cache(self, k, v, lens, table):
        lens_t = self.torch.tensor(lens, dtype=self.torch.int32, device=self.device)
        return self.sv.KvCache(k, v, lens_t, max(lens), table)

    def kv_bytes(self, lens, n_kv_heads, n_layers):
        return 2 * sum(lens) * n_kv_heads * self.D * 2 * n_layers

    def ws(self, cache, n_q_heads, gamma):
        return self.torch.empty(max(256, self.sv.attn_workspace_bytes(cache, self.B, n_q_heads, gamma)),
                                dtype=self.torch.uint8, device=self.device)


def run_workloads(args):
    """Every call of the path on workloads 2-5 (and the tiny workload 1), one JSON line per
    workload: median device time of 20 graph replays behind an L2 flush, K/V GB/s and the fraction
    of the measured HBM peak where the call is a stream.  Workload 4 sweeps the retention (5, 10,
    20, 50 %), workload 5 the draft length gamma (3..8); workload 5 runs batched and paged."""
    import torch
    from paper_2508_16201_b200 import specvlm, synth
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    gt = GraphTimer(device, eager=args.eager)
    reps = args.iters if args.iters > 10 else 20
    which = [int(x) for x in args.workloads.split(",")]

    def rec(us, mn, nbytes=None, chunks=1):
        """us, mn, nbytes: of one layer chunk; the call's time is the chunk's time x chunks."""
        r = {"us": round(us * chunks, 2), "min_us": round(mn * chunks, 2)}
        if chunks > 1:
            r["layer_chunks"] = chunks
        if nbytes:
            r["gbs"] = round(nbytes / (us * 1e-6) / 1e9, 1)
            r["frac_of_measured_%d" % int(peaks["hbm_gbs"])] = round(r["gbs"] / peaks["hbm_gbs"], 4)
            r["frac_of_nominal_8000"] = round(r["gbs"] / HBM_NOMINAL_GBS, 4)
        return r

    for i in which:
        w = synth.workload(i)
        sweep_ret = [50, 100, 200, 500] if i == 4 else [w.retention_permille]
        sweep_gamma = list(range(3, 9)) if i == 5 else [w.gamma]
        B, D = w.batch, w.head_dim
        # verifier layers held at once: all of them when its K/V fits in 60 % of the free memory
        free, _ = torch.cuda.mem_get_info(device)
        per_layer = 2 * sum(w.seq_len(b) + 9 + 64 for b in range(B)) * w.t_kv_heads * D * 2
        t_layers = w.t_layers
        while t_layers > 1 and t_layers * per_layer > 0.6 * free:
            t_layers = (t_layers + 1) // 2
        c = WorkloadCase(w, device, max(sweep_gamma), max(sweep_ret), t_layers)
        ch = c.t_chunks
        L_t = c.t_layers * ch                                  # layers the chunked time stands for (>= w.t_layers)
        out = {"workload": w.name, "batch": B, "paged": c.t_table is not None,
               "verifier_layers_held": c.t_layers, "verifier_layer_chunks": ch,
               "launch": "eager" if args.eager else "one CUDA graph per call, replayed behind a 512 MB L2 flush (written, then read back)",
               "reps": reps, "calls": {}, "sweeps": {}}
        calls = out["calls"]
        # ---- prune side
        calls["row_lse"] = rec(*gt.time(lambda: specvlm.stage1_row_lse(c.prompt, c.q_text, c.text_cu, c.nv, c.scale,
                                                                       row_lse=c.row_lse, d_status=c.status), reps), chunks=ch)
        calls["scores_given_lse"] = rec(*gt.time(lambda: specvlm.stage1_scores(
            c.prompt, c.q_text, c.text_cu, c.nv, [0] * B, c.nv, c.video_cu, c.scale, scores=c.scores, ws=c.ws_scores,
            d_status=c.status, row_lse=c.row_lse), reps), chunks=ch)
        n_exp = sum(w.t_q_heads * c.nt[b] * c.nv[b] for b in range(B)) * float(L_t)
        calls["scores_given_lse"]["gex2_per_s"] = round(n_exp / (calls["scores_given_lse"]["us"] * 1e-6) / 1e9, 1)
        sel, gat, dec = {}, {}, {}
        for ret in sweep_ret:
            wr = synth.workload(i, retention_permille=ret)
            kt = [wr.k_total(b) for b in range(B)]
            k1 = [wr.k_stage1(b) for b in range(B)]
            kept_cu = [0] + [sum(kt[:b + 1]) for b in range(B)]
            kept = torch.empty(max(kept_cu[-1], 1), dtype=torch.int32, device=device)
            sel[ret] = rec(*gt.time(lambda: specvlm.select(c.scores, c.video_cu, list(w.n_frames), w.tokens_per_frame,
                                                           k1, kt, kept_cu, kept_idx=kept, d_status=c.status), reps))
            plens = [kt[b] + c.nt[b] for b in range(B)]
            pruned = c.cache(c.pk, c.pv, plens, c.p_table)
            src_len = [c.nv[b] + c.nt[b] for b in range(B)]
            gat[ret] = rec(*gt.time(lambda: specvlm.gather_kv(c.dsrc, kept, kept_cu, [0] * B, c.nv, src_len, pruned,
                                                              d_status=c.status), reps),
                           nbytes=2 * c.kv_bytes(plens, w.d_kv_heads, w.d_layers))
            ws_d = c.ws(pruned, w.d_q_heads, 0)
            copies = [c.cache(pk, pv, plens, pt) for pk, pv, pt in c.pcopies]

            def five_steps():
                for pc in copies:
                    specvlm.draft_decode_attn(pc, c.q_dec, c.scale, out=c.o_dec, ws=ws_d, d_status=c.status)
            us5, mn5 = gt.time(five_steps, reps)
            dec[ret] = rec(us5 / 5, mn5 / 5, nbytes=c.kv_bytes(plens, w.d_kv_heads, w.d_layers))
            dec[ret]["timed_as"] = "5 calls on 5 copies of the cache in one graph, per call"
            dec[ret]["tokens"] = plens if B > 1 else plens[0]
        base = w.retention_permille
        calls["select"], calls["gather"], calls["decode_pruned"] = sel[base], gat[base], dec[base]
        if len(sweep_ret) > 1:
            out["sweeps"]["retention_permille"] = {str(r): {"select": sel[r], "gather": gat[r], "decode_pruned": dec[r]}
                                                   for r in sweep_ret}
        ws_u = c.ws(c.dsrc, w.d_q_heads, 0)
        calls["decode_unpruned"] = rec(*gt.time(lambda: specvlm.draft_decode_attn(
            c.dsrc, c.q_dec, c.scale, out=c.o_dec, ws=ws_u, d_status=c.status), reps),
            nbytes=c.kv_bytes([c.nv[b] + c.nt[b] for b in range(B)], w.d_kv_heads, w.d_layers))
        # ---- verification and acceptance
        ver, acc = {}, {}
        for g in sorted(set(sweep_gamma + [0])):
            lens = [c.nv[b] + c.nt[b] + g + 1 for b in range(B)]
            tc = c.cache(c.tk, c.tv, lens, c.t_table)
            q = synth.randn_bf16((c.t_layers, B, g + 1, w.t_q_heads, D), device, 0, "Qv", g)
            o = torch.empty_like(q)
            ws_v = c.ws(tc, w.t_q_heads, g)
            ver[g] = rec(*gt.time(lambda: specvlm.verify_attn(tc, q, g, c.scale, out=o, ws=ws_v, d_status=c.status),
                                  reps), nbytes=c.kv_bytes(lens, w.t_kv_heads, c.t_layers), chunks=ch)
            ver[g]["rows_per_kv_head"] = (g + 1) * (w.t_q_heads // w.t_kv_heads)
            if g == 0:
                continue
            lg = c.logits[:, :g + 1].contiguous()
            dr = c.drafts[:, :g].contiguous()
            a_out = (torch.empty(B, dtype=torch.int32, device=device), torch.empty(B, dtype=torch.int32, device=device), None)
            ws_a = torch.empty(specvlm.accept_workspace_bytes(B, g, w.vocab), dtype=torch.uint8, device=device)
            acc[g] = rec(*gt.time(lambda: specvlm.accept(lg, dr, ws=ws_a, out=a_out), reps), nbytes=B * (g + 1) * w.vocab * 4)
            # the same call four times in one graph, each on its own logits: what the call costs inside
            # a longer graph (a lone graph launch adds about 4 us between the event and the first kernel)
            lgs = [lg] + [torch.randn_like(lg) for _ in range(3)]

            def four_calls():
                for x in lgs:
                    specvlm.accept(x, dr, ws=ws_a, out=a_out)
            us4, mn4 = gt.time(four_calls, reps)
            acc[g]["in_graph_of_4"] = rec(us4 / 4, mn4 / 4, nbytes=B * (g + 1) * w.vocab * 4)
            del lgs
            del q, o, ws_v
        calls["verify"], calls["accept"], calls["target_decode_T_t"] = ver[w.gamma], acc[w.gamma], ver[0]
        if len(sweep_gamma) > 1:
            out["sweeps"]["gamma"] = {str(g): {"verify": ver[g], "accept": acc[g]} for g in sweep_gamma}
        assert int(c.status.item()) == 0, "a device-side check or wait reported an error"
        calls["prune_us"] = round(calls["row_lse"]["us"] + calls["scores_given_lse"]["us"] + calls["select"]["us"], 2)
        calls["prune_us_with_caller_lse"] = round(calls["scores_given_lse"]["us"] + calls["select"]["us"], 2)
        t_d, t_t, t_v = calls["decode_pruned"]["us"], calls["target_decode_T_t"]["us"], calls["verify"]["us"]
        out["latency_model_eq1_3"] = {
            "T_d_us": t_d, "T_t_us": t_t, "T_t_gamma_us": t_v, "verify_over_target_decode": round(t_v / t_t, 4),
            "illustrative_speedup_tau_2.79": round(sd_projection(2.79, w.gamma, t_d, t_t, t_v), 3),
            "note": "attention-only times in the paper's latency model; tau is the paper's printed chain figure"}
        print(json.dumps(out), flush=True)
        del c
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, help="run one call only (small case for profiling / sweeps)")
    ap.add_argument("--workloads", default=None, help="comma-separated workload numbers (e.g. 2,3,4,5): time every "
                                                      "call of the path on each, with the sweeps; one JSON line each")
    ap.add_argument("--layers", type=int, default=0)
    ap.add_argument("--frames", type=int, default=0)
    ap.add_argument("--workload", type=int, default=2)
    ap.add_argument("--gamma", type=int, default=None)
    ap.add_argument("--nodes", type=int, default=16, help="draft-tree nodes of --case verify_tree")
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--flush", action="store_true", help="write and read back a 512 MB buffer before each launch")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--eager", action="store_true", help="launch every call from the host instead of replaying "
                                                         "per-call CUDA graphs")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.workloads:
        run_workloads(args)
        return
    if args.case:
        run_case(args)
        return
    if args.impl == "reference":
        run_reference(args, rank)
        return
    args.warmup = max(args.warmup, 3)
    if world > 1 or rank != 0:
        args.cpu_baseline = False
    run_ours(args, rank, world)


if __name__ == "__main__":
    main()
