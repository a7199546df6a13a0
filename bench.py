#!/usr/bin/env python
"""Benchmark of the WindowKV prefill-compression hot path (score -> pool -> top-k -> gather).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C3]

One step = one `wkv_compress_group` call on one layer group of the workload
(leader scoring + selection, then the shared-index gather of all gamma layers),
rotating over the model's groups so that every step reads cold HBM.  Prints one
JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_17922_b200 import workloads as wl   # noqa: E402

METRIC = "prefill-compression tokens/s per layer group"
UNIT = "tokens/s"


def pick_workload(name: str):
    if name == "C2":
        return wl.llama8b_single_group(wl.TASK_AGGREGATION)
    if name == "C4":
        return wl.mistral_needle(32768, 0.5)
    if name == "C5-small":
        return wl.batched_ragged_small()
    return wl.ALL_CONFIGS[name]()


def algorithmic_bytes(w, prob) -> dict:
    """Bytes the method must move for one group (leader K once, Q_obs, and read+write of the
    retained rows of K and V of every layer) with the per-stage split."""
    e = 4 if w.dtype == "f32" else 2
    tokens = int(w.seqlens().sum())
    score = tokens * w.n_kv_heads * w.head_dim * e + w.batch * w.n_q_heads * w.l_obs * w.head_dim * e
    keep_rows = 0
    for n, b in zip(w.seqlens(), w.budgets()):
        k = min(max(0, (int(b) - w.l_obs) // w.window), -(-max(int(n) - w.l_obs, 0) // w.window))
        keep_rows += k * w.window + min(w.l_obs, int(n))
    gather = w.gamma * 2 * 2 * keep_rows * w.n_kv_heads * w.head_dim * e
    return {"score": score, "gather": gather, "total": score + gather, "tokens": tokens}


def lse_obs_of(w, d):
    """Harness input of the given-normaliser stage: log-sum-exp of the causal logits of every
    observation row, float32 [B, H_q, alpha], as the leader layer's prefill attention would return
    it.  Plain torch ops on the synthetic inputs."""
    import torch
    q, k = d["q"].float(), d["k"][0].float()                     # [B, H_q, alpha, d], [B, H_kv, N, d]
    B, n, a, G = w.batch, w.max_seqlen, w.l_obs, w.n_q_heads // w.n_kv_heads
    logits = torch.einsum("bhgad,bhnd->bhgan", q.view(B, w.n_kv_heads, G, a, w.head_dim), k) / w.head_dim ** 0.5
    pos = torch.arange(n - a, n, device=q.device).view(1, 1, 1, a, 1)
    logits = logits.masked_fill(torch.arange(n, device=q.device).view(1, 1, 1, 1, n) > pos, float("-inf"))
    return torch.logsumexp(logits, dim=-1).reshape(B, w.n_q_heads, a).contiguous()


def peaks() -> dict:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops", 1590.0)),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


def score_other_floors(w, pk, ex2_per_s: float) -> dict:
    """What else bounds the score stage besides the bytes of K: the exponentials (one per row and
    key in each of the two sweeps, at the rate the ex2 probe measured on this GPU in this run) and
    the contraction (2 * R * d flops per key and sweep, against the measured bf16 GEMM rate).
    Milliseconds per launch."""
    keys = int(w.seqlens().sum()) * w.n_kv_heads          # (unit, key) pairs
    rows = w.rows
    exps = 2.0 * keys * rows
    flops = 2.0 * 2.0 * keys * rows * w.head_dim
    return {"ex2_floor_ms": exps / ex2_per_s * 1e3, "ex2_per_s_measured": ex2_per_s,
            "ex2_per_clk_per_sm_at_1965mhz": ex2_per_s / (148 * 1.965e9),
            "tensor_floor_ms": flops / (pk["bf16_tflops"] * 1e12) * 1e3}


KERNEL_SOURCES = ("score_tc.cu", "score_math.cuh", "tc_common.cuh", "topk_block.cuh", "wkv_internal.cuh", "gather.cu")


def kernel_source_hash() -> str:
    """Fingerprint of the sources of the two kernels of the default path (score + selection, gather): the
    ncu traffic figures are only quoted while it is unchanged."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2503_17922_b200", "csrc")
    for name in KERNEL_SOURCES:
        h.update(name.encode())
        h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of the kernel from the committed ncu capture, or None when there is no
    capture of this kernel on this workload or the kernel sources have changed since it was taken."""
    p = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    if not os.path.exists(p):
        return None
    found, current = None, False
    for line in open(p):
        f = line.split()
        if len(f) == 2 and f[0] == "sources":
            current = f[1] == kernel_source_hash()
        if len(f) == 3 and f[0] == kernel and f[1] == workload:
            found = int(f[2])
    return found if current else None


class ClockSampler:
    """Read-only sampling of the current GPU's clocks with nvidia-smi (selected by UUID, so that
    CUDA_VISIBLE_DEVICES cannot point it at another GPU), written to a file so that no sample is lost
    when the sampler is stopped.  It runs for the whole process; `mark()` notes the start and end of
    the timed region, and the summary says how many samples fell inside it."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str, period_ms: int = 20):
        import tempfile
        self.uuid, self.period_ms = uuid, period_ms
        self.proc, self.marks = None, []
        self.path = os.path.join(tempfile.gettempdir(), f"wkv_clocks_{os.getpid()}.csv")

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.uuid}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms),
                                          "-f", self.path], stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def mark(self):
        self.marks.append(time.time())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(2.5 * self.period_ms / 1e3)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        import datetime
        rows = []
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(f[1]), float(f[2]), f[4:8]))
                except ValueError:
                    continue
            os.remove(self.path)
        except OSError:
            pass
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

        def summary(sel):
            reasons = set()
            for _, _, _, flags in sel:
                for nm, val in zip(names, flags):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
            return {"sm_mhz": statistics.median(r[1] for r in sel) if sel else None,
                    "sm_max_mhz": max((r[2] for r in sel), default=None), "samples": len(sel),
                    "reasons": sorted(reasons)}
        inside = [r for r in rows if len(self.marks) >= 2 and self.marks[0] <= r[0] <= self.marks[1]]
        out = summary(inside)
        if len(inside) < 3:
            # the timed region is shorter than a few sampling periods: report what the GPU did while this
            # process had it under load (warm-up, timed region and the stage timings that follow)
            out = summary(rows)
            out["window"] = "whole process (timed region shorter than the sampling period)"
        else:
            out["window"] = "timed region"
        if not rows:
            out["reasons"] = ["no sample could be read from nvidia-smi"]
        return out


def time_oracle_groups(w, groups, min_seconds: float, max_groups: int):
    """Runs the CPU oracle on whole groups until `min_seconds` of work; returns (tokens/s, n_groups, s)."""
    import oracle
    tokens = int(w.seqlens().sum())
    done, spent = 0, 0.0
    while (spent < min_seconds and done < max_groups) or done == 0:
        grp = groups[done % len(groups)]
        t0 = time.perf_counter()
        oracle.compress_group(grp["q_obs"], grp["k_layers"], grp["v_layers"], n_kv_heads=w.n_kv_heads,
                              l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                              max_seqlen=w.max_seqlen, budgets=grp["budgets"], cu_seqlens=grp["cu_seqlens"])
        spent += time.perf_counter() - t0
        done += 1
    return tokens * done / spent, done, spent


def run_reference(args) -> None:
    """The reference arm: the CPU oracle, as it stands, on the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    w = pick_workload(args.workload)
    n_distinct = min(w.n_groups, 2)
    groups = [wl.make_group(w, g) for g in range(n_distinct)]
    tokens = int(w.seqlens().sum())

    def step(i):
        grp = groups[i % n_distinct]
        oracle.compress_group(grp["q_obs"], grp["k_layers"], grp["v_layers"], n_kv_heads=w.n_kv_heads,
                              l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                              max_seqlen=w.max_seqlen, budgets=grp["budgets"], cu_seqlens=grp["cu_seqlens"])
    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(i)
    dt = time.perf_counter() - t0
    value = tokens * args.steps / dt
    cores = oracle.num_threads()
    sample = f"one whole layer group ({w.gamma} layers, {tokens} tokens) per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype,
        "data": "synthetic (seeded; shapes of the paper's long-context workloads)",
        "config": {"workload": w.name, "batch": w.batch, "seq_len": w.max_seqlen, "layers_per_group": w.gamma},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=40)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3", choices=["C1", "C2", "C3", "C4", "C5", "C5-small"])
    ap.add_argument("--score-impl", default="auto", choices=["auto", "simt", "tcgen05", "pipelined"])
    ap.add_argument("--groups", type=int, default=0, help="distinct groups kept on the device (0 = all)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 4000:
            args.steps, args.warmup = 8, 3
        run_reference(args)
        return

    import torch
    from paper_2503_17922_b200 import binding, replicas

    # replicas only: every rank runs the whole path on its own copy of the workload (no exchange step).
    # Asked for N > 1 as a plain command (no launcher environment), the benchmark starts its N ranks itself.
    if args.gpus > 1 and not replicas.launcher_present():
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus}: only {torch.cuda.device_count()} CUDA devices are visible")
        sys.exit(replicas.relaunch_under_launcher(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    rank, world, local = replicas.rank_env()
    torch.cuda.set_device(local)
    replicas.init("nccl", torch.device("cuda", local))
    binding.lib()          # fails loudly if the CUDA library is missing
    sampler = None
    if rank == 0:
        uuid = str(torch.cuda.get_device_properties(local).uuid)
        sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
        sampler.start()

    w = pick_workload(args.workload)
    impl = {"auto": binding.WKV_SCORE_AUTO, "simt": binding.WKV_SCORE_SIMT,
            "tcgen05": binding.WKV_SCORE_TCGEN05, "pipelined": binding.WKV_SCORE_TCGEN05_PIPELINED}[args.score_impl]
    prob = binding.Problem.from_workload(w, score_impl=impl)
    prob_pipe = binding.Problem.from_workload(w, score_impl=binding.WKV_SCORE_TCGEN05_PIPELINED) \
        if (impl == binding.WKV_SCORE_AUTO and w.dtype == "bf16" and w.rows <= 128) else None
    alg = algorithmic_bytes(w, prob)
    tokens = alg["tokens"]
    warmup = max(args.warmup, 3)

    # ---- inputs: every group of the model resident in HBM (each rank its own copy: weak scaling)
    n_groups = w.n_groups if args.groups <= 0 else min(args.groups, w.n_groups)
    host_groups, dev_groups = [], []
    for g in range(n_groups):
        grp = wl.make_group(w, g)
        if g < 2:
            host_groups.append(grp)
        dev_groups.append({"q": binding.to_device(grp["q_obs"]),
                           "k": [binding.to_device(x) for x in grp["k_layers"]],
                           "v": [binding.to_device(x) for x in grp["v_layers"]]})
    out = prob.alloc_outputs(w.gamma)
    work = prob.alloc_workspace()
    stream = torch.cuda.Stream()           # everything below is launched and timed on this stream
    torch.cuda.synchronize()
    resident = sum(t.numel() * t.element_size() for d in dev_groups for t in d["k"] + d["v"])
    flush = None
    if resident < 512 * 1024 * 1024:       # small workloads fit L2: flush between steps
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")

    # the calls of the timed loop, marshalled once (one per resident group)
    cap = out["keep_capacity"]
    group_calls = [binding.prepare_compress_group(prob, d["q"], d["k"], d["v"], out["k_out"], out["v_out"],
                                                  out["window_scores"], out["window_idx"], out["kept_len"], work,
                                                  keep_capacity=cap, stream=stream) for d in dev_groups]
    score_calls = [binding.prepare_score_windows(prob, d["q"], d["k"][0], out["window_scores"], None, work,
                                                 stream=stream) for d in dev_groups]
    leader_calls = [binding.prepare_select_leader_windows(prob, d["q"], d["k"][0], out["window_scores"],
                                                          out["window_idx"], out["kept_len"], work, stream=stream)
                    for d in dev_groups]
    pipe_calls = None
    if prob_pipe is not None:
        pipe_calls = [binding.prepare_compress_group(prob_pipe, d["q"], d["k"], d["v"], out["k_out"],
                                                        out["v_out"], out["window_scores"], out["window_idx"],
                                                        out["kept_len"], work, keep_capacity=cap, stream=stream)
                         for d in dev_groups]
    select_call = binding.prepare_select_topk_windows(prob, out["window_scores"], out["window_idx"],
                                                      out["kept_len"], stream=stream)
    gather_calls = [binding.prepare_gather_kv(prob, d["k"], d["v"], out["window_idx"], out["k_out"], out["v_out"],
                                              keep_capacity=cap, stream=stream) for d in dev_groups]

    # the call of the timed loop: the group recorded once per resident group (wkv_group_plan_create),
    # replayed with wkv_group_plan_launch, as an engine with static buffers would issue it
    plans = [binding.GroupPlan(prob, d["q"], d["k"], d["v"], out["k_out"], out["v_out"], out["window_scores"],
                               out["window_idx"], out["kept_len"], work, keep_capacity=cap) for d in dev_groups]

    barrier = replicas.barrier

    with torch.cuda.stream(stream):
        for i in range(warmup):
            if flush is not None:
                flush.fill_(i & 0xFF)
            plans[i % n_groups].launch(stream)
        barrier()
        if sampler:
            sampler.mark()
        launches0 = binding.wkv_launch_count()
        if flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(args.steps):
                plans[i % n_groups].launch(stream)
            e1.record(stream)
            barrier()
            ms_total = e0.elapsed_time(e1)
        else:                               # time each step alone so that the flush is not counted
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(args.steps)]
            for i in range(args.steps):
                flush.fill_(i & 0xFF)
                evs[i][0].record(stream)
                plans[i % n_groups].launch(stream)
                evs[i][1].record(stream)
            barrier()
            ms_total = sum(a.elapsed_time(b) for a, b in evs)
        launches = binding.wkv_launch_count() - launches0
        if sampler:
            sampler.mark()
        ms_total = replicas.max_over_ranks(ms_total, "cuda")
        ms_per_step = ms_total / args.steps
        value = replicas.whole_job_rate(tokens, world, ms_per_step)
        if binding.device_status(work) != 0:
            raise RuntimeError("a kernel reported an expired wait: results invalid")

        # ---- per-kernel device times: the same launches, captured once in a CUDA graph and replayed, so
        # that only device time is between the two events (still the same rotation over cold groups)
        def time_stage(calls, reps_target_ms: float = 30.0) -> float:
            n = len(calls)
            for c in calls:
                c.run()
            stream.synchronize()
            if flush is not None:           # L2-resident workload: time each launch alone behind a flush
                pairs = []
                for i in range(32):
                    flush.fill_(i & 0xFF)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    calls[i % n].run()
                    b.record(stream)
                    pairs.append((a, b))
                stream.synchronize()
                return sum(a.elapsed_time(b) for a, b in pairs) / len(pairs)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for c in calls:
                    c.run()
            g.replay()
            stream.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            g.replay()
            b.record(stream)
            stream.synchronize()
            reps = max(3, int(reps_target_ms / max(a.elapsed_time(b), 1e-3)))
            a.record(stream)
            for _ in range(reps):
                g.replay()
            b.record(stream)
            stream.synchronize()
            return a.elapsed_time(b) / (reps * n)

        # the same group through the direct entry point, call by call (two launches on the stream per step)
        ms_direct = None
        if flush is None:
            n_direct = min(args.steps, 1000)
            d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            d0.record(stream)
            for i in range(n_direct):
                group_calls[i % n_groups].run()
            d1.record(stream)
            stream.synchronize()
            ms_direct = d0.elapsed_time(d1) / n_direct
        ms_fused = time_stage(group_calls)                 # the group call's launch(es), graph replay
        ms_score = time_stage(score_calls)                 # scores and pooling only
        ms_score_select = time_stage(leader_calls)         # scores, pooling and selection in one launch, timed directly
        ms_pipe = time_stage(pipe_calls) if pipe_calls else None   # the opt-in single-launch form of the group
        # the special-function rate of this GPU, measured: 148 x 4 blocks of 1024 threads, 8 chains each
        probe_scratch = torch.zeros(4, dtype=torch.float32, device="cuda")
        binding.wkv_probe_ex2_rate(probe_scratch, 592, 1024, 64, stream=stream)
        pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pa.record(stream)
        n_ex2 = binding.wkv_probe_ex2_rate(probe_scratch, 592, 1024, 4096, stream=stream)
        pb.record(stream)
        stream.synchronize()
        ex2_per_s = n_ex2 / (pa.elapsed_time(pb) * 1e-3)
        ms_select = time_stage([select_call])              # stand-alone selection kernel (not on the fused path)
        ms_gather = time_stage(gather_calls)
        # the variant that takes Eq. 1's normalisers from the caller (no statistics sweep); the inputs of
        # this stage are made here with torch ops, outside any timed region
        ms_given_lse = None
        if not w.ragged:
            lse = [lse_obs_of(w, d) for d in dev_groups]
            lse_calls = [binding.prepare_compress_group_lse(prob, d["q"], l, d["k"], d["v"], out["k_out"],
                                                            out["v_out"], out["window_scores"], out["window_idx"],
                                                            out["kept_len"], work, keep_capacity=cap, stream=stream)
                         for d, l in zip(dev_groups, lse)]
            ms_given_lse = time_stage(lse_calls)
    clocks = sampler.stop() if sampler else None
    if clocks and clocks.get("sm_mhz"):
        # the step in SM clock cycles: comparable between runs that saw different clocks
        clocks["sm_cycles_per_step"] = ms_per_step * 1e-3 * clocks["sm_mhz"] * 1e6

    pk = peaks()
    floors = score_other_floors(w, pk, ex2_per_s)
    floors["hbm_floor_ms"] = alg["score"] / (pk["hbm_gbs"] * 1e9) * 1e3
    launches_per_step = launches / args.steps
    if launches_per_step < 1.5:
        # the whole group is ONE launch (scores, selection and gather in the pipelined kernel): its
        # duration is the time per step of the timed region, its bytes are the path's
        dom_ms, dom_bytes, kernel_key = ms_per_step, alg["total"], "group_pipeline"
        roofline = {"bound": "hbm", "kernel": "group_pipeline_tc (scores + pooling + selection + gather, one launch)",
                    "achieved": dom_bytes / (dom_ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "peak_source": pk["source"], "traffic": ncu_traffic(kernel_key, w.name),
                    "algorithmic_bytes_per_launch": dom_bytes, "launch_ms": dom_ms,
                    "launch_ms_source": "timed region / launches (CUDA events on the launching stream)",
                    "score_stage_floors": floors}
    else:
        dominant = "gather" if ms_gather >= ms_score_select else "score"
        dom_ms = ms_gather if dominant == "gather" else ms_score_select
        other = "score" if dominant == "gather" else "gather"
        other_ms = ms_score_select if dominant == "gather" else ms_gather
        names = {"gather": "gather_kv_kernel", "score": "score kernel (both sweeps + pooling + selection)"}
        roofline = {"bound": "hbm", "kernel": names[dominant], "achieved": alg[dominant] / (dom_ms * 1e-3) / 1e9,
                    "peak": pk["hbm_gbs"], "unit": "GB/s", "peak_source": pk["source"],
                    "traffic": ncu_traffic(dominant, w.name), "algorithmic_bytes_per_launch": alg[dominant],
                    "launch_ms": dom_ms, "launch_ms_source": "the launch alone, graph replay between CUDA events",
                    "score_stage_floors": floors,
                    "other_kernel": {"kernel": names[other], "launch_ms": other_ms,
                                     "achieved": alg[other] / (other_ms * 1e-3) / 1e9}}
    roofline["frac"] = roofline["achieved"] / pk["hbm_gbs"]
    path_frac = alg["total"] / (ms_per_step * 1e-3) / 1e9 / pk["hbm_gbs"]

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed)
    e2e = None
    if not args.no_e2e:
        pin = lambda a: binding.to_device(a, "cpu").pin_memory()
        hsets = []
        for grp in host_groups:
            hsets.append({"q": pin(grp["q_obs"]), "k": [pin(x) for x in grp["k_layers"]],
                          "v": [pin(x) for x in grp["v_layers"]]})
        h_k_out = [torch.empty_like(t, device="cpu").pin_memory() for t in out["k_out"]]
        h_v_out = [torch.empty_like(t, device="cpu").pin_memory() for t in out["v_out"]]
        h_idx = torch.empty_like(out["window_idx"], device="cpu").pin_memory()
        h_kept = torch.empty_like(out["kept_len"], device="cpu").pin_memory()
        stage = dev_groups[0]

        def e2e_step(i):
            hs = hsets[i % len(hsets)]
            binding.wkv_compress_group_host(prob, hs["q"], hs["k"], hs["v"], h_k_out, h_v_out, h_idx, h_kept,
                                            stage["q"], stage["k"], stage["v"], out["k_out"], out["v_out"],
                                            out["window_idx"], out["kept_len"], out["keep_capacity"], work,
                                            stream=stream)
        e2e_steps = 12
        for i in range(2):
            e2e_step(i)
        barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            e2e_step(i)
        barrier()
        dt = time.perf_counter() - t0
        dt = replicas.max_over_ranks(dt, "cuda")
        nb = lambda t: t.numel() * t.element_size()
        h2d = nb(hsets[0]["q"]) + sum(nb(x) for x in hsets[0]["k"] + hsets[0]["v"])
        d2h = sum(nb(x) for x in h_k_out + h_v_out) + nb(h_idx) + nb(h_kept)
        e2e = {"value": tokens * world * e2e_steps / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps}

    # ---- the oracle on the host cores (rank 0, single-GPU runs only)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        v, n_done, spent = time_oracle_groups(w, host_groups, 10.0, 24)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"{n_done} whole layer groups of {w.name} ({spent:.1f} s)"}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "accum_dtype": "f32",
            "data": "synthetic (seeded; shapes of the paper's long-context workloads)",
            "config": {"workload": w.name, "batch": w.batch, "seq_len": w.max_seqlen, "layers_per_group": w.gamma,
                       "groups_rotated": n_groups, "l_obs": w.l_obs, "window": w.window,
                       "budget_tokens": int(w.budgets()[0]), "score_impl": args.score_impl,
                       "call": "wkv_group_plan_launch (one recorded group per step)",
                       "cold_cache": "flush of 256 MB between steps" if flush is not None
                       else f"{n_groups} groups rotated ({resident / 1e9:.2f} GB resident, larger than L2)"},
            "gpu_launches": int(launches),
            "path_hbm_frac": path_frac,
            "path_algorithmic_bytes": alg["total"],
            "stages_ms": {"group_graph_replay": ms_fused, "group_pipelined_single_launch_form": ms_pipe,
                          "score_select_one_launch": ms_score_select,
                          "score_only": ms_score, "select_standalone": ms_select, "gather_standalone": ms_gather,
                          "group_given_lse_graph_replay": ms_given_lse,
                          "group_direct_call": ms_direct},
            "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu_baseline, "clocks": clocks,
        }))
    replicas.shutdown()


if __name__ == "__main__":
    main()
