"""Rates of the two instructions that bound the score stage, measured on the current GPU.

    python -m paper_2503_17922_b200.probes

Prints one JSON line: exponentials (ex2.approx.ftz.f32) per second and per clock per SM, and block
elements per second of the cross-lane column sum a single-sweep kernel would need, each timed with
CUDA events around one launch of the library's probe kernels (after a warm-up launch), with the SM
clock nvidia-smi reports right after.
"""
from __future__ import annotations

import json
import subprocess


def measure() -> dict:
    import torch
    from . import binding
    scratch = torch.zeros(4, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    out = {"sms": sms}
    for name, fn, iters in (("ex2", binding.wkv_probe_ex2_rate, 4096), ("colsum", binding.wkv_probe_colsum_rate, 512)):
        fn(scratch, sms * 4, 1024, 64)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        n = fn(scratch, sms * 4, 1024, iters)
        b.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(b)
        out[name + "_per_s"] = n / (ms * 1e-3)
        out[name + "_launch_ms"] = ms
    try:
        mhz = subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader,nounits"],
                             capture_output=True, text=True, timeout=10).stdout.strip().splitlines()[0]
        out["sm_mhz_after"], out["sm_max_mhz"] = [float(x) for x in mhz.split(",")]
    except Exception:
        out["sm_mhz_after"] = out["sm_max_mhz"] = None
    clk = (out["sm_max_mhz"] or 1965.0) * 1e6
    out["ex2_per_clk_per_sm_at_max_clock"] = out["ex2_per_s"] / (sms * clk)
    out["colsum_elements_per_clk_per_sm_at_max_clock"] = out["colsum_per_s"] / (sms * clk)
    return out


if __name__ == "__main__":
    print(json.dumps(measure()))
