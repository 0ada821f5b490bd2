#!/usr/bin/env python
"""Benchmark of the Lory MoE layer (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl ours|reference]

One step = one forward + backward pass of the whole layer over one batch of synthetic
input (x, dY ~ N(0,1); weights ~ N(0, 0.02); bf16).  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "Lory MoE-layer fwd+bwd tokens/s (bf16, 1 B200)"
UNIT = "tokens/s"


PROF_RECORDS = 8192   # capacity of the library's per-launch event table


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(source="measured", hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]))
    return dict(source="fallback", hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0)


def flops_per_step(wl):
    """Appendix B count: forward = 6*tokens*d*f (FFN) + 6*E*d*f per segment (merge); backward = 2x."""
    return 18 * wl.d * wl.f * (wl.T + wl.E) * wl.S


# algorithmic FLOPs of one launch of each labelled kernel (three launches share "merge", "wgrad", ...)
def kernel_flops(wl):
    tok, S, d, f, E = wl.tokens, wl.S, wl.d, wl.f, wl.E
    return {
        "merge": 3 * 2 * S * E * d * f,      # all three matrices
        "gemm1_swiglu": 4 * tok * d * f,
        "gemm2": 2 * tok * d * f,
        "dh_dswiglu": 2 * tok * d * f,
        "wgrad": 2 * tok * d * f,            # per matrix
        "dx": 4 * tok * d * f,
        "dtheta": 2 * S * E * d * f,         # per matrix
        "dw": 2 * S * E * d * f,             # per matrix
        "stage2": 3 * 4 * S * E * d * f,     # all three matrices, both products
    }


# Which roofline bounds a labelled kernel: the dense contractions are tensor-core work, the routing-weighted sums
# over the experts (merge, its adjoint) and the pooling stream the method's tensors through HBM.
KERNEL_BOUND = {"gemm1_swiglu": "tensor", "gemm2": "tensor", "dh_dswiglu": "tensor", "wgrad": "tensor", "dx": "tensor",
                "merge": "hbm", "stage2": "hbm", "pool_router": "hbm"}


def compulsory_bytes(wl):
    """What the method itself has to move per step: x read in the forward and in the backward, y written, dY read,
    dX written (5 activation tensors), the experts read in the forward and in the backward and their gradients
    written (3 passes over E * 3 * d * f parameters); bf16.  Merged weights, their gradients and saved activations
    are choices of an implementation and are not in here."""
    return 5 * wl.tokens * wl.d * 2 + 3 * wl.E * 3 * wl.d * wl.f * 2


# algorithmic bytes of one launch of each labelled kernel: only tensors the method defines (x, y, dY, dX, the
# experts, their gradients), each once.  The HBM-bound kernels are measured against these.
def method_bytes(wl):
    act = 2 * wl.tokens * wl.d
    Pb = 2 * wl.d * wl.f                      # one expert matrix
    launches_256 = (wl.S + 255) // 256
    return {
        "pool_router": act,                                  # x
        "merge": 3 * wl.E * Pb,                              # the experts, once
        "gemm1_swiglu": act,                                 # x
        "gemm2": act,                                        # y
        "dh_dswiglu": act,                                   # dY
        "wgrad": 2 * wl.tokens * (wl.d + wl.f),              # per launch: its two activation operands
        "stage2": 2 * 3 * wl.E * Pb,                         # the experts in, their gradients out
        "dx": act,                                           # dX
        "_launches_256": launches_256,
    }


# HBM bytes per step of each labelled kernel AS IMPLEMENTED (per launch for the three "wgrad" launches): inputs read
# once + outputs written once, merged weights, their gradients and the saved activations included; bf16
def implementation_bytes(wl):
    tok, S, d, f, E = wl.tokens, wl.S, wl.d, wl.f, wl.E
    P1 = d * f
    launches_256 = (S + 255) // 256
    return {
        # the merge and its adjoint take one launch per 256 segments; every launch reads the experts, and the
        # adjoint's launches after the first re-read and re-write the expert gradients
        "merge": 3 * 2 * (launches_256 * E * P1 + S * P1),        # all three matrices: read W, write Wbar
        "dtheta": 2 * (S * P1 + E * P1),
        "dw": 2 * (S * P1 + E * P1),
        "stage2": 3 * 2 * (S * P1 + (3 * launches_256 - 1) * E * P1),   # read dWbar and W, write (re-read) dW
        "pool_router": 2 * tok * d,
        "add_pool_grad": 4 * tok * d,
        # grouped GEMMs: operands once + outputs once
        "gemm1_swiglu": 2 * (tok * d + 2 * S * P1 + 3 * tok * f),   # x, Wbar1, Wbar3 -> G, U, H
        "gemm2": 2 * (tok * f + S * P1 + tok * d),                  # H, Wbar2 -> y
        "dh_dswiglu": 2 * (tok * d + S * P1 + 4 * tok * f),         # dY, Wbar2, G, U -> dG, dU
        "wgrad": 2 * (tok * (d + f) + S * P1),                      # per matrix: two activations -> dWbar
        "dx": 2 * (2 * tok * f + 2 * S * P1 + tok * d),             # dG, dU, Wbar1, Wbar3 -> dx
    }


def implementation_bytes_per_step(wl):
    kb = implementation_bytes(wl)
    return (kb["merge"] + kb["stage2"] + kb["gemm1_swiglu"] + kb["gemm2"] + kb["dh_dswiglu"] + 3 * kb["wgrad"]
            + kb["dx"] + kb["pool_router"])


# DRAM traffic of one launch (dram__bytes_read.sum + dram__bytes_write.sum) from a one-pass ncu capture of one
# step of the named workload.  The figures hold only for the kernel sources the capture ran: `sources_sha1` is
# the digest of the CUDA sources at that time, and a different digest turns the reported traffic into null.
NCU_TRAFFIC = {
    "C3": {
        "sources_sha1": "cebe8cf3fc030c69f7acb3f3be5693b7b1ceb632",
        "bytes": {"pool_router": 68e6, "merge": 2792e6, "gemm1_swiglu": 2017e6, "gemm2": 964e6, "dh_dswiglu": 1486e6,
                  "wgrad": 908e6, "stage2": 3238e6, "router_backward": 3e6, "dx": 1875e6},
    },
}


def cuda_sources_sha1():
    import hashlib
    root = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2405_03133_b200", "csrc")
    h = hashlib.sha1()
    for name in sorted(os.listdir(root)):
        if name.endswith((".cu", ".cuh")):
            with open(os.path.join(root, name), "rb") as fh:
                h.update(name.encode() + b"\0" + fh.read())
    return h.hexdigest()


def measured_traffic(wl_name, label):
    ent = NCU_TRAFFIC.get(wl_name)
    if ent is None or ent["sources_sha1"] != cuda_sources_sha1():
        return None
    return ent["bytes"].get(label)


class ClockSampler:
    """Samples nvidia-smi clocks while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, smax, reasons = [], None, set()
        rows = [l for t, l in self.lines if t0 <= t <= t1 + 0.2] or [l for _, l in self.lines]
        for l in rows:
            parts = [x.strip() for x in l.split(",")]
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except (ValueError, IndexError):
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=smax, reasons=sorted(reasons),
                    samples=len(sm))


def oracle_sample(wl, n_segments=2):
    """A bounded sample of the workload for the CPU oracle: the first `n_segments` segments of one
    sequence (the second is routed by the first, so the shift is exercised)."""
    from paper_2405_03133_b200.workloads import make_inputs
    small = wl.with_(B=1, L=n_segments * wl.T)
    return small, make_inputs(small)


def time_oracle(small, inp, repeats=1):
    from oracle import lory_oracle as O
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], small.T)
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        O.forward(*a)
        O.backward(*a, inp["dy"])
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i["num_threads"] for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count()


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    small, inp = oracle_sample(wl, 2)
    times = []
    for i in range(args.warmup + args.steps):
        t = time_oracle(small, inp)
        if i >= args.warmup:
            times.append(t)
    total = sum(times)
    value = small.tokens * len(times) / total
    sample = f"first 2 segments of one sequence ({small.tokens} tokens) of {wl.name}, oracle forward+backward, float64"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def aggregate_over_ranks(ms_total_local, steps, tokens_per_rank, world, dist, device):
    """Replicas only: every rank runs the whole layer on its own batch, nothing is exchanged on the data path.
    The step time of the job is the slowest rank's; the job's throughput is all ranks' tokens over that time."""
    ms_total = ms_total_local
    if dist is not None and world > 1:
        import torch
        t = torch.tensor([ms_total_local], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_per_step = ms_total / steps
    return ms_per_step, world * tokens_per_rank / (ms_per_step * 1e-3)


def workload_config(wl):
    return {"workload": f"{wl.name}: B={wl.B} L={wl.L} T={wl.T} d_model={wl.d} d_ff={wl.f} E={wl.E} bf16, "
                        f"fwd+bwd, segments={wl.S}",
            "tokens_per_step": wl.tokens, "l2": "working set (merged weights, activations: several GB) exceeds L2; no flush"}


def run_decode(args, wl):
    """Prompt-only routing at inference (Section 3.1): one prefill over the prompt fixes a merged FFN per sequence;
    every later call applies it to n new tokens per sequence.  A call has to read each sequence's merged weights
    once (B * 3 * d * f * 2 bytes) whatever n is, so it is bound by HBM: reported are the device time per call
    (CUDA events over a run of back-to-back calls), tokens/s, the merged-weight bytes over that time against the
    measured copy bandwidth, and the host time the call itself takes (the floor of a latency-bound decode loop)."""
    import torch
    import paper_2405_03133_b200 as lory
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(4321)

    def normal(shape, std):
        return (torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)

    peaks = load_peaks()
    w_r, W1 = normal((wl.E, wl.d), 0.02), normal((wl.E, wl.f, wl.d), 0.02)
    W2, W3 = normal((wl.E, wl.d, wl.f), 0.02), normal((wl.E, wl.f, wl.d), 0.02)
    prompt = normal((wl.B, wl.L, wl.d), 1.0)
    pdims = lory.make_dims(wl.B, wl.L, wl.L, wl.d, wl.f, wl.E, "bf16")
    fwd_b, _ = lory.lory_moe_workspace_bytes(pdims)
    ws = torch.empty(fwd_b, dtype=torch.uint8, device=dev)
    y = torch.empty_like(prompt)
    rw = torch.empty((wl.B, wl.E), dtype=torch.float32, device=dev)
    lory.lory_moe_forward(pdims, prompt, w_r, W1, W2, W3, y, rw, None, ws)
    lory.lory_check_status(pdims, ws)
    merged_bytes = wl.B * 3 * wl.d * wl.f * 2
    rows = []
    for n in (1, 4, 16, 64):
        ddims = lory.make_dims(wl.B, n, n, wl.d, wl.f, wl.E, "bf16", lory.LORY_FLAG_REUSE_MERGED)
        x_new = normal((wl.B, n, wl.d), 1.0)
        y_new = torch.empty_like(x_new)
        for _ in range(max(args.warmup, 3)):
            lory.lory_moe_ffn(ddims, x_new, None, W1, W2, W3, y_new, ws)
        torch.cuda.synchronize()
        calls = 200
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        ev0.record()
        for _ in range(calls):
            lory.lory_moe_ffn(ddims, x_new, None, W1, W2, W3, y_new, ws)
        ev1.record()
        host_us = (time.perf_counter() - t0) / calls * 1e6
        torch.cuda.synchronize()
        dev_us = ev0.elapsed_time(ev1) / calls * 1e3
        lory.lory_check_status(ddims, ws)
        # per-kernel times of a few more calls (events around every launch; not part of the figures above)
        lory.lory_profile_enable(True)
        for _ in range(20):
            lory.lory_moe_ffn(ddims, x_new, None, W1, W2, W3, y_new, ws)
        per = {}
        for label, ms in lory.lory_profile_read():
            per.setdefault(label, []).append(ms * 1e3)
        lory.lory_profile_enable(False)
        rows.append({"new_tokens_per_sequence": n, "device_us_per_call": dev_us, "host_us_per_call": host_us,
                     "kernel_us": {k: sum(v) / len(v) for k, v in per.items()},
                     "tokens_per_s": wl.B * n / (dev_us * 1e-6), "launches_per_call": lory.lory_last_launch_count(),
                     "merged_weight_gbs": merged_bytes / (dev_us * 1e-6) / 1e9,
                     "frac_of_hbm_peak": merged_bytes / (dev_us * 1e-6) / 1e9 / peaks["hbm_gbs"]})
    print(json.dumps({"metric": "Lory prompt-routed decode (cached merged FFN), tokens/s", "unit": UNIT,
                      "config": {"workload": f"{wl.name}: B={wl.B} prompt={wl.L} d_model={wl.d} d_ff={wl.f} E={wl.E} bf16",
                                 "merged_weight_bytes_per_call": merged_bytes}, "dtype": "bf16", "data": "synthetic",
                      "hbm_peak_gbs": peaks["hbm_gbs"], "calls": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=0, help="override the number of sequences B (profiling on a small case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the second timed region of >= 1 s")
    ap.add_argument("--chunked-adjoint", action="store_true",
                    help="A/B: run the backward with LORY_FLAG_CHUNKED_ADJOINT (per-segment weight gradients kept in "
                         "an L2-sized buffer, one parameter rectangle at a time) instead of the default")
    ap.add_argument("--graph", action="store_true",
                    help="capture one forward+backward (the same C-ABI calls on one stream) in a CUDA graph and time "
                         "its replays instead of plain launches (measured the same at C3: 2.707 vs 2.710 ms)")
    ap.add_argument("--decode", action="store_true",
                    help="measure the inference path instead: prefill with prompt-only routing, then decode calls")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2405_03133_b200.workloads import CONFIGS
    wl = CONFIGS[args.workload]
    if args.batch > 0:
        wl = wl.with_(B=args.batch, name=f"{wl.name}_B{args.batch}")
    if args.impl == "reference":
        run_reference(args, wl)
        return
    if args.decode:
        run_decode(args, wl)
        return

    import torch
    import paper_2405_03133_b200 as lory

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    dev = torch.device("cuda", local_rank)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)

    def normal(shape, std):
        return (torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)

    x = normal((wl.B, wl.L, wl.d), 1.0)
    w_r = normal((wl.E, wl.d), 0.02)
    W1 = normal((wl.E, wl.f, wl.d), 0.02)
    W2 = normal((wl.E, wl.d, wl.f), 0.02)
    W3 = normal((wl.E, wl.f, wl.d), 0.02)
    dy = normal((wl.B, wl.L, wl.d), 1.0)
    dims = lory.make_dims(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, "bf16",
                          lory.LORY_FLAG_CHUNKED_ADJOINT if args.chunked_adjoint else 0)
    _, bwd_bytes = lory.lory_moe_workspace_bytes(dims)
    ws = torch.empty(bwd_bytes, dtype=torch.uint8, device=dev)
    y = torch.empty_like(x)
    dx = torch.empty_like(x)
    route_w = torch.empty((wl.S, wl.E), dtype=torch.float32, device=dev)
    dw_r = torch.empty_like(w_r)
    dW1, dW2, dW3 = torch.empty_like(W1), torch.empty_like(W2), torch.empty_like(W3)

    launches = [0]
    # a stream of our own: the calls below name it, the events of the timed region are recorded on it
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    sp = stream.cuda_stream

    def step_calls():
        lory.lory_moe_forward(dims, x, w_r, W1, W2, W3, y, route_w, None, ws, stream=sp)
        n = lory.lory_last_launch_count()
        lory.lory_moe_backward(dims, x, w_r, W1, W2, W3, dy, dx, dw_r, dW1, dW2, dW3, None, ws, stream=sp)
        launches[0] = n + lory.lory_last_launch_count()

    step = step_calls
    if args.graph:
        for _ in range(2):          # first calls set per-device function attributes: not inside a capture
            step_calls()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step_calls()
        torch.cuda.set_stream(stream)
        step = graph.replay

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    lory.lory_check_status(dims, ws)
    barrier()

    def timed_region(n_steps, per_kernel=False, settle=True):
        """n_steps back to back, device-resident inputs, CUDA events on the launch stream around the whole region;
        SM clocks sampled meanwhile.  per_kernel: the library's profiling hooks also put an event pair around every
        kernel (26 events per step, which cost 2-3 % of the step: the headline region runs without them).
        settle=False: no pause before the region (it follows another one and should see the same clocks)."""
        sampler = ClockSampler(local_rank)
        if rank == 0:
            sampler.start()
            if settle:
                time.sleep(0.3)
        lory.lory_profile_enable(per_kernel)
        run = step_calls if per_kernel else step   # a replayed graph holds no per-kernel events: plain launches there
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_wall0 = time.time()
        ev0.record()
        for _ in range(n_steps):
            run()
        ev1.record()
        barrier()
        t_wall1 = time.time()
        ms = ev0.elapsed_time(ev1)
        recs = lory.lory_profile_read()
        lory.lory_profile_enable(False)
        lory.lory_check_status(dims, ws)
        return ms, recs, (sampler.stop(t_wall0, t_wall1) if rank == 0 else None)

    ms_total, _, clocks = timed_region(args.steps)
    ms_per_step, value = aggregate_over_ranks(ms_total, args.steps, wl.tokens, world, dist, dev)
    # the same K steps once more with an event pair around every kernel: per-kernel times and shares
    ms_prof, records, clocks_prof = timed_region(args.steps, per_kernel=True)

    peaks = load_peaks()
    # Which measured tensor peak a run is compared with: the burst figure while the SM clock stays near its maximum
    # (a short timed region), the sustained one once the power cap has pulled the clock down (a long region).
    def regime(clk):
        if clk and clk.get("sm_mhz") and clk.get("sm_max_mhz") and clk["sm_mhz"] < 0.9 * clk["sm_max_mhz"]:
            return "sustained", peaks["bf16_tflops_sustained"]
        return "burst", peaks["bf16_tflops"]

    def kernel_stats(recs, n_steps, clk):
        """Per label: time, share, and the fraction of the roofline that bounds it (tensor peak for the
        contractions, HBM bandwidth over the method's own bytes for the streaming kernels)."""
        _, tensor_peak = regime(clk)
        per = {}
        for label, ms in recs:
            per.setdefault(label, []).append(ms)
        kf, mb, ib = kernel_flops(wl), method_bytes(wl), implementation_bytes(wl)
        tot = sum(sum(v) for v in per.values())
        out = {}
        for label, v in per.items():
            avg = sum(v) / len(v)
            ent = {"launches_per_step": len(v) / n_steps, "avg_ms": avg, "share": sum(v) / tot}
            if clk and clk.get("sm_mhz"):
                ent["ms_x_mhz"] = avg * clk["sm_mhz"]       # constant over clocks for a kernel bound on the SMs
            # flops / bytes are per step for a label (per launch for the three weight-gradient GEMMs); a label may
            # take several launches per step (one per 256 segments for the merge and its adjoint)
            t_step = sum(v) / n_steps / (3.0 if label == "wgrad" else 1.0) * 1e-3
            bound = KERNEL_BOUND.get(label)
            if label in kf:
                ent["tflops"] = kf[label] / t_step / 1e12
            if label in mb:
                ent["algorithmic_gbs"] = mb[label] / t_step / 1e9
            if label in ib:
                ent["implementation_gbs"] = ib[label] / t_step / 1e9
            if bound == "tensor":
                ent.update(bound="tensor", frac=ent["tflops"] / tensor_peak)
            elif bound == "hbm":
                ent.update(bound="hbm", frac=ent["algorithmic_gbs"] / peaks["hbm_gbs"])
            out[label] = ent
        return out

    kernels = kernel_stats(records, args.steps, clocks_prof)
    reg_name, tensor_peak = regime(clocks_prof)   # the per-kernel figures and `roofline` belong to the second region
    top = max(kernels, key=lambda k: kernels[k]["share"]) if kernels else None
    roofline = None
    if top is not None and kernels[top].get("bound"):
        e = kernels[top]
        traffic = measured_traffic(wl.name, top)
        alg_bytes = method_bytes(wl).get(top)
        roofline = {"kernel": top, "bound": e["bound"], "frac": e["frac"], "traffic": traffic,
                    "algorithmic_bytes": alg_bytes,
                    "traffic_ratio": (traffic / alg_bytes) if (traffic and alg_bytes) else None}
        if e["bound"] == "tensor":
            roofline.update(achieved=e["tflops"], peak=tensor_peak, unit="TFLOP/s",
                            peak_source=f"{peaks['source']} ({reg_name})")
        else:
            roofline.update(achieved=e["algorithmic_gbs"], peak=peaks["hbm_gbs"], unit="GB/s",
                            peak_source=peaks["source"])
    # the whole layer: Appendix B's flop count over the step time, against the slower of flops at the tensor peak
    # and compulsory bytes at the copy bandwidth
    F, CB = flops_per_step(wl), compulsory_bytes(wl)
    reg_name, tensor_peak = regime(clocks)        # the layer figures belong to the headline region
    t_roof = max(F / (tensor_peak * 1e12), CB / (peaks["hbm_gbs"] * 1e9))
    layer_tflops = F / (ms_per_step * 1e-3) / 1e12
    step_traffic = None
    ent = NCU_TRAFFIC.get(wl.name)
    if ent is not None and ent["sources_sha1"] == cuda_sources_sha1():
        step_traffic = sum(b * (3 if k == "wgrad" else 1) for k, b in ent["bytes"].items())
    layer = {"algorithmic_tflop_per_step": F / 1e12, "achieved_tflops": layer_tflops,
             "frac": t_roof / (ms_per_step * 1e-3), "frac_peak": f"{reg_name} bf16 peak, {peaks['source']}",
             "frac_of_burst_peak": layer_tflops / peaks["bf16_tflops"],
             "frac_of_sustained_peak": layer_tflops / peaks["bf16_tflops_sustained"],
             "compulsory_bytes": CB, "implementation_bytes": implementation_bytes_per_step(wl),
             "traffic": step_traffic, "traffic_ratio": (step_traffic / CB) if step_traffic else None}

    # ---- the same step held for at least a second: the power cap pulls the SM clock down ----
    sustained = None
    if not args.no_sustained:
        n_long = max(400, int(1.2e3 / ms_per_step))
        ms_long, _, clk_long = timed_region(n_long)
        ms_step_long, value_long = aggregate_over_ranks(ms_long, n_long, wl.tokens, world, dist, dev)
        tf_long = F / (ms_step_long * 1e-3) / 1e12
        # per-kernel times in the same regime: a shorter instrumented region straight after it
        n_k = min(100, PROF_RECORDS // max(1, launches[0]))
        _, rec_long, clk_k = timed_region(n_k, per_kernel=True, settle=False)
        k_long = kernel_stats(rec_long, n_k, clk_k)
        sustained = {"steps": n_long, "ms_per_step": ms_step_long, "value": value_long, "unit": UNIT,
                     "clocks": clk_long, "achieved_tflops": tf_long,
                     "frac_of_sustained_peak": tf_long / peaks["bf16_tflops_sustained"],
                     "kernels": {k: {kk: v[kk] for kk in ("avg_ms", "ms_x_mhz", "frac") if kk in v}
                                 for k, v in k_long.items()}}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- end to end through the host-buffer entry point --------------------------------------
    e2e = None
    if not args.no_e2e:
        xh, dyh = x.cpu().pin_memory(), dy.cpu().pin_memory()
        n_e2e = max(4, min(args.steps, 10))
        act = wl.tokens * wl.d * 2

        # (1) one synchronous call per step: the latency of a single step fed from the host
        arena = torch.empty(lory.lory_moe_step_host_bytes(dims), dtype=torch.uint8, device=dev)
        yh, dxh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
        rwh = torch.empty((wl.S, wl.E), dtype=torch.float32).pin_memory()
        for _ in range(3):
            lory.lory_moe_step_host(dims, xh, dyh, w_r, W1, W2, W3, yh, dxh, rwh, dw_r, dW1, dW2, dW3, arena)
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            lory.lory_moe_step_host(dims, xh, dyh, w_r, W1, W2, W3, yh, dxh, rwh, dw_r, dW1, dW2, dW3, arena)
        dt_serial = (time.perf_counter() - t0) / n_e2e
        del arena

        # (2) the two-slot pipeline a training loop uses: every step still copies its x, dY in and its y, dX,
        # routing weights out, but the copies of neighbouring steps overlap the kernels; the host reads each
        # step's routing weights as soon as the step has landed
        pipe_bytes = lory.lory_moe_step_host_pipeline_bytes(dims)
        arena = torch.empty(pipe_bytes, dtype=torch.uint8, device=dev)
        yh2 = [yh, torch.empty_like(xh).pin_memory()]
        dxh2 = [dxh, torch.empty_like(xh).pin_memory()]
        rwh2 = [rwh, torch.empty_like(rwh).pin_memory()]
        checksum = [0.0]

        def pipelined(n):
            for i in range(n):
                slot = i & 1
                if i >= 2:
                    lory.lory_moe_step_host_wait(slot)
                    checksum[0] += float(rwh2[slot][0, 0])
                lory.lory_moe_step_host_enqueue(dims, slot, xh, dyh, w_r, W1, W2, W3, yh2[slot], dxh2[slot],
                                                rwh2[slot], dw_r, dW1, dW2, dW3, arena)
            for slot in ((n - 2) & 1, (n - 1) & 1):
                lory.lory_moe_step_host_wait(slot)
                checksum[0] += float(rwh2[slot][0, 0])

        pipelined(4)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        pipelined(n_e2e)
        dt = (time.perf_counter() - t0) / n_e2e
        lory.lory_check_status(dims, arena[pipe_bytes - bwd_bytes:])
        e2e = {"value": world * wl.tokens / dt, "unit": UNIT, "h2d_bytes_per_step": 2 * act,
               "d2h_bytes_per_step": 2 * act + wl.S * wl.E * 4, "ms_per_step": dt * 1e3,
               "single_step_latency_ms": dt_serial * 1e3, "steps": n_e2e,
               "note": "lory_moe_step_host_enqueue/_wait, two slots: each step copies x, dY from pinned host memory "
                       "and y, dX, routing weights back; copies of neighbouring steps overlap the kernels; "
                       "single_step_latency_ms is the synchronous lory_moe_step_host; parameters and their "
                       "gradients stay on the device"}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        small, inp = oracle_sample(wl, 2)
        t = time_oracle(small, inp)
        reps = 1
        while t * reps < 10.0 and reps < 8:
            t = min(t, time_oracle(small, inp))
            reps += 1
        cpu = {"value": small.tokens / t, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"first 2 segments of one sequence ({small.tokens} tokens) of {wl.name}, oracle "
                         f"forward+backward in float64 (numpy/OpenBLAS), best of {reps}"}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": dict(workload_config(wl), **({"backward": "chunked adjoint (LORY_FLAG_CHUNKED_ADJOINT), workspace "
                                                f"{bwd_bytes / 1e9:.2f} GB"} if args.chunked_adjoint else {})),
        "clocks": clocks, "e2e": e2e,
        "gpu_launches": launches[0] * args.steps, "roofline": roofline, "cpu_baseline": cpu, "layer": layer,
        "sustained": sustained, "kernels": kernels,
        "kernels_note": "per-kernel times come from a second region of the same K steps, plain launches with a "
                        f"CUDA-event pair around every launch ({ms_prof / args.steps:.3f} ms per step that way)",
    }
    out["config"]["launch"] = ("one CUDA graph per step (lory_moe_forward + lory_moe_backward captured once), replayed"
                               if args.graph else "plain launches")
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
