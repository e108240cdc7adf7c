#!/usr/bin/env python
"""Benchmark of the MoE FFN layer forward (route -> permute -> hot/cold expert FFN ->
combine) on synthetic Switch / NLLB-shaped workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3|C2|C1|HOTPROBE|C4:...] [--impl ours|reference]

One JSON line on stdout (rank 0).  A step is one pass of the whole layer over one
batch of T tokens.  The headline workload is C3, the NLLB-MoE-like layer (the largest
stated single-GPU configuration); the same line carries, under `per_workload`, the same
measurements for C2 (the decode step the cold-streaming target is quoted on), C1 and the
compute-bound probe of the hot tiling (`--no-sub-workloads` leaves them out).  `value` is tokens/s with inputs resident in HBM; `e2e` is the
same layer called with the step's tokens in pinned host memory (H2D copy of x and
D2H copy of the output for every step inside the timed region; `binding.HostPipeline`
overlaps the copies of neighbouring steps with the compute, `e2e.serial_value` is the
unpipelined copy - compute - copy - wait figure).  `roofline` describes the dominant
call (the expert FFN) from CUDA events taken inside the timed region; `cpu_baseline`
is the fp64 CPU oracle timed on this host on a bounded sample of the same workload.

With N > 1 (launched under torchrun, one rank per GPU) every rank runs an independent
replica of the layer on its own batch: the path has no exchange step on one node, so
no collective is on the data path; only the barrier and the max-over-ranks of the
device time use torch.distributed.

`--impl reference` times the CPU oracle (the only reference implementation there is
for this paper: it published no code) on the host cores, on a bounded sample per step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2405_18832_b200 import synthetic as S  # noqa: E402

METRIC = "moe_ffn_layer_tokens_per_s"
UNIT = "tokens/s"

# DRAM bytes (read + write) of one launch of the dominant kernel.  Not measured in this run: taken
# from the ncu captures summarised under profiles/ (a profiler cannot run inside a timed benchmark).
# C3's weights (8.6 GB) are above the size a capture may hold, so its figure is C2's measured
# traffic per activated expert's weight byte (460.4 MB for 27 experts x 16.78 MB = 1.0163) times
# C3's own weight bytes; traffic grows in proportion because DRAM reads are the weights read once.
NCU_TRAFFIC = {
    "C1": (634.8e6, "profiles/expert_ffn_kernel_C1_C2.md (ncu, one launch), not this run"),
    "C2": (460.4e6, "profiles/expert_ffn_kernel_C1_C2.md (ncu, one launch), not this run"),
    "C3": (1.0163 * 128 * 2 * 2048 * 8192 * 2, "scaled from the C2 capture by activated weight bytes, not this run"),
    "HOTPROBE": (1.71e9, "profiles/expert_ffn_kernel_hot_probe.md (ncu, one launch), not this run"),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        m = json.load(open(path))
        return dict(hbm_gbs=float(m["hbm_gbs"]), bf16_tflops=float(m["bf16_tflops"]),
                    bf16_tflops_sustained=float(m.get("bf16_tflops_sustained", m["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def ffn_algorithmic_bytes(p: S.Problem, counts: np.ndarray) -> float:
    """Bytes the expert FFN must move: each activated expert's W1 and W2 once (Eq. 1 of the
    paper per expert: 2*d_model*d_ff parameters), x_perm read, h written and read, y_perm
    written, for every routed row."""
    s = p.elem_bytes
    active = int((counts > 0).sum())
    A = int(counts.sum())
    return active * 2.0 * p.d_model * p.d_ff * s + A * (2.0 * p.d_model + 2.0 * p.d_ff) * s


def ffn_flops(p: S.Problem, counts: np.ndarray) -> float:
    return 4.0 * float(counts.sum()) * p.d_model * p.d_ff


class ClockSampler:
    """SM clock and throttle reasons sampled through NVML (read-only) every millisecond on a thread
    while the timed region runs."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, uuid: str):
        import threading
        self.samples, self.bits, self.max_mhz, self.err = [], 0, None, None
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                pynvml.nvmlDeviceGetCurrentClocksThrottleReasons

            def loop():
                while not self._stop.is_set():
                    try:
                        self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        self.bits |= int(reasons_fn(h))
                    except Exception as e:   # keep the bench alive; report what happened
                        self.err = repr(e)
                        return
                    time.sleep(0.001)
            self._thread = threading.Thread(target=loop, daemon=True)
            self._thread.start()
        except Exception as e:
            self.err = repr(e)
            self._thread = None

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        reasons = sorted(n for bit, n in self.REASONS.items() if self.bits & bit)
        out = {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
               "samples": len(self.samples), "reasons": reasons}
        if self.err:
            out["error"] = self.err
        return out


def oracle_sample_run(w: S.Workload, host, n_tokens: int, nthreads: int = 0):
    """Whole layer through the CPU oracle on the first n_tokens tokens; returns seconds."""
    import oracle
    p = w.problem
    t0 = time.perf_counter()
    oracle.moe_layer(host["x"][:n_tokens], host["Wg"], host["bg"], host["W1"], host["b1"], host["W2"], host["b2"],
                     p.top_k, p.renormalize, p.hot_threshold, p.act, nthreads)
    return time.perf_counter() - t0


def host_inputs(g):
    return {k: S.as_numpy(v) for k, v in g.items()}


def pick_sample_tokens(w, host, target_s: float) -> int:
    import oracle
    cores = oracle.usable_cores()
    probe = min(w.problem.T, max(cores, 8))
    dt = oracle_sample_run(w, host, probe)
    n = int(probe * target_s / max(dt, 1e-6))
    return max(1, min(w.problem.T, n))


def generate_inputs(w: S.Workload, device):
    g = S.generate(w, with_weights=False)
    gw = S.generate(w, weights_device=device)
    for k in ("W1", "W2", "b1", "b2"):
        g[k] = gw[k]
    return g


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    host = host_inputs(generate_inputs(w, dev))
    cores = oracle.usable_cores()
    per_step = max(0.5, min(5.0, 150.0 / max(1, args.steps + args.warmup)))
    n_tok = pick_sample_tokens(w, host, per_step)
    for _ in range(args.warmup):
        oracle_sample_run(w, host, n_tok)
    t = [oracle_sample_run(w, host, n_tok) for _ in range(args.steps)]
    sec = sum(t) / len(t)
    value = n_tok / sec
    sample = f"whole layer on the first {n_tok} of {w.problem.T} tokens per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def dist_setup(backend: str, device=None):
    """Joins the process group that torchrun describes in the environment (one rank per GPU).
    Returns (dist module or None, rank, world, local_rank)."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1:
        return None, rank, world, local
    import torch.distributed as dist
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        dist.init_process_group(backend)
    return dist, rank, world, local


def max_over_ranks(dist, value: float, device="cpu") -> float:
    """Slowest rank's device time: what a job of independent replicas has to wait for."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_workload(w, rank: int, world: int):
    """Every replica gets its own batch (same layer, different tokens)."""
    if world == 1:
        return w
    import dataclasses
    return dataclasses.replace(w, seed=w.seed + 1000 * rank)


def aggregate_tokens_per_s(tokens_per_step_per_gpu: int, world: int, ms_per_step: float) -> float:
    return world * tokens_per_step_per_gpu / (ms_per_step * 1e-3)


def workload_config(w):
    p = w.problem
    return {"workload": f"{w.name}: E={p.E} top-{p.top_k} d_model={p.d_model} d_ff={p.d_ff} T={p.T} {p.dtype} "
                        f"{p.act} hot_threshold={p.hot_threshold} zipf_alpha={w.zipf_alpha}",
            "tokens_per_step_per_gpu": p.T, "seed": w.seed,
            "l2": "512 MiB scratch write between timed steps (L2 flush); active weights also exceed L2",
            "parallelism": "independent replicas, one per GPU, no data-path collective"}


def use_fused_combine(args, p) -> bool:
    """The layer is timed in the faster of its two bit-identical forms: FFN + combine in one call where that
    wins (top-1 routing, bf16: `binding.fused_combine_wins`), four calls otherwise; the flags force either."""
    from paper_2405_18832_b200 import binding as B
    if p.dtype != "bf16" or args.no_fuse_combine:
        return False
    return True if args.fuse_combine else B.fused_combine_wins(p)


def measure(args, w, dist, rank, world, dev, steps, with_cpu_baseline, weights=None, light=False):
    """All measurements of one workload on this rank's GPU; returns the result record (rank 0) or None.
    `weights`: expert weights already on the device (same seed and shapes), `light`: no host-buffer runs."""
    from paper_2405_18832_b200 import binding as B
    p = w.problem
    w = replica_workload(w, rank, world)
    if weights is None:
        g = generate_inputs(w, dev)
    else:
        g = S.generate(w, with_weights=False)
        g.update(weights)
    d = {k: (None if v is None else v.to(dev)) for k, v in g.items()}
    buf = B.LayerBuffers(p, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)      # four times the 126 MB L2
    stream = torch.cuda.current_stream()
    L = B.lib()
    warmup = max(args.warmup, 3)

    fuse = use_fused_combine(args, p)

    def layer(ev=None):
        if ev is not None:
            ev[0].record(stream)
        B.monde_route(p, d["x"], d["Wg"], d["bg"], buf.topk_idx, buf.topk_w, buf.counts, buf.offsets, buf.cls,
                      buf.hot_ids, buf.cold_ids, buf.n_hot_cold, None, buf.ws)
        if args.policy == "top_h":     # the paper's placement rule replaces the threshold classes
            B.monde_classify_top_h(p, buf.counts, args.alpha, args.bw_hot, args.bw_cold, buf.cls, buf.hot_ids,
                                   buf.cold_ids, buf.n_hot_cold)
        if ev is not None:
            ev[1].record(stream)
        B.monde_permute(p, d["x"], buf.topk_idx, buf.offsets, buf.perm, buf.inv_perm, buf.x_perm, buf.ws)
        if ev is not None:
            ev[2].record(stream)
        if fuse:       # three-call form: the FFN's last store applies the gate weight and writes `out`
            B.monde_moe_ffn_combine_fwd(p, buf.x_perm, d["W1"], d["b1"], d["W2"], d["b2"], buf.counts, buf.offsets,
                                        buf.cls, buf.perm, buf.topk_w, buf.out, buf.ws)
            if ev is not None:
                ev[3].record(stream)
                ev[4].record(stream)
            return
        B.monde_moe_ffn_fwd(p, buf.x_perm, d["W1"], d["b1"], d["W2"], d["b2"], buf.counts, buf.offsets, buf.cls,
                            buf.hot_ids, buf.cold_ids, buf.n_hot_cold, buf.y_perm, buf.ws)
        if ev is not None:
            ev[3].record(stream)
        B.monde_combine(p, buf.y_perm, buf.inv_perm, buf.topk_w, buf.out)
        if ev is not None:
            ev[4].record(stream)

    for _ in range(warmup):
        flush.fill_(1)
        layer()
    B.monde_poll_device_status(buf.ws)
    counts = buf.counts.cpu().numpy()
    n_hot_used = int(buf.n_hot_cold.cpu()[0])

    # ---- timed region: device-resident inputs --------------------------------------
    # Events bracket whole steps only: the four calls overlap through programmatic dependent
    # launch, and an event recorded between two calls would serialise them.
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    switch_interval = sys.getswitchinterval()
    sys.setswitchinterval(2e-4)      # let the sampling thread run while this one enqueues work
    launches0 = L.monde_kernel_launches()
    wall0 = time.perf_counter()
    for a, b in events:
        flush.fill_(1)
        a.record(stream)
        layer()
        b.record(stream)
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    launches = L.monde_kernel_launches() - launches0
    if dist is not None:
        dist.barrier()
    B.monde_poll_device_status(buf.ws)
    step_ms = [a.elapsed_time(b) for a, b in events]
    total_ms = max_over_ranks(dist, sum(step_ms), dev)
    ms_per_step = total_ms / steps
    value = aggregate_tokens_per_s(p.T, world, ms_per_step)

    # ---- per-call pass: the same K steps again with an event between the calls, which gives
    # each call's own duration (and the dominant kernel's, for the roofline) at the price of
    # the overlap between calls.  The clock sampler keeps running: same load, more samples.
    call_events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
    for ev in call_events:
        flush.fill_(2)
        layer(ev)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    sys.setswitchinterval(switch_interval)
    call_ms = [[e[i].elapsed_time(e[i + 1]) for e in call_events] for i in range(4)]
    # What a pair of events around ONE call costs by itself: the routing call of an empty batch launches a
    # single one-CTA kernel that writes a few hundred bytes.  Every per-call figure above contains this much
    # launch and event latency; the back-to-back step does not (its calls overlap).
    import dataclasses
    p0 = dataclasses.replace(p, T=0)
    buf0 = B.LayerBuffers(p0, device=dev)
    floor_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
    for _ in range(8):          # half a millisecond of queued work first, so that the GPU, not the host, paces the events
        flush.fill_(4)
    for a, b in floor_ev:
        a.record(stream)
        B.monde_route(p0, buf0.x_dev, d["Wg"], d["bg"], buf0.topk_idx, buf0.topk_w, buf0.counts, buf0.offsets, buf0.cls,
                      buf0.hot_ids, buf0.cold_ids, buf0.n_hot_cold, None, buf0.ws)
        b.record(stream)
    torch.cuda.synchronize()
    call_floor_ms = statistics.median(a.elapsed_time(b) for a, b in floor_ev)

    e2e = None
    if not light:
        e2e = measure_host_buffers(B, p, g, d, buf, flush, stream, steps, warmup, dist, dev, world, fuse)
    del flush

    if rank != 0:
        return None
    rec = summarise(args, w, p, counts, n_hot_used, steps, warmup, world, ms_per_step, step_ms, call_ms, value, clocks,
                    launches, wall, e2e, g, with_cpu_baseline)
    rec["calls_ms"]["empty_call_floor"] = call_floor_ms
    return rec


def measure_host_buffers(B, p, g, d, buf, flush, stream, steps, warmup, dist, dev, world, fuse):
    # ---- end to end: tokens in pinned host memory ----------------------------------
    # Every step copies its tokens host -> device and its result device -> host.  Serial form:
    # copy, four calls, copy, wait (per-step latency).  Pipelined form (the e2e figure): the same
    # work per step on three streams, so the copies of neighbouring steps overlap the compute;
    # timed from before the first copy in to after the last copy out.  No L2 flush in this loop:
    # the weights streamed by one step are several times the L2 and the tokens arrive by DMA.
    x_host = g["x"].pin_memory()
    out_host = torch.empty((p.T, p.d_model), dtype=p.torch_dtype).pin_memory()
    for _ in range(3):
        B.moe_ffn_layer_forward_host(p, x_host, out_host, d["Wg"], d["bg"], d["W1"], d["b1"], d["W2"], d["b2"], buf,
                                     fuse_combine=fuse)
    e2e_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    torch.cuda.synchronize()
    for a, b in e2e_ev:
        flush.fill_(3)
        a.record(stream)
        B.moe_ffn_layer_forward_host(p, x_host, out_host, d["Wg"], d["bg"], d["W1"], d["b1"], d["W2"], d["b2"], buf,
                                     fuse_combine=fuse)
        b.record(stream)
    torch.cuda.synchronize()
    serial_ms = max_over_ranks(dist, sum(a.elapsed_time(b) for a, b in e2e_ev), dev)
    e2e_serial_value = aggregate_tokens_per_s(p.T, world, serial_ms / steps)
    assert torch.equal(out_host, buf.out.cpu())

    pipe = B.HostPipeline(p, depth=2, device=dev, fuse_combine=fuse)
    weights = (d["Wg"], d["bg"], d["W1"], d["b1"], d["W2"], d["b2"])
    out_host.zero_()
    for _ in range(warmup):
        pipe.submit(x_host, out_host, *weights)
    pipe.wait()
    torch.cuda.synchronize()
    p_start, p_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    p_start.record(pipe.s_in)
    for _ in range(steps):
        pipe.submit(x_host, out_host, *weights)
    p_end.record(pipe.s_out)
    pipe.wait()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(dist, p_start.elapsed_time(p_end), dev)
    e2e_value = aggregate_tokens_per_s(p.T, world, e2e_ms / steps)
    assert torch.equal(out_host, buf.out.cpu())
    del pipe
    return {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": x_host.numel() * x_host.element_size(),
            "d2h_bytes_per_step": out_host.numel() * out_host.element_size(),
            "mode": "pipelined over 3 streams, 2 buffer sets: every step does its own H2D, 4 calls and D2H",
            "serial_value": e2e_serial_value, "ms_per_step": e2e_ms / steps}


def summarise(args, w, p, counts, n_hot_used, steps, warmup, world, ms_per_step, step_ms, call_ms, value, clocks, launches,
              wall, e2e, g, with_cpu_baseline):
    fuse = use_fused_combine(args, p)
    peaks = measured_peaks()
    ffn_ms = statistics.mean(call_ms[2])
    bytes_ffn = ffn_algorithmic_bytes(p, counts)
    achieved = bytes_ffn / (ffn_ms * 1e-3) / 1e9
    tflops = ffn_flops(p, counts) / (ffn_ms * 1e-3) / 1e12
    traffic, traffic_source = NCU_TRAFFIC.get(w.name, (None, "no capture for this workload"))
    tensor_bound = w.name == "HOTPROBE"      # the one workload whose experts sit far above the ridge
    common = {"kernel": "expert_ffn_kernel via " + ("monde_moe_ffn_combine_fwd (hot + cold expert FFN, both layers, gate "
                                                    "weight applied in the last store)" if fuse else
                                                    "monde_moe_ffn_fwd (hot + cold expert FFN, both layers)"),
              "peak_source": peaks["source"], "traffic": traffic, "traffic_source": traffic_source,
              "algorithmic_bytes": bytes_ffn, "algorithmic_flops": ffn_flops(p, counts), "ms": ffn_ms,
              "units_per_launch": int((counts > 0).sum()), "unit": "GB/s",
              "timing": "CUDA events around the call on its stream, per-call pass of the same K steps",
              "hbm_gbs": achieved, "hbm_frac_of_measured": achieved / peaks["hbm_gbs"],
              "hbm_frac_of_nominal_8000": achieved / 8000.0,
              "tflops": tflops, "tensor_frac_of_measured_burst": tflops / peaks["bf16_tflops"],
              "tensor_frac_of_nominal_2250": tflops / 2250.0}
    if tensor_bound:
        roofline = dict(common, bound="tensor", achieved=tflops, peak=peaks["bf16_tflops"], unit="TFLOP/s",
                        frac=tflops / peaks["bf16_tflops"])
    else:
        roofline = dict(common, bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], frac=achieved / peaks["hbm_gbs"])
    elementwise_bytes = (2 * p.A + 2 * p.T) * p.d_model * p.elem_bytes + p.T * p.d_model * p.elem_bytes
    layer_floor_ms = (bytes_ffn + elementwise_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3

    def layer_lower_bound_ms(tflops_peak, gbs):
        # per activated expert the slower of its flops at the tensor peak and its bytes at the HBM peak,
        # plus the elementwise stages' bytes (router input, gather, combine)
        m = counts[counts > 0].astype(np.float64)
        flops_e = 4.0 * m * p.d_model * p.d_ff
        bytes_e = 2.0 * p.d_model * p.d_ff * p.elem_bytes + m * (2.0 * p.d_model + 2.0 * p.d_ff) * p.elem_bytes
        return (np.maximum(flops_e / (tflops_peak * 1e12), bytes_e / (gbs * 1e9)).sum()
                + elementwise_bytes / (gbs * 1e9)) * 1e3

    lb_measured = layer_lower_bound_ms(peaks["bf16_tflops"], peaks["hbm_gbs"])
    lb_nominal = layer_lower_bound_ms(2250.0, 8000.0)

    # ---- CPU baseline: the oracle as it stands, on a bounded sample ------------------
    cpu = None
    if with_cpu_baseline and world == 1:
        import oracle
        host = host_inputs(g)
        n_tok = pick_sample_tokens(w, host, 12.0)
        sec = oracle_sample_run(w, host, n_tok)
        n_one = max(1, min(n_tok, int(n_tok / sec * 3.0 / max(oracle.usable_cores(), 1))))   # about 3 s on one thread
        sec_one = oracle_sample_run(w, host, n_one, nthreads=1)
        cpu = {"value": n_tok / sec, "unit": UNIT, "cores": oracle.usable_cores(), "kind": "oracle",
               "sample": f"whole layer on the first {n_tok} of {p.T} tokens, {sec:.1f} s",
               "one_thread": {"value": n_one / sec_one, "sample": f"first {n_one} tokens, {sec_one:.1f} s"}}
        del host

    return {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": p.dtype, "data": "synthetic", "config": workload_config(w),
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": launches,
        "roofline": roofline, "cpu_baseline": cpu,
        "calls_ms": {"route": statistics.mean(call_ms[0]), "permute": statistics.mean(call_ms[1]),
                     "ffn": ffn_ms, "combine": 0.0 if fuse else statistics.mean(call_ms[3])},
        "calls_ms_sum": sum(statistics.mean(c) for c in call_ms[:3 if fuse else 4]),
        # whole step against the layer's roofline (per expert the slower of its flops and its bytes, measured
        # peaks); the bytes-only floor is kept beside it: the two differ only for a compute-bound workload
        "layer_hbm_floor_ms": layer_floor_ms, "layer_hbm_floor_frac": layer_floor_ms / ms_per_step,
        "layer_roofline_frac": lb_measured / ms_per_step,
        "layer_lower_bound": {"formula": "sum over activated experts of max(flops / tensor peak, bytes / HBM peak) "
                                         "+ elementwise bytes / HBM peak",
                              "ms_of_measured_peaks": lb_measured, "frac_of_measured": lb_measured / ms_per_step,
                              "ms_of_nominal_peaks": lb_nominal, "frac_of_nominal": lb_nominal / ms_per_step},
        "step_ms": {"mean": ms_per_step, "median": statistics.median(step_ms), "min": min(step_ms)},
        "calls": "route, permute, ffn+combine (fused last store)" if fuse else "route, permute, ffn, combine",
        "policy": args.policy if args.policy == "threshold" else
        f"top_h alpha={args.alpha} bw_hot={args.bw_hot} bw_cold={args.bw_cold}",
        "routing": {"active": int((counts > 0).sum()), "hot": n_hot_used,
                    "max_count": int(counts.max()), "assignments": int(counts.sum())},
        "wall_s_timed_region": wall,
    }


SUB_WORKLOADS = ("C2", "C1", "HOTPROBE")
SUB_KEYS = ("value", "unit", "steps", "ms_per_step", "config", "clocks", "e2e", "roofline", "calls_ms", "calls_ms_sum",
            "layer_lower_bound", "layer_roofline_frac", "layer_hbm_floor_frac", "step_ms", "routing", "gpu_launches", "calls")


def sub_steps(name: str, steps: int) -> int:
    """Steps of a sub-workload: at least the headline's K, and enough of them that the timed region
    spans some 40 ms, so that the clock record has a dozen samples even for a 0.1 ms step."""
    floor_ms = {"C1": 0.16, "C2": 0.11, "HOTPROBE": 1.0}.get(name, 1.0)
    return max(steps, int(40.0 / floor_ms))


SWEEP_D = (1024, 2048, 4096)
SWEEP_T = (1, 8, 64, 512, 4096)
SWEEP_ALPHA = (0.0, 1.2)
SWEEP_THETA = (4, 16, 64)


def run_sweep(args):
    """The crossover sweep (E=64, top-2, d_ff = 4 d_model, GELU): all 90 points, one JSON line each appended
    to `--sweep-out`; points already in the file are skipped, so an interrupted sweep resumes."""
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    done = set()
    if os.path.exists(args.sweep_out):
        for ln in open(args.sweep_out):
            try:
                r = json.loads(ln)
                done.add((r["d_model"], r["T"], r["zipf_alpha"], r["hot_threshold"]))
            except Exception:
                pass
    os.makedirs(os.path.dirname(os.path.abspath(args.sweep_out)), exist_ok=True)
    for d_model in SWEEP_D:
        weights = None
        for T in SWEEP_T:
            for alpha in SWEEP_ALPHA:
                for theta in SWEEP_THETA:
                    if (d_model, T, alpha, theta) in done:
                        continue
                    w = S.sweep_point(d_model, T, alpha, theta)
                    if weights is None:      # same seed and tensor ids at every point of this d_model
                        gw = S.generate(w, weights_device=dev)
                        weights = {k: gw[k] for k in ("W1", "W2", "b1", "b2")}
                    steps = max(args.steps, int(20.0 / (0.08 + 3.0e-8 * T * d_model)))    # about 20 ms of timed steps at least
                    rec = measure(args, w, None, 0, 1, dev, min(steps, 200), False, weights=weights, light=True)
                    ro = rec["roofline"]
                    row = {"d_model": d_model, "T": T, "zipf_alpha": alpha, "hot_threshold": theta,
                           "active": rec["routing"]["active"], "hot": rec["routing"]["hot"],
                           "max_count": rec["routing"]["max_count"], "steps": rec["steps"],
                           "layer_us": rec["ms_per_step"] * 1e3, "ffn_us": ro["ms"] * 1e3,
                           "calls_us": {k: v * 1e3 for k, v in rec["calls_ms"].items()},
                           "ffn_hbm_frac_of_measured": ro["hbm_frac_of_measured"], "ffn_tflops": ro["tflops"],
                           "ffn_tensor_frac_of_measured_burst": ro["tensor_frac_of_measured_burst"],
                           "layer_lower_bound_frac_of_measured": rec["layer_lower_bound"]["frac_of_measured"],
                           "layer_lower_bound_frac_of_nominal": rec["layer_lower_bound"]["frac_of_nominal"],
                           "cold_kernel": "tcgen05 weight-streaming tiling (no CUDA-core FMA arm exists)",
                           "sm_mhz": rec["clocks"]["sm_mhz"], "clock_reasons": rec["clocks"]["reasons"]}
                    with open(args.sweep_out, "a") as f:
                        f.write(json.dumps(row) + "\n")
                    print(json.dumps(row), flush=True)
                    torch.cuda.empty_cache()
        del weights
        torch.cuda.empty_cache()


def run_ours(args, w):
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    dist, rank, world, local = dist_setup("nccl")
    dev = torch.device("cuda", local)
    line = measure(args, w, dist, rank, world, dev, args.steps, not args.no_cpu_baseline)
    if not args.no_sub_workloads and w.name == "C3":
        per = {}
        for name in SUB_WORKLOADS:
            torch.cuda.empty_cache()
            rec = measure(args, S.config(name), dist, rank, world, dev, sub_steps(name, args.steps), False)
            if rec is not None:
                per[name] = {k: rec[k] for k in SUB_KEYS}
        if line is not None:
            line["per_workload"] = per
    if line is not None:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="C3",
                    help="C3 (default, with C2 / C1 / HOTPROBE as sub-records), C2, C1, HOTPROBE, or a crossover-sweep "
                         "point C4:<d_model>:<T>:<zipf alpha>:<threshold>")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sub-workloads", action="store_true",
                    help="headline workload only (no per_workload records for C2, C1 and the hot-tiling probe)")
    ap.add_argument("--sweep", action="store_true",
                    help="run the 90-point crossover sweep (resumable) instead of a single workload")
    ap.add_argument("--sweep-out", default=os.path.join(ROOT, "gpurun_out", "sweep_C4.jsonl"))
    ap.add_argument("--fuse-combine", action="store_true",
                    help="bf16 workloads: always monde_moe_ffn_combine_fwd (default: where it is the faster form, top-1)")
    ap.add_argument("--no-fuse-combine", action="store_true",
                    help="always the four-call form: monde_moe_ffn_fwd + monde_combine")
    ap.add_argument("--policy", default="threshold", choices=["threshold", "top_h"],
                    help="hot/cold rule: count >= hot_threshold, or the paper's top-H rule (Eq. 6)")
    ap.add_argument("--alpha", type=float, default=1.0, help="Eq. 6 tuning factor (top_h)")
    ap.add_argument("--bw-hot", type=float, default=3.9, help="TB/s at which the hot tiling consumes weights (top_h)")
    ap.add_argument("--bw-cold", type=float, default=7.0, help="TB/s at which the cold tiling streams weights (top_h)")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.workload.startswith("C4:"):
        _, d_model, T, zipf, theta = args.workload.split(":")
        w = S.sweep_point(int(d_model), int(T), float(zipf), int(theta))
    else:
        w = S.config(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
