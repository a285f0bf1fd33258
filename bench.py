#!/usr/bin/env python
"""LASAD operator benchmark on B200: prefill tokens/s and decode us/step against the rooflines.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A *step* is one full-sequence prefill (`lasad_forward`) over the prefill workload; the headline
`value` is prefill tokens/s with inputs resident in HBM.  The same run then times the decode
workload (`lasad_decode_step`, one sweep = one step per grid position against the persistent
fp32 state) in its own region and reports it under "decode".  One JSON line goes to stdout.

Multi-GPU (torchrun, one rank per GPU): the operator has no cross-(batch, head) term, so every
rank runs the same per-GPU workload on its own seed with no data-path collective ("weak"
scaling); the time is the max over ranks and `value` sums all ranks' tokens.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum per launch) from the ncu captures
# summarised under profiles/; None until a capture of that kernel exists.
NCU_TRAFFIC_BYTES = {
    # prefill_pair_kernel (the default on config 5b): 385.4 MB measured on the 405.8 MB capture case
    # (config 5a), scaled by tokens to config 5b
    "prefill": 863_400_000,
    # decode_kernel, config 4, inside the kernel (the rest of the written state drains from L2 later)
    "decode": 112_500_000,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "source": "measured"}
    return {**FALLBACK_PEAKS, "source": "fallback"}


# --------------------------------------------------------------------------------------------
# clocks under load (read-only NVML polling in a thread)
# --------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.001):
        self.period = period_s
        self.samples, self.reason_bits = [], 0
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            self._nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # NVML unavailable: report that instead of inventing numbers
            self.error = repr(e)
            self._h = None

    def _poll(self):
        nv = self._nv
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(get_reasons(self._h))
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._h is not None:
            self._stop.clear()
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self):
        if self._h is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [],
                    "note": "NVML clocks unavailable: " + getattr(self, "error", "no samples")}
        reasons = sorted(name for bit, name in self.REASONS.items() if self.reason_bits & bit)
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------
# multi-rank bookkeeping (replicas only: no data-path collective)
# --------------------------------------------------------------------------------------------
def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own replica of the workload."""
    return base_seed + 1000 * rank


def max_over_ranks(x: float, world: int, device) -> float:
    """Slowest rank's time (the only value exchanged between ranks)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist

    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world: int, ms_per_step: float) -> float:
    """Units processed by all ranks per second, given the slowest rank's time per step."""
    return world * units_per_rank / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------------------------
# algorithmic traffic
# --------------------------------------------------------------------------------------------
def prefill_bytes(wl) -> int:
    """q, k, v read once and o written once, plus the final fp32 state."""
    return wl.B * wl.T * wl.H * 4 * wl.d * wl.elem_bytes + wl.B * wl.H * wl.d * wl.d * 4


def prefill_flops(wl, chunk: int) -> int:
    """Executed flops of the chunked method with dense C x C tiles: 4 dk dv + 2 C (dk + dv)."""
    return wl.B * wl.T * wl.H * (4 * wl.d * wl.d + 2 * chunk * 2 * wl.d)


def decode_bytes(wl) -> int:
    """fp32 state read + written, q, k, v read and o written, per step."""
    return wl.B * wl.H * (8 * wl.d * wl.d + 4 * wl.d * wl.elem_bytes)


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2507_01652_b200 import binding, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the LASAD operator has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_ranks(x: float) -> float:
        return max_over_ranks(x, world, dev)

    peaks = load_peaks()
    ctx = binding.Lasad(local)
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, args.prefill_impl)
    K, W = args.steps, max(args.warmup, 3)
    wl = workloads.WORKLOADS[args.prefill_workload]
    if args.prefill_batch:
        wl = wl.scaled(B=args.prefill_batch)
    wl = dataclasses.replace(wl, seed=rank_seed(wl.seed, rank))
    stream = torch.cuda.current_stream()
    if args.only == "decode":
        dec = run_decode(args, ctx, peaks, dev, rank, barrier, max_ranks, K)
        if rank == 0:
            print(json.dumps({"decode": dec}), flush=True)
        ctx.close()
        return
    if args.only == "gated":
        res = gated_sweep(ctx, peaks, dev, [wl], decode=False, reps=K)
        if rank == 0:
            print(json.dumps({"gated": res}), flush=True)
        ctx.close()
        return

    # ---- prefill: inputs resident in HBM -------------------------------------------------
    hq, hk, hv = [t.pin_memory() for t in workloads.make_qkv(wl)]
    g = workloads.make_decay(wl).to(dev)
    q, k, v = hq.to(dev), hk.to(dev), hv.to(dev)
    o = torch.empty_like(v)
    s_out = torch.empty(wl.B, wl.H, wl.d, wl.d, dtype=torch.float32, device=dev)
    fwd = lambda: ctx.lasad_forward(q, k, v, g, wl.grid_w, prefix_len=wl.prefix_len, o=o,
                                    state_out=s_out)
    for _ in range(W):
        fwd()
    # One CUDA-event pair around the K back-to-back launches: nothing but the kernels sits between
    # them on the stream (an event record between two launches would serialise them fully, and the
    # prefill kernel lets the next launch's CTAs set up on SMs it has already left).
    t_beg, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    n0 = ctx.launch_count
    barrier()
    with sampler:
        t_beg.record(stream)
        for _ in range(K):
            fwd()
        t_end.record(stream)
        torch.cuda.synchronize()
    barrier()
    launches = ctx.launch_count - n0
    assert ctx.device_status() == 0, "a device-side wait timed out during the timed region"
    total_ms = max_ranks(t_beg.elapsed_time(t_end))
    ms_per_step = total_ms / K
    kern_ms = ms_per_step          # average launch duration over the timed region (one launch per step)
    tokens_per_step = wl.B * wl.T
    value = whole_job_rate(tokens_per_step, world, ms_per_step)
    pf_bytes = prefill_bytes(wl)
    achieved = pf_bytes / (kern_ms * 1e-3) / 1e9
    chunk = args.chunk_for_flops
    tc_tflops = prefill_flops(wl, chunk) / (kern_ms * 1e-3) / 1e12

    # ---- prefill end to end: host buffers through the C ABI (lasad_forward_host): the copies of
    #      q, k, v in and of o out are inside the timed region, pipelined with the kernels ------
    ho = torch.empty(o.shape, dtype=o.dtype).pin_memory()
    hg = g.cpu().pin_memory()
    Ke = max(3, min(K, 20))

    def e2e_step():
        ctx.lasad_forward_host(hq, hk, hv, hg, wl.grid_w, ho, prefix_len=wl.prefix_len)

    for _ in range(2):
        e2e_step()
    barrier()
    e_beg, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_beg.record(stream)
    for _ in range(Ke):
        e2e_step()
    e_end.record(stream)
    torch.cuda.synchronize()
    barrier()
    e2e_ms = max_ranks(e_beg.elapsed_time(e_end)) / Ke
    e2e_ok = bool(torch.equal(ho, o.cpu()))     # same bytes as the device-resident path produced
    h2d = 3 * hq.numel() * hq.element_size()
    d2h = ho.numel() * ho.element_size()
    del hq, hk, hv, ho, q, k, v, o
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)

    # ---- the other prefill configurations (context for the headline; rank 0 reports) ----------
    sweep = None
    if args.only == "all" and not args.no_sweep:
        sweep = prefill_sweep(ctx, peaks, dev, ("config1", "config2", "config3", "config5a", "config5b@1"))
    gated = None
    if args.only == "all" and not args.no_sweep:
        gated = gated_sweep(ctx, peaks, dev)

    decode = None
    decode_others = None
    if args.only != "prefill":
        decode = run_decode(args, ctx, peaks, dev, rank, barrier, max_ranks, K)
        if args.only == "all" and not args.no_sweep:
            decode_others = [run_decode(args, ctx, peaks, dev, rank, barrier, max_ranks, K, workload=name, hot=False)
                             for name in ("config2", "config3")]
    host_cost = None
    scaling = None
    if args.only == "all" and not args.no_sweep and rank == 0:
        host_cost = host_cost_per_call(ctx, dev)
        scaling = scaling_sweep(ctx, dev, cpu=(world == 1 and not args.no_cpu_baseline))

    # ---- CPU baseline: the oracle as it stands on this machine's host cores (rank 0, N = 1) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(wl)

    # ---- the headline workload again, launched back to back for seconds: what the board's power
    #      limit leaves of the short timed region's rate (last, so that nothing above runs warm) ----
    sustained = None
    if args.only == "all" and not args.no_sweep and rank == 0 and args.sustained_seconds > 0:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, args.prefill_impl)
        sustained = sustained_prefill(ctx, wl, peaks, dev, seconds=args.sustained_seconds)

    if rank == 0:
        line = {
            "metric": "lasad_prefill_tokens_per_s", "value": round(value, 1), "unit": "tokens/s",
            "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": round(ms_per_step, 5),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": f"{wl.name}: B={wl.B} H={wl.H} T={wl.T} ({wl.grid_h}x{wl.grid_w} grid) "
                                   f"d_k=d_v={wl.d}, {wl.dtype} I/O, fp32 accumulate and state",
                       "prefill_impl": args.prefill_impl, "per_gpu_tokens": tokens_per_step, "parallelism": f"replicated x{world}, no collective",
                       "l2_policy": "inputs larger than L2 (q,k,v,o = %.0f MB)" % (pf_bytes / 1e6)},
            "e2e": {"value": round(whole_job_rate(tokens_per_step, world, e2e_ms), 1), "unit": "tokens/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 4),
                    "api": "lasad_forward_host (pinned host buffers, copies pipelined per batch element)",
                    "matches_device_path": e2e_ok,
                    "steps": Ke},
            "gpu_launches": int(launches),
            "clocks": sampler.summary(),
            "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": round(achieved / peaks["hbm_gbs"], 4),
                         "traffic": NCU_TRAFFIC_BYTES["prefill"] if (wl.name == "config5b" and args.prefill_impl in (0, 5)) else None,
                         "peak_source": peaks["source"],
                         "kernel_ms": round(kern_ms, 5), "bytes_per_launch": pf_bytes,
                         "timed": "one CUDA-event pair around the K back-to-back launches of the timed region, divided by K"},
            "tensor": {"executed_tflops": round(tc_tflops, 1), "chunk": chunk,
                       "frac_of_bf16_peak": round(tc_tflops / peaks["bf16_tflops"], 4)},
            "decode": decode,
            "decode_other_configs": decode_others,
            "host_us_per_call": host_cost,
            "prefill_vs_n": scaling,
            "prefill_sustained": sustained,
            "prefill_sweep": sweep,
            "gated": gated,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


L2_BYTES = 126 << 20


class L2Flush:
    """Keeps a launch from finding its inputs in L2.  Workloads whose tensors exceed twice the L2
    need nothing (back-to-back launches: what one launch leaves in L2 is the end of its data, the
    next one starts at the beginning).  For smaller ones a 256 MiB buffer is READ between launches
    (a reduction kernel): that fills L2 with clean lines, so the timed kernel neither hits its
    inputs nor has to wait for dirty lines of the flush to drain to DRAM."""

    def __init__(self, dev):
        import torch
        self.words = torch.zeros(32 << 20, dtype=torch.int64, device=dev)

    def policy(self, nbytes: int) -> str:
        return "back-to-back launches (tensors larger than 2x L2)" if nbytes > 2 * L2_BYTES else \
            "256 MiB read between launches"

    def __call__(self, nbytes: int):
        if nbytes <= 2 * L2_BYTES:
            self.words.sum()


def prefill_sweep(ctx, peaks, dev, names, reps: int = 10):
    """Kernel time of one prefill per named workload (CUDA events around each launch, median of
    `reps`), with the L2 policy of `L2Flush`."""
    import torch

    from paper_2507_01652_b200 import workloads

    stream = torch.cuda.current_stream()
    flush = L2Flush(dev)
    out = []
    for name in names:
        # "name@B": the named workload at another batch size (e.g. one image at a time)
        wl = workloads.WORKLOADS[name.split("@")[0]]
        if "@" in name:
            wl = wl.scaled(B=int(name.split("@")[1]))
        q, k, v = [t.to(dev) for t in workloads.make_qkv(wl)]
        g = workloads.make_decay(wl).to(dev)
        o = torch.empty_like(v)
        s_out = torch.empty(wl.B, wl.H, wl.d, wl.d, dtype=torch.float32, device=dev)
        nbytes = prefill_bytes(wl)
        ms = _time_launches(stream, flush, nbytes, reps,
                            lambda: ctx.lasad_forward(q, k, v, g, wl.grid_w, prefix_len=wl.prefix_len, o=o, state_out=s_out))
        out.append({"workload": f"{wl.name}: B={wl.B} H={wl.H} T={wl.T} d={wl.d} {wl.dtype}",
                    "kernel_us": round(ms * 1e3, 2), "tokens_per_s": round(wl.B * wl.T / (ms * 1e-3), 1),
                    "algorithmic_gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                    "frac_of_hbm_peak": round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                    "l2_policy": flush.policy(nbytes)})
        del q, k, v, o, s_out
    return out


def _time_launches(stream, flush, nbytes, reps, launch):
    """CUDA-event time (ms) of one `launch()`: for workloads that need the L2 cleared, the median over
    `reps` launches, each between its own pair of events behind the clearing read; for workloads
    larger than twice the L2, `reps` back-to-back launches between one pair of events, divided by
    `reps` (as the main timed region does).  3 warm-up launches either way."""
    import torch

    if nbytes > 2 * L2_BYTES:
        for _ in range(3):
            launch()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            launch()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps
    evs = []
    for it in range(reps + 3):
        flush(nbytes)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        launch()
        b.record(stream)
        if it >= 3:
            evs.append((a, b))
    torch.cuda.synchronize()
    return statistics.median(a.elapsed_time(b) for a, b in evs)


def gated_sweep(ctx, peaks, dev, wls=None, decode: bool = True, reps: int = 10):
    """The data-dependent (gated) form: time of one prefill call (tensor-core kernel plus the
    CUDA-core kernel behind it that redoes flagged chains; L2 flushed between calls) on the
    config 2, 3 and 5b shapes and of one decode step on the config 4 shape (rotating state
    sets), with a seeded logistic-normal gate and the key given explicitly."""
    import torch

    from paper_2507_01652_b200 import workloads

    stream = torch.cuda.current_stream()
    flush = L2Flush(dev)
    out = {"prefill": [], "decode": None}
    if wls is None:
        wls = [workloads.WORKLOADS[name] for name in ("config2", "config3", "config5b")]
    for wl in wls:
        q, k, v = [t.to(dev) for t in workloads.make_qkv(wl)]
        lam = workloads.make_gate(wl).to(dev)
        o = torch.empty_like(v)
        s_out = torch.empty(wl.B, wl.H, wl.d, wl.d, dtype=torch.float32, device=dev)
        nbytes = wl.B * wl.T * wl.H * 5 * wl.d * wl.elem_bytes + wl.B * wl.H * wl.d * wl.d * 4   # q,k,v,gate in, o out
        ms = _time_launches(stream, flush, nbytes, reps,
                            lambda: ctx.lasad_forward_gated(q, k, v, lam, wl.grid_w, prefix_len=wl.prefix_len, o=o,
                                                            state_out=s_out))
        out["prefill"].append({"workload": f"{wl.name}: B={wl.B} H={wl.H} T={wl.T} d={wl.d} {wl.dtype}",
                               "kernel_us": round(ms * 1e3, 2), "tokens_per_s": round(wl.B * wl.T / (ms * 1e-3), 1),
                               "algorithmic_gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                               "frac_of_hbm_peak": round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                               "l2_policy": flush.policy(nbytes)})
        del q, k, v, lam, o, s_out
    # Algorithm 1's loop body as one call (SiLU, Sigmoid, tied key, operator, RMS norm) against the
    # same computation as separate kernels: torch's element-wise kernels around lasad_forward_gated
    out["fused"] = []
    for wl in wls[1:]:
        gen = torch.Generator().manual_seed(wl.seed + 11)
        qp = torch.randn(wl.B, wl.T, wl.H, wl.d, generator=gen).to(wl.torch_dtype).to(dev)
        gp = (torch.randn(wl.B, wl.T, wl.H, wl.d, generator=gen) + 2.0).to(wl.torch_dtype).to(dev)
        v = workloads.make_qkv(wl)[2].to(dev)
        o = torch.empty_like(v)
        s_out = torch.empty(wl.B, wl.H, wl.d, wl.d, dtype=torch.float32, device=dev)
        unit = wl.B * wl.T * wl.H * wl.d * wl.elem_bytes       # one [B,T,H,d] tensor
        state_b = wl.B * wl.H * wl.d * wl.d * 4
        fused_bytes = 4 * unit + state_b                       # q~, gate~, v in, o out
        unfused_bytes = 2 * unit + 2 * unit + 3 * unit + (4 * unit + state_b) + 2 * unit   # SiLU, Sigmoid, 1 - lambda, operator, norm

        def unfused(norm=True):
            lam = torch.sigmoid(gp)
            oo, _ = ctx.lasad_forward_gated(torch.nn.functional.silu(qp), 1.0 - lam, v, lam, wl.grid_w,
                                            prefix_len=wl.prefix_len, o=o, state_out=s_out)
            return torch.nn.functional.rms_norm(oo, (wl.d,), eps=1e-6) if norm else oo

        ms_f = _time_launches(stream, flush, fused_bytes, reps,
                              lambda: ctx.lasad_forward_fused(qp, None, v, gp, wl.grid_w, prefix_len=wl.prefix_len, o=o,
                                                              state_out=s_out, norm_eps=1e-6))
        ms_u = _time_launches(stream, flush, fused_bytes, reps, unfused)
        ms_u0 = _time_launches(stream, flush, fused_bytes, reps, lambda: unfused(False))
        out["fused"].append({"workload": f"{wl.name}: B={wl.B} H={wl.H} T={wl.T} d={wl.d} {wl.dtype}, key tied to the gate",
                             "fused_us": round(ms_f * 1e3, 2), "unfused_us": round(ms_u * 1e3, 2),
                             "unfused_without_norm_us": round(ms_u0 * 1e3, 2),
                             "fused_bytes": fused_bytes, "unfused_bytes": unfused_bytes,
                             "fused_frac_of_hbm_peak": round(fused_bytes / (ms_f * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                             "unfused": "torch.sigmoid, F.silu, 1 - lambda, lasad_forward_gated, F.rms_norm (torch's norm kernel is slow "
                                        "on rows of 64 channels: the sequence without it is given as well)"})
        del qp, gp, v, o, s_out
    if not decode:
        return out
    dw = workloads.WORKLOADS["config4"]
    T = 16
    q, k, v = [t.to(dev) for t in workloads.make_qkv(dw, T)]
    lam = workloads.make_gate(dw, T).to(dev)
    states = [torch.zeros(dw.B, dw.H, dw.d, dw.d, dtype=torch.float32, device=dev) for _ in range(3)]
    do = torch.empty(dw.B, dw.H, dw.d, dtype=q.dtype, device=dev)
    tok = [(q[:, t], k[:, t], v[:, t], lam[:, t]) for t in range(T)]     # views made outside the timed loop
    def sweep():
        for t in range(T):
            tq, tk, tv, tl = tok[t]
            ctx.lasad_decode_step_gated(tq, tk, tv, tl, states[t % 3], dw.grid_w, dw.prefix_len, dw.prefix_len + t, o=do)
    sweep()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(reps):
        sweep()
    b.record(stream)
    torch.cuda.synchronize()
    us = a.elapsed_time(b) * 1e3 / (reps * T)
    dbytes = dw.B * dw.H * (8 * dw.d * dw.d + 5 * dw.d * dw.elem_bytes)
    out["decode"] = {"workload": f"{dw.name}: B={dw.B} H={dw.H} d={dw.d}, rotating states, per-step launches",
                     "us_per_step": round(us, 3), "algorithmic_gbs": round(dbytes / (us * 1e-6) / 1e9, 1),
                     "frac_of_hbm_peak": round(dbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"], 4)}
    return out


def sustained_prefill(ctx, wl, peaks, dev, seconds: float = 1.5, batch: int = 200):
    """Back-to-back launches of the prefill on `wl` for `seconds`; the last batch is timed with one
    CUDA-event pair and the SM clock is sampled over it.  A copy at the measured HBM bandwidth
    alone draws most of the board's power limit, so a kernel that computes at that rate runs under
    sw_power_cap once the limit's averaging window has filled."""
    import torch
    from paper_2507_01652_b200 import workloads
    q, k, v = [t.to(dev) for t in workloads.make_qkv(wl)]
    g = workloads.make_decay(wl).to(dev)
    o = torch.empty_like(v)
    s_out = torch.empty(wl.B, wl.H, wl.d, wl.d, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    fwd = lambda: ctx.lasad_forward(q, k, v, g, wl.grid_w, prefix_len=wl.prefix_len, o=o, state_out=s_out)
    t0 = time.time()
    while time.time() - t0 < seconds:
        for _ in range(batch):
            fwd()
        torch.cuda.synchronize()
    sampler = ClockSampler(dev.index)
    beg, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with sampler:
        beg.record(stream)
        for _ in range(batch):
            fwd()
        end.record(stream)
        torch.cuda.synchronize()
    ms = beg.elapsed_time(end) / batch
    gbs = prefill_bytes(wl) / (ms * 1e-3) / 1e9
    return {"workload": wl.name, "seconds_before": seconds, "launches_timed": batch, "kernel_us": round(ms * 1e3, 2),
            "tokens_per_s": round(wl.B * wl.T / (ms * 1e-3), 1), "hbm_frac": round(gbs / peaks["hbm_gbs"], 4),
            "clocks": sampler.summary()}


def host_cost_per_call(ctx, dev, calls: int = 1000):
    """Host time of one library call: wall clock of `calls` enqueue-only calls (no synchronisation
    inside the loop) on shapes whose kernels are shorter than the call, through the Python binding
    (its ctypes marshalling is part of the figure)."""
    import torch

    out = {}
    B, T, H, d = 1, 128, 2, 64
    q = torch.zeros(B, T, H, d, dtype=torch.bfloat16, device=dev)
    g = torch.full((H,), 0.95, device=dev)
    o = torch.empty_like(q)
    s = torch.zeros(B, H, d, d, device=dev)
    q1, o1 = q[:, 0], o[:, 0]          # one token's [B,H,d] views, taken outside the timed loop
    for name, fn in (
        ("lasad_forward", lambda: ctx.lasad_forward(q, q, q, g, 16, o=o, state_out=s)),
        ("lasad_decode_step", lambda: ctx.lasad_decode_step(q1, q1, q1, g, s, 16, 0, 5, o=o1)),
    ):
        for _ in range(20):
            fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(calls):
            fn()
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        out[name] = round((t1 - t0) / calls * 1e6, 2)
    out["note"] = f"{calls} enqueue-only calls each, B={B} H={H} T={T} (prefill) / one token (decode), Python binding included"
    return out


def scaling_sweep(ctx, dev, cpu: bool, grids=(16, 24, 32, 64, 96), reps: int = 10):
    """Prefill throughput against sequence length N on the config 5 shape (B=8, H=24, d=64, bf16):
    the GPU kernel (library default), and on the host cores the oracle's recurrent form (linear in N)
    and its quadratic form (the explicit masked-decay sum, N^2).  The oracle runs on a subset of the
    (batch, head) chains -- every chain costs the same -- and its time is scaled to all of them."""
    import torch

    from paper_2507_01652_b200 import workloads

    stream = torch.cuda.current_stream()
    flush = L2Flush(dev)
    base = workloads.WORKLOADS["config5b"]
    points = []
    for gsz in grids:
        wl = dataclasses.replace(base, grid_h=gsz, grid_w=gsz, name=f"config5 shape, {gsz}x{gsz} grid")
        q, k, v = workloads.make_qkv(wl)
        g = workloads.make_decay(wl)
        dq, dk, dv, dg = q.to(dev), k.to(dev), v.to(dev), g.to(dev)
        o = torch.empty_like(dv)
        s_out = torch.empty(wl.B, wl.H, wl.d, wl.d, dtype=torch.float32, device=dev)
        nbytes = prefill_bytes(wl)
        ms = _time_launches(stream, flush, nbytes, reps,
                            lambda: ctx.lasad_forward(dq, dk, dv, dg, wl.grid_w, o=o, state_out=s_out))
        pt = {"N": wl.T, "grid": f"{gsz}x{gsz}", "gpu_kernel_us": round(ms * 1e3, 2),
              "gpu_tokens_per_s": round(wl.B * wl.T / (ms * 1e-3), 1), "l2_policy": flush.policy(nbytes)}
        del dq, dk, dv, o
        if cpu:
            from oracle import lasad_oracle as orc

            # batch 0, as many heads as there are host threads (at most all 24)
            nh = max(1, min(wl.H, orc.threads()))
            sl = (slice(0, 1), slice(None), slice(0, nh))
            q64, k64, v64 = [t[sl].to(torch.float64).numpy() for t in (q, k, v)]
            g64 = g[:nh].to(torch.float64).numpy()
            scale_up = wl.B * wl.H / nh
            for form, fn in (("recurrent", orc.recurrent), ("quadratic", orc.quadratic)):
                best = None
                for _ in range(2 if wl.T <= 1024 else 1):
                    t0 = time.perf_counter()
                    fn(q64, k64, v64, g64, wl.grid_w)
                    dt = time.perf_counter() - t0
                    best = dt if best is None else min(best, dt)
                pt[f"oracle_{form}_tokens_per_s"] = round(wl.B * wl.T / (best * scale_up), 1)
                pt[f"oracle_{form}_sample_s"] = round(best, 3)
            pt["oracle_sample"] = f"batch 0, heads 0..{nh - 1} ({nh} of {wl.B * wl.H} chains, {orc.threads()} threads), time scaled by {scale_up:g}"
        points.append(pt)
    return {"shape": "B=8 H=24 d=64 bf16 (config 5), prefill, library default kernel", "points": points}


def run_decode(args, ctx, peaks, dev, rank, barrier, max_ranks, K, workload=None, hot: bool = True):
    """Decode sweep: persistent fp32 state, one `lasad_decode_step` per grid position (`workload`:
    a configuration's name; default: --decode-workload, the config 4 shape)."""
    import torch

    from paper_2507_01652_b200 import workloads

    stream = torch.cuda.current_stream()
    sampler = ClockSampler(dev.index)
    dw = workloads.WORKLOADS[workload or args.decode_workload]
    if args.decode_batch and workload is None:
        dw = dw.scaled(B=args.decode_batch)
    dw = dataclasses.replace(dw, seed=rank_seed(dw.seed, rank))
    P = dw.prefix_len
    dq, dk_, dv_ = [t.to(dev) for t in workloads.make_qkv(dw)]
    dg = workloads.make_decay(dw).to(dev)
    # rotating state sets: together > 2x L2, so no step finds its state in L2
    state_bytes = dw.B * dw.H * dw.d * dw.d * 4
    n_sets = max(3, -(-2 * L2_BYTES // state_bytes) + 1)
    states = [torch.zeros(dw.B, dw.H, dw.d, dw.d, dtype=torch.float32, device=dev) for _ in range(n_sets)]
    do = torch.empty(dw.B, dw.H, dw.d, dtype=dq.dtype, device=dev)
    positions = list(range(P, dw.T))
    sweeps = max(2, min(10, K // 10))

    def reset_states():
        for s_ in states:
            if P:
                ctx.lasad_forward(dq[:, :P], dk_[:, :P], dv_[:, :P], dg, dw.grid_w, prefix_len=P,
                                  state_out=s_, want_state=True)
            else:
                s_.zero_()

    # each position's [B,H,d] views, made once: slicing three tensors per step would cost the host
    # more than the call itself
    tok = [(dq[:, t], dk_[:, t], dv_[:, t]) for t in positions]

    def sweep(cold: bool):
        for n, t in enumerate(positions):
            tq, tk, tv = tok[n]
            ctx.lasad_decode_step(tq, tk, tv, dg, states[n % n_sets if cold else 0], dw.grid_w, P, t, o=do)

    dec = {}
    for mode, cold in (("cold", True), ("hot", False)) if hot else (("cold", True),):
        reset_states()
        sweep(cold)  # warm-up sweep
        barrier()
        d_beg, d_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with sampler:
            d_beg.record(stream)
            for _ in range(sweeps):
                sweep(cold)
            d_end.record(stream)
            torch.cuda.synchronize()
        barrier()
        us = max_ranks(d_beg.elapsed_time(d_end)) * 1e3 / (sweeps * len(positions))
        dec[mode] = us
    # the same cold sweep replayed as a CUDA graph: kernel time without per-launch host cost
    graph_us = None
    try:
        reset_states()
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            sweep(True)
            torch.cuda.synchronize()
            with torch.cuda.graph(gr, stream=side):
                sweep(True)
        torch.cuda.synchronize()
        gr.replay()
        barrier()
        g_beg, g_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with sampler:
            g_beg.record(stream)
            for _ in range(sweeps):
                gr.replay()
            g_end.record(stream)
            torch.cuda.synchronize()
        barrier()
        graph_us = max_ranks(g_beg.elapsed_time(g_end)) * 1e3 / (sweeps * len(positions))
    except Exception as e:  # pragma: no cover - reported, never hidden
        dec["graph_error"] = repr(e)
    assert ctx.device_status() == 0
    dbytes = decode_bytes(dw)
    best_us = graph_us if graph_us is not None else dec["cold"]
    decode = {
        "workload": f"{dw.name}: B={dw.B} H={dw.H} d={dw.d} grid={dw.grid_h}x{dw.grid_w} prefix={P}, "
                    f"{len(positions)} positions, bf16 q/k/v/o, fp32 state",
        "us_per_step_cold_stream": round(dec["cold"], 3),
        "us_per_step_hot_stream": round(dec["hot"], 3) if "hot" in dec else None,
        "us_per_step_cold_graph": None if graph_us is None else round(graph_us, 3),
        "bytes_per_step": dbytes,
        "states_rotated": n_sets,
        "roofline": {"bound": "hbm", "achieved": round(dbytes / (best_us * 1e-6) / 1e9, 1),
                     "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": round(dbytes / (best_us * 1e-6) / 1e9 / peaks["hbm_gbs"], 4),
                     "traffic": NCU_TRAFFIC_BYTES["decode"] if (dw.name == "config4" and dw.B == 256) else None,
                     "peak_source": peaks["source"],
                     "timed": "cold sweep, CUDA graph" if graph_us is not None else "cold sweep, stream"},
    }
    if "graph_error" in dec:
        decode["graph_error"] = dec["graph_error"]

    decode["clocks"] = sampler.summary()
    return decode


# --------------------------------------------------------------------------------------------
# CPU baseline / reference arm: the oracle, as it stands, on the host cores
# --------------------------------------------------------------------------------------------
def _oracle_sample(wl, units_b: int, reps: int):
    import numpy as np
    import torch

    from oracle import lasad_oracle as orc
    from paper_2507_01652_b200 import workloads

    sub = dataclasses.replace(wl, B=units_b)
    q, k, v = [t.to(torch.float64).numpy() for t in workloads.make_qkv(sub)]
    g = workloads.make_decay(sub).to(torch.float64).numpy()
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        orc.recurrent(q, k, v, g, sub.grid_w, sub.prefix_len)
        times.append(time.perf_counter() - t0)
    return sub, times, orc.threads()


def cpu_baseline(wl, budget_s: float = 12.0):
    """The oracle's recurrent form over whole batches of the workload, repeated for about
    `budget_s` seconds of CPU work; the best repetition is reported."""
    units_b = min(wl.B, 4)
    sub, times, threads = _oracle_sample(wl, units_b, 2)
    reps = max(1, min(60, int(budget_s / max(min(times), 1e-3)) - 2))
    times += _oracle_sample(wl, units_b, reps)[1]
    best = min(times)
    return {"value": round(sub.B * sub.T / best, 1), "unit": "tokens/s", "cores": threads,
            "kind": "oracle",
            "sample": f"oracle recurrent form (fp64, OpenMP over batch x head) on batch 0..{sub.B - 1} of "
                      f"{wl.name} (all {wl.H} heads, T={wl.T}); best of {len(times)} runs, {best:.2f} s each, "
                      f"{sum(times):.1f} s of CPU work in total"}


def run_reference(args):
    """The reference arm of this tier is the CPU oracle, timed on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    from paper_2507_01652_b200 import workloads

    wl = workloads.WORKLOADS[args.prefill_workload]
    K, W = max(1, min(args.steps, 5)), max(1, min(args.warmup, 2))
    sub, times, threads = _oracle_sample(wl, 1, K + W)
    timed = times[W:]
    ms = 1e3 * sum(timed) / len(timed)
    value = sub.B * sub.T / (ms * 1e-3)
    sample = (f"oracle recurrent form (fp64) on batch 0 of {wl.name} (all {wl.H} heads, T={wl.T}) per step; "
              f"{len(timed)} timed steps after {W} warm-up")
    line = {
        "impl": "reference", "metric": "lasad_prefill_tokens_per_s", "value": round(value, 1),
        "unit": "tokens/s", "n_gpus": world, "steps": len(timed), "warmup": W,
        "ms_per_step": round(ms, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{wl.name}: B={wl.B} H={wl.H} T={wl.T} ({wl.grid_h}x{wl.grid_w} grid) "
                               f"d_k=d_v={wl.d}; bounded sample: batch 0 only"},
        "cpu_baseline": {"value": round(value, 1), "unit": "tokens/s", "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(value, 1), "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--prefill-workload", default="config5b")
    ap.add_argument("--decode-workload", default="config4")
    ap.add_argument("--chunk-for-flops", type=int, default=128,
                    help="chunk length used to count executed tensor flops")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-configuration prefill sweep")
    ap.add_argument("--prefill-impl", type=int, default=0, choices=[0, 1, 2, 3, 4, 5],
                    help="prefill kernel: 0 library default, 1 CUDA cores, 2 tcgen05 CTA-per-chain, 3 tcgen05 task-streaming, "
                         "4 as 2 with few long chains cut into segments, 5 tcgen05 balanced (one CTA per SM, two pipelines)")
    ap.add_argument("--only", choices=["all", "prefill", "decode", "gated"], default="all",
                    help="time only one of the kernels (small profiling runs); gated = the gated prefill "
                         "on --prefill-workload")
    ap.add_argument("--prefill-batch", type=int, default=0, help="override the prefill workload's batch")
    ap.add_argument("--sustained-seconds", type=float, default=1.5,
                    help="back-to-back launches before the prefill_sustained block is timed; 0 skips the block")
    ap.add_argument("--decode-batch", type=int, default=0, help="override the decode workload's batch")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
