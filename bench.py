#!/usr/bin/env python
"""Throughput of the signSGD / Signum majority-vote step on B200.

One "step" is one pass of the whole hot path -- per-worker momentum update fused
with 1-bit sign packing, majority vote over the M packed vectors, unpack-and-apply
to x -- over one batch of synthetic gradients.  The default workload is the
Resnet-50-sized vector (d = 25,557,056 with per-tensor padding, M = 7 workers,
Signum beta = 0.9).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With --impl reference the CPU oracle is timed instead, on
a bounded slice of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "parameters_per_second_pack_vote_apply"
UNIT = "params/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel,
# from the ncu capture summarised in profiles/; valid only while the kernel source is unchanged.
NCU_TRAFFIC = {
    "source_sha256": "02dbe7eb10a46ec6d0b079026d61e5054a950444d468d14358424998f0538bc3",
    "workload": "resnet50_d25557056_M7",
    "bytes_per_launch": 1.533647e9 + 792.951296e6,
}


KERNEL_SOURCES = ("signsgd.cu", "device_common.cuh", "host_common.h")


def kernel_source_digest():
    import hashlib
    h = hashlib.sha256()
    try:
        for name in KERNEL_SOURCES:
            with open(os.path.join(ROOT, "paper_1802_04434_b200", "csrc", name), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return h.hexdigest()


def ncu_traffic(workload_name: str):
    if kernel_source_digest() == NCU_TRAFFIC["source_sha256"] and workload_name == NCU_TRAFFIC["workload"]:
        return NCU_TRAFFIC["bytes_per_launch"]
    return None


def fused_bytes_per_param(M: int, momentum: bool) -> float:
    """Algorithmic bytes of the fused step kernel: g (+ m read and written) and one sign bit per worker,
    one voted bit, x read and written.  The separate vote kernel's re-read of the sign words is gone."""
    return (12.125 if momentum else 4.125) * M + 8.125


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def get_workload(name: str):
    from paper_1802_04434_b200 import workloads as wl
    if name == "resnet50":
        return wl.resnet50_signum()
    if name == "small":
        return wl.small_signum()
    if name == "tie":
        return wl.tie_zero_stress()
    if name == "bert":
        return wl.bert_large_signum()
    if name.startswith("sweep:"):
        d, M = name.split(":")[1].split("x")
        return wl.sweep_point(int(d), int(M))
    raise SystemExit("unknown workload %r" % name)


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the GPU is under load."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
               0x10: "sync_boost", 0x100: "display_clock_setting"}

    def __init__(self, torch_device_index: int, period_s: float = 0.02):
        self.period = period_s
        self.samples, self.reason_bits = [], 0
        self.max_mhz, self.ok = None, False
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # no NVML: report that clocks could not be sampled
            self.err = repr(e)

    def _reasons(self):
        nv = self.nv
        for fn in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            if hasattr(nv, fn):
                return int(getattr(nv, fn)(self.h))
        return 0

    def sample_once(self):
        self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
        self.reason_bits |= self._reasons()

    def _run(self):
        while not self._stop.is_set():
            try:
                self.sample_once()
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.ok:
            self._stop.clear()
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self, note=None):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable"]}
        s = sorted(self.samples)
        out = {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
               "reasons": [n for b, n in sorted(self.REASONS.items()) if self.reason_bits & b],
               "samples": len(s)}
        if note:
            out["note"] = note
        return out


# ----------------------------------------------------------------------------- the oracle arm

def oracle_rate(cfg, n_sample: int, steps: int, warmup: int):
    """Time the CPU oracle's whole step on the first n_sample elements of the workload."""
    import numpy as np
    import oracle
    n = min(n_sample, cfg.d)
    shared = cfg.shared("cpu")
    g = cfg.g(0, "cpu", shared)[:, :n].contiguous().numpy().reshape(-1)
    x = cfg.x0("cpu")[:n].contiguous().numpy()
    m = np.zeros(cfg.M * n, dtype=np.float32) if cfg.momentum_buffer else None
    for _ in range(warmup):
        oracle.signsgd_step(x, g, m, cfg.M, n, cfg.beta, cfg.delta)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.signsgd_step(x, g, m, cfg.M, n, cfg.beta, cfg.delta)
    dt = time.perf_counter() - t0
    return n * steps / dt, dt / steps, n


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = get_workload(args.workload)
    # size each step's slice so that the whole run stays near a minute of CPU time
    rate, _, _ = oracle_rate(cfg, 1 << 18, 1, 1)
    budget_s = 60.0
    n = int(rate * budget_s / max(args.steps + args.warmup, 1))
    n = max(1 << 12, min(cfg.d, n)) // 32 * 32
    value, s_per_step, n = oracle_rate(cfg, n, args.steps, args.warmup)
    sample = "first %d of %d elements per step, all M=%d workers, single thread" % (n, cfg.d, cfg.M)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": s_per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": workload_config(cfg, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg, n_gpus):
    return {"workload": cfg.name, "d": cfg.d, "M": cfg.M, "beta": cfg.beta, "delta": cfg.delta,
            "parallelism": "independent shard of d per GPU, no collective" if n_gpus > 1 else "single GPU",
            "l2": "g + m per step exceed L2 (no flush needed)" if not needs_l2_flush(cfg)
            else "L2 flushed between timed steps by writing a 256 MiB buffer; step time = sum of per-step event pairs"}


def needs_l2_flush(cfg) -> bool:
    """True when one step's inputs would stay resident in the 126 MB L2 from one step to the next."""
    return 2 * cfg.M * cfg.ld * 4 <= (256 << 20)


# ----------------------------------------------------------------------------- the CUDA arm

def run_ours(args):
    import torch
    from paper_1802_04434_b200 import binding as B
    from paper_1802_04434_b200 import multi

    rank, local_rank, world = multi.env_ranks()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    multi.init(dev)
    B.lib()  # fail here, loudly, if the CUDA library is missing

    cfg = get_workload(args.workload)
    cfg.seed = multi.shard_seed(rank)   # every rank owns an independent shard of a larger vector
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    momentum = cfg.momentum_buffer
    shared = cfg.shared(dev)
    x = cfg.x0(dev)
    m = cfg.m0(dev) if momentum else None
    g = cfg.g(0, dev, shared)
    del shared
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=dev)
    vote = torch.zeros(W, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    fused = M <= B.FUSED_MAX_WORKERS

    def step_with_events(ev):
        # With few workers one step is one call of the step entry point = one fused kernel launch, and
        # the event pair around it times that kernel.  With more workers the step entry point issues the
        # worker, vote and apply kernels; the same three entry points are then called here one by one so
        # that the event pair can sit around the dominant (worker) kernel inside the timed region.
        ev[0].record(stream)
        if fused:
            B.signsgd_step(x, g, m, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote, stream)
            ev[1].record(stream)
            return
        if momentum:
            B.signum_momentum_pack(g, m, M, d, ld, cfg.beta, bits, ldw, stream)
        else:
            B.sign_pack(g, M, d, ld, bits, ldw, stream)
        ev[1].record(stream)
        B.majority_vote(bits, M, d, ldw, vote, stream)
        B.sign_apply(x, vote, d, cfg.delta, stream)

    def barrier():
        multi.barrier(dev)

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if needs_l2_flush(cfg) else None
    K, Wm = args.steps, args.warmup
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    scratch_ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
    for _ in range(Wm):
        step_with_events(scratch_ev)
    sampler = ClockSampler(local_rank)
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    t_start.record(stream)
    step_ends = []
    for k in range(K):
        step_with_events(events[k])
        if flush is not None:
            e = torch.cuda.Event(enable_timing=True)
            e.record(stream)
            step_ends.append(e)
            flush.zero_()
    t_end.record(stream)
    barrier()
    sampler.stop()
    elapsed_ms = t_start.elapsed_time(t_end)
    if flush is not None:       # leave the flush writes out: each step from its first event to its own end
        elapsed_ms = sum(events[k][0].elapsed_time(step_ends[k]) for k in range(K))
    clock_note = None
    if sampler.ok and len(sampler.samples) < 5:
        # timed region too short for the sampling period: keep sampling under the same load
        clock_note = "timed region shorter than 5 sampling periods; sampled under the same load right after it"
        sampler.start()
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < 0.5:
            for _ in range(20):
                step_with_events(scratch_ev)
            torch.cuda.synchronize()
        sampler.stop()
    worker_ms = sum(a.elapsed_time(b) for a, b in events) / K

    elapsed_ms, worker_ms = multi.max_over_ranks([elapsed_ms, worker_ms], dev)
    value = multi.whole_job_rate(d, K, elapsed_ms, world)
    ms_per_step = elapsed_ms / K

    # end to end through the host-buffer entry point: gradients start in pinned host memory,
    # the voted words come back to the host, every step
    Ke = max(3, min(K, args.e2e_steps))
    g_host = torch.empty(M, ld, dtype=torch.float32).pin_memory()
    g_host.copy_(g)
    vote_host = torch.zeros(W, dtype=torch.int32).pin_memory()
    for _ in range(3):
        B.signsgd_step_host(x, g_host, m, M, d, ld, cfg.beta, cfg.delta, g, bits, ldw, vote, vote_host, stream)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(Ke):
        B.signsgd_step_host(x, g_host, m, M, d, ld, cfg.beta, cfg.delta, g, bits, ldw, vote, vote_host, stream)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    (e2e_ms,) = multi.max_over_ranks([e2e_ms], dev)
    e2e_value = multi.whole_job_rate(d, Ke, e2e_ms, world)

    if rank == 0:
        peak, peak_kind = measured_peak()
        bpp = fused_bytes_per_param(M, momentum) + (0.0 if fused else (M + 1) / 8.0 - 0.125)
        wbytes = (fused_bytes_per_param(M, momentum) if fused else (12.125 if momentum else 4.125) * M) * d
        achieved = wbytes / (worker_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": workload_config(cfg, world),
            "step_hbm_gbs": bpp * d / (ms_per_step * 1e-3) / 1e9,
            "step_frac_of_nominal_8TBs": bpp * d / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "step_bytes_per_param": bpp,
            "roofline": {"kernel": "fused_step_kernel (momentum + sign + pack, vote, apply)" if fused else
                         "worker_pack_kernel (momentum + sign + pack)", "bound": "hbm", "achieved": achieved, "peak": peak,
                         "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                         "ms_per_launch": worker_ms, "bytes_per_launch": wbytes,
                         "traffic": ncu_traffic(cfg.name)},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": M * ld * 4,
                    "d2h_bytes_per_step": W * 4, "steps": Ke, "ms_per_step": e2e_ms / Ke},
            "gpu_launches": K if fused else 3 * K,
            "clocks": sampler.summary(clock_note),
        }
        if not args.no_cpu_baseline and world == 1:
            rate, _, _ = oracle_rate(cfg, 1 << 18, 1, 1)
            n = max(1 << 16, min(cfg.d, int(rate * 4.0))) // 32 * 32      # ~4 s per step, 3 timed steps
            v, _, n = oracle_rate(cfg, n, 3, 1)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": "first %d of %d elements, M=%d, 3 steps, single thread" % (n, d, M)}
        print(json.dumps(line), flush=True)
    multi.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="resnet50",
                    help="resnet50 | small | tie | bert | sweep:<d>x<M>")
    ap.add_argument("--e2e-steps", type=int, default=40)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
