#!/usr/bin/env python
"""Throughput of the signSGD / Signum majority-vote step on B200.

One "step" is one pass of the whole hot path -- per-worker momentum update fused
with 1-bit sign packing, majority vote over the M packed vectors, unpack-and-apply
to x -- over one batch of synthetic gradients, issued as ONE call of the step entry
point.  The default workload is the largest single-GPU configuration: the
BERT-large-sized vector (d = 335,141,888, M = 16 workers, Signum beta = 0.9, 45 GB
on the device), which takes the worker + vote + apply kernels; `--workload
resnet50` (d = 25,557,056, M = 7) takes the single fused kernel.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload bert|resnet50|small|tie|sweep:<d>x<M>] [--seed S]
                    [--mode shards|workers]

Prints ONE JSON line.  After the timed region a second pass over the same buffers
takes per-kernel CUDA-event times (`kernels`), the same step is timed end to end
from host buffers (`e2e`), and the CPU oracle is timed on a bounded sample on one
thread and on all host cores (`cpu_baseline`, `cpu_baseline_all_cores`).  With
--impl reference only the CPU oracle is timed.  `--mode workers` runs Algorithm 3
with one worker per GPU (an all-gather of the sign words between the ranks).
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

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per parameter of one launch, from the ncu
# captures summarised in profiles/.  At the captured size the figure is the capture's own; at another d
# with the same M it is scaled (the path is elementwise, so traffic grows in proportion to d as long as
# the operands exceed L2).  Valid only while the kernel sources are unchanged.
NCU_TRAFFIC = {
    "source_sha256": "7257bc4e8464b4bc301ae59fd613c1dba7194e2a8919a9ec618576fd181ce183",
    "per_param": {
        # profiles/dram_bytes_worker_vote_apply_bertlarge_M16_full_size.md: a one-pass capture of the full-size
        # default workload (d = 335,141,888)
        "worker_pack_kernel:M16": {"bytes_per_param": (42899410688 + 22068347136) / 335141888, "d": 335141888},
        "vote_kernel:M16": {"bytes_per_param": (670312448 + 36816640) / 335141888, "d": 335141888},
        "apply_kernel:M16": {"bytes_per_param": (1382548480 + 1277543680) / 335141888, "d": 335141888},
        # profiles/fused_step_kernel_resnet50_M7_ncu_full.md (captured at full size)
        "fused_step_kernel:M7": {"bytes_per_param": (1.533634e9 + 793.212160e6) / 25557056, "d": 25557056},
    },
}

KERNEL_SOURCES = ("signsgd.cu", "device_common.cuh", "host_common.h", "vote_launch.h", "step_rows.cuh")


def kernel_source_digest():
    """sha256 of the kernel sources with comments and white space removed: an edit of a comment does not
    invalidate the ncu figures, an edit of the code does."""
    import hashlib
    import re
    h = hashlib.sha256()
    try:
        for name in KERNEL_SOURCES:
            with open(os.path.join(ROOT, "paper_1802_04434_b200", "csrc", name), "r") as fh:
                text = fh.read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            text = re.sub(r"//[^\n]*", "", text)
            h.update("".join(text.split()).encode())
    except OSError:
        return None
    return h.hexdigest()


def ncu_traffic(kernel: str, M: int, d: int):
    """(bytes per launch, note) scaled from the capture, or (None, why)."""
    if kernel_source_digest() != NCU_TRAFFIC["source_sha256"]:
        return None, "kernel sources changed since the ncu capture"
    rec = NCU_TRAFFIC["per_param"].get("%s:M%d" % (kernel, M))
    if rec is None:
        return None, "no ncu capture of this kernel at this M"
    if rec["d"] == d:
        return rec["bytes_per_param"] * d, "ncu capture at this size"
    return rec["bytes_per_param"] * d, "scaled by d from the ncu capture at d = %d" % rec["d"]


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def get_workload(name: str, seed: int = 0):
    from paper_1802_04434_b200 import workloads as wl
    if name == "resnet50":
        cfg = wl.resnet50_signum()
    elif name == "small":
        cfg = wl.small_signum()
    elif name == "tie":
        cfg = wl.tie_zero_stress()
    elif name == "bert":
        cfg = wl.bert_large_signum()
    elif name.startswith("sweep:"):
        d, M = name.split(":")[1].split("x")
        cfg = wl.sweep_point(int(d), int(M))
    else:
        raise SystemExit("unknown workload %r" % name)
    cfg.seed = seed
    return cfg


# algorithmic bytes per parameter of each kernel (fp32 state in place, 1 bit per sign)
def worker_bpp(M: int, momentum: bool) -> float:
    return (12.125 if momentum else 4.125) * M


def vote_bpp(M: int) -> float:
    return (M + 1) / 8.0


APPLY_BPP = 8.125


def fused_bpp(M: int, momentum: bool) -> float:
    """The fused step kernel never reads the sign words back: worker bytes + apply bytes."""
    return worker_bpp(M, momentum) + APPLY_BPP


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) while the GPU is under load."""
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

def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_inputs(cfg, n: int):
    """Host arrays (x [n], g [M, n], m [M, n] or None) of the first n parameters of the workload.

    Only the sample is drawn, never the whole vector.  The random draws run on the GPU when there is
    one (same recipe, much faster for the large samples of the all-cores leg), else on the CPU."""
    import numpy as np
    import torch
    sub = cfg.prefix(n // 32 * 32 if n >= 32 else n)
    n = sub.d
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    g = sub.g(0, dev, sub.shared(dev))[:, :n].contiguous().cpu().numpy()
    x = sub.x0(dev)[:n].contiguous().cpu().numpy()
    m = np.zeros((cfg.M, n), dtype=np.float32) if cfg.momentum_buffer else None
    if dev == "cuda":
        torch.cuda.empty_cache()
    return x, g, m


def oracle_rate(cfg, n_sample: int, steps: int, warmup: int, threads: int = 1):
    """Time the CPU oracle's whole step, as it stands, on the first n_sample parameters.

    threads == 1: one call per step.  threads > 1: the sample is cut into `threads` contiguous slices
    with 32-aligned starts and the same oracle function runs on every slice at once from Python threads
    (ctypes releases the interpreter lock during the call; the oracle itself is untouched).
    Returns (params/s, seconds per step, parameters per step)."""
    import numpy as np
    import oracle
    x, g, m = oracle_inputs(cfg, min(n_sample, cfg.d))
    n = x.size
    M = cfg.M
    if threads <= 1:
        gf = g.reshape(-1)
        mf = None if m is None else m.reshape(-1)

        def one_step():
            oracle.signsgd_step(x, gf, mf, M, n, cfg.beta, cfg.delta)
    else:
        from concurrent.futures import ThreadPoolExecutor
        per = max(32, (n // threads) // 32 * 32)
        cuts = [min(n, t * per) for t in range(threads)] + [n]
        parts = []
        for a, b in zip(cuts[:-1], cuts[1:]):
            if b > a:
                parts.append((np.ascontiguousarray(x[a:b]), np.ascontiguousarray(g[:, a:b]).reshape(-1),
                              None if m is None else np.ascontiguousarray(m[:, a:b]).reshape(-1), b - a))
        del x, g, m
        pool = ThreadPoolExecutor(max_workers=len(parts))

        def run_part(p):
            oracle.signsgd_step(p[0], p[1], p[2], M, p[3], cfg.beta, cfg.delta)

        def one_step():
            list(pool.map(run_part, parts))
        threads = len(parts)
    for _ in range(warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(steps):
        one_step()
    dt = time.perf_counter() - t0
    return n * steps / dt, dt / steps, n, max(threads, 1)


ORACLE_SAMPLE_MAX_FLOATS = 1 << 28      # M * n of the sample: 1 GiB of gradients (and as much momentum) at most


def oracle_sample_size(cfg, seconds_per_step: float, threads: int = 1, probe=None) -> int:
    """Parameters per step that keep one oracle step near `seconds_per_step` (3 s at most) and the
    sample's host buffers bounded."""
    rate = probe if probe is not None else oracle_rate(cfg, 1 << 17, 1, 1)[0]
    n = int(rate * min(seconds_per_step, 3.0)) * max(threads, 1)
    n = min(n, cfg.d, ORACLE_SAMPLE_MAX_FLOATS // cfg.M)
    return max(1 << 12, n) // 32 * 32


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = get_workload(args.workload, args.seed)
    cores = host_cores()
    threads = cores if args.ref_threads <= 0 else min(args.ref_threads, cores)
    # size each step's slice so that the whole run stays near a minute of wall time
    budget_s = 60.0
    per_step = budget_s / max(args.steps + args.warmup, 1)
    n = args.ref_sample if args.ref_sample > 0 else oracle_sample_size(cfg, per_step, threads)
    value, s_per_step, n, used = oracle_rate(cfg, n, args.steps, args.warmup, threads)
    sample = ("first %d of %d parameters per step, all M=%d workers, %d thread(s) on disjoint 32-aligned "
              "slices, unmodified oracle" % (n, cfg.d, cfg.M, used))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": s_per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": workload_config(cfg, args.gpus, args.mode),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "host_cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg, n_gpus, mode="shards"):
    if mode == "workers":
        par = ("Algorithm 3 with one worker per GPU: M = %d ranks, each packs its own sign row, every row reaches "
               "every rank, local vote and apply" % n_gpus)
    else:
        par = "independent shard of d per GPU, no collective" if n_gpus > 1 else "single GPU"
    return {"workload": cfg.name, "d": cfg.d, "M": cfg.M if mode != "workers" else n_gpus, "beta": cfg.beta,
            "delta": cfg.delta, "seed": cfg.seed, "mode": mode, "parallelism": par,
            "l2": "g + m per step exceed L2 (no flush needed)" if not needs_l2_flush(cfg)
            else L2Flush.NOTE}


class L2Flush:
    """Empties the 126 MB L2 of a workload's data between timed steps: writes a 256 MiB buffer, then reads
    another one, so that the cache is left full of CLEAN foreign lines.  After the write alone it would be
    full of dirty lines whose write-back the next step would pay for (measured: a 46.7 MB step then takes
    15 us instead of 10)."""

    NOTE = ("L2 flushed between timed steps by writing a 256 MiB buffer and then reading another (the cache is left "
            "with clean lines); step time = sum of per-step event pairs")

    def __init__(self, torch, dev):
        self.torch = torch
        self.w = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        self.r = torch.zeros(64 << 20, dtype=torch.float32, device=dev)
        self.sink = torch.zeros((), dtype=torch.float32, device=dev)

    def __call__(self):
        self.w.zero_()
        self.torch.sum(self.r, dim=0, out=self.sink)


def needs_l2_flush(cfg) -> bool:
    """True when one step's inputs would stay resident in the 126 MB L2 from one step to the next."""
    return 2 * cfg.M * cfg.ld * 4 <= (256 << 20)


# ----------------------------------------------------------------------------- the CUDA arm

class Buffers:
    """Device state of one workload: x, g, m, the word workspaces."""

    def __init__(self, cfg, dev):
        import torch
        self.cfg = cfg
        shared = cfg.shared(dev)
        self.x = cfg.x0(dev)
        self.m = cfg.m0(dev) if cfg.momentum_buffer else None
        self.g = cfg.g(0, dev, shared)
        del shared
        self.bits = torch.zeros(cfg.M, cfg.ldw, dtype=torch.int32, device=dev)
        self.vote = torch.zeros(cfg.words, dtype=torch.int32, device=dev)


def make_step(B, b, stream):
    cfg = b.cfg

    def step():
        B.signsgd_step(b.x, b.g, b.m, cfg.M, cfg.d, cfg.ld, cfg.beta, cfg.delta, b.bits, cfg.ldw, b.vote, stream)
    return step


def timed_block(step, K, stream, flush, torch):
    """K steps between two events; with a flush buffer, each step between its own pair and the flush outside."""
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if flush is None:
        t0.record(stream)
        for _ in range(K):
            step()
        t1.record(stream)
        return lambda: t0.elapsed_time(t1)
    pairs = []
    for _ in range(K):
        a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        step()
        e.record(stream)
        flush()
        pairs.append((a, e))
    return lambda: sum(a.elapsed_time(e) for a, e in pairs)


def per_kernel_pass(B, b, K, stream, flush, torch):
    """Second pass over the same buffers: CUDA-event pairs around every kernel of the step.

    Where the step is one fused kernel it is timed as such; otherwise the three entry points the step
    entry point issues are called one by one so that events can sit between the kernels."""
    cfg = b.cfg
    M, d, ld, ldw = cfg.M, cfg.d, cfg.ld, cfg.ldw
    momentum = cfg.momentum_buffer
    fused = B.step_is_fused(M, d, momentum)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = []
    for _ in range(K):
        e = [ev()]
        e[0].record(stream)
        if fused:
            B.signsgd_step(b.x, b.g, b.m, M, d, ld, cfg.beta, cfg.delta, b.bits, ldw, b.vote, stream)
            e.append(ev()); e[-1].record(stream)
        else:
            if momentum:
                B.signum_momentum_pack(b.g, b.m, M, d, ld, cfg.beta, b.bits, ldw, stream)
            else:
                B.sign_pack(b.g, M, d, ld, b.bits, ldw, stream)
            e.append(ev()); e[-1].record(stream)
            B.majority_vote(b.bits, M, d, ldw, b.vote, stream)
            e.append(ev()); e[-1].record(stream)
            B.sign_apply(b.x, b.vote, d, cfg.delta, stream)
            e.append(ev()); e[-1].record(stream)
        if flush is not None:
            flush()
        marks.append(e)
    torch.cuda.synchronize()
    n = len(marks[0]) - 1
    ms = [sum(e[i].elapsed_time(e[i + 1]) for e in marks) / K for i in range(n)]
    if fused:
        names = [(B.step_kernel_name(M, d, momentum), "ssgd_signsgd_step", fused_bpp(M, momentum))]
    else:
        names = [("worker_pack_kernel", "ssgd_signum_momentum_pack" if momentum else "ssgd_sign_pack",
                  worker_bpp(M, momentum)),
                 ("vote_kernel", "ssgd_majority_vote", vote_bpp(M)),
                 ("apply_kernel", "ssgd_sign_apply", APPLY_BPP)]
    return [(k, ep, bpp, t) for (k, ep, bpp), t in zip(names, ms)]


def kernel_entry(kernel, entry_point, bpp, ms, cfg, peak, launches):
    gbs = bpp * cfg.d / (ms * 1e-3) / 1e9
    traffic, note = ncu_traffic(kernel, cfg.M, cfg.d)
    return {"kernel": kernel, "entry_point": entry_point, "workload": cfg.name, "M": cfg.M,
            "bytes_per_param": bpp, "units_per_launch": cfg.d, "bytes_per_launch": bpp * cfg.d,
            "launches_timed": launches, "ms_per_launch": ms, "achieved_gbs": gbs, "frac": gbs / peak,
            "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "traffic": traffic, "traffic_note": note}


def host_buffer(torch, shape, dtype):
    """Page-locked host tensor if the box grants it, else pageable; returns (tensor, kind)."""
    try:
        return torch.empty(shape, dtype=dtype, pin_memory=True), "pinned"
    except Exception:
        return torch.empty(shape, dtype=dtype), "pageable"


class _SkipE2E(Exception):
    """--e2e-steps 0."""


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
    if args.mode == "workers":
        return run_workers(args, torch, B, multi, dev, rank, local_rank, world)

    cfg = get_workload(args.workload, args.seed + multi.shard_seed(rank))  # an independent shard per rank
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    momentum = cfg.momentum_buffer
    free, _ = torch.cuda.mem_get_info()
    need = (2 if momentum else 1) * M * ld * 4 + 4 * d * 4 + (2 << 30)
    if free < need:
        raise SystemExit("workload %s needs %.1f GB of device memory, %.1f GB are free" % (cfg.name, need / 1e9, free / 1e9))
    b = Buffers(cfg, dev)
    stream = torch.cuda.current_stream()
    step = make_step(B, b, stream)
    fused = B.step_is_fused(M, d, momentum)
    flush = L2Flush(torch, dev) if needs_l2_flush(cfg) else None
    K, Wm = args.steps, args.warmup

    for _ in range(Wm):
        step()
    sampler = ClockSampler(local_rank)
    multi.barrier(dev)
    sampler.start()
    read_ms = timed_block(step, K, stream, flush, torch)
    multi.barrier(dev)
    elapsed_ms = read_ms()
    # The clock samples must be of timed work: when the K steps end before five sampling periods have
    # passed, the same K-step block is repeated (each block timed the same way) until they have.
    extra = []
    while sampler.ok and len(sampler.samples) < 5 and len(extra) < 2000:
        r = timed_block(step, K, stream, flush, torch)
        torch.cuda.synchronize(dev)
        extra.append(r())
    sampler.stop()
    clock_note = None
    if extra:
        clock_note = ("the %d-step block was repeated %d more times inside the sampling window (median block "
                      "%.4f ms); value is the first block's" % (K, len(extra), sorted(extra)[len(extra) // 2]))

    kernels = per_kernel_pass(B, b, K, stream, flush, torch)
    (elapsed_ms, *kms) = multi.max_over_ranks([elapsed_ms] + [t for *_, t in kernels], dev)
    kernels = [(k, ep, bpp, t) for (k, ep, bpp, _), t in zip(kernels, kms)]
    value = multi.whole_job_rate(d, K, elapsed_ms, world)
    ms_per_step = elapsed_ms / K

    # end to end through the host-buffer entry point: every step copies that step's gradients from host
    # memory to the device, runs the step and copies the voted words back to the host
    Ke = max(1, min(K, args.e2e_steps))
    e2e = None
    try:
        if args.e2e_steps <= 0:                      # profiling runs that want the step's kernels only
            raise _SkipE2E
        g_host, host_kind = host_buffer(torch, (M, ld), torch.float32)
        g_host.copy_(b.g)
        vote_host, _ = host_buffer(torch, (W,), torch.int32)
        host_step = lambda: B.signsgd_step_host(b.x, g_host, b.m, M, d, ld, cfg.beta, cfg.delta, b.g, b.bits, ldw,
                                                b.vote, vote_host, stream)
        for _ in range(max(1, min(3, args.e2e_warmup))):
            host_step()
        multi.barrier(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(Ke):
            host_step()
        e1.record(stream)
        multi.barrier(dev)
        (e2e_ms,) = multi.max_over_ranks([e0.elapsed_time(e1)], dev)
        e2e = {"value": multi.whole_job_rate(d, Ke, e2e_ms, world), "unit": UNIT, "h2d_bytes_per_step": M * ld * 4,
               "d2h_bytes_per_step": W * 4, "steps": Ke, "ms_per_step": e2e_ms / Ke, "host_memory": host_kind,
               "entry_point": "ssgd_signsgd_step_host",
               "h2d_gbs": M * ld * 4 / (e2e_ms / Ke * 1e-3) / 1e9}
        del g_host, vote_host
    except _SkipE2E:
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": M * ld * 4, "d2h_bytes_per_step": W * 4,
               "skipped": "--e2e-steps 0"}
        multi.barrier(dev)
    except (RuntimeError, MemoryError) as exc:   # the host could not hold one step's gradients
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": M * ld * 4, "d2h_bytes_per_step": W * 4,
               "error": "host buffer of %.1f GB not granted: %s" % (M * ld * 4 / 1e9, str(exc)[:120])}
        multi.barrier(dev)

    if rank != 0:
        multi.finish()
        return
    peak, peak_kind = measured_peak()
    step_bpp = fused_bpp(M, momentum) if fused else worker_bpp(M, momentum) + vote_bpp(M) + APPLY_BPP
    entries = [kernel_entry(k, ep, bpp, t, cfg, peak, K) for k, ep, bpp, t in kernels]
    dom = max(entries, key=lambda e: e["ms_per_launch"])
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": workload_config(cfg, world),
        "entry_point": "ssgd_signsgd_step",
        "step_bytes_per_param": step_bpp,
        "step_hbm_gbs": step_bpp * d / (ms_per_step * 1e-3) / 1e9,
        "step_frac_of_nominal_8TBs": step_bpp * d / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "roofline": {"kernel": dom["kernel"], "bound": "hbm", "achieved": dom["achieved_gbs"], "peak": peak,
                     "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": dom["frac"],
                     "frac_of_nominal_8TBs": dom["frac_of_nominal_8TBs"], "ms_per_launch": dom["ms_per_launch"],
                     "bytes_per_launch": dom["bytes_per_launch"], "traffic": dom["traffic"],
                     "traffic_note": dom["traffic_note"],
                     "timed_in": "second pass over the same buffers right after the timed region, %d launches, "
                                 "CUDA events around each kernel" % K},
        "kernels": entries,
        "kernels_sum_ms": sum(e["ms_per_launch"] for e in entries),
        "e2e": e2e,
        "gpu_launches": K * len(entries),
        "clocks": sampler.summary(clock_note),
    }
    if not fused and d % 512 != 0:
        line["gpu_launches_note"] = "plus one-warp tail launches per step (d is not a multiple of the 512-element span)"
    if world == 1 and not args.no_extra_kernels and not fused:
        # the fused kernel (the path for M <= 8) as one more entry, on the Resnet-50-sized workload
        del b, step
        torch.cuda.empty_cache()
        cfg2 = get_workload("resnet50", args.seed)
        b2 = Buffers(cfg2, dev)
        step2 = make_step(B, b2, stream)
        for _ in range(max(3, Wm)):
            step2()
        k2 = per_kernel_pass(B, b2, max(K, 20), stream, None, torch)
        line["kernels"] += [kernel_entry(k, ep, bpp, t, cfg2, peak, max(K, 20)) for k, ep, bpp, t in k2]
        del b2, step2
        torch.cuda.empty_cache()
    if not args.no_cpu_baseline and world == 1:
        probe = oracle_rate(cfg, 1 << 17, 1, 1)[0]
        v, _, n, _ = oracle_rate(cfg, oracle_sample_size(cfg, 3.0, 1, probe), 3, 1)
        cores = host_cores()
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "host_cores": cores, "kind": "oracle",
                                "sample": "first %d of %d parameters, M=%d, 3 steps, one thread" % (n, d, M)}
        va, _, na, used = oracle_rate(cfg, oracle_sample_size(cfg, 2.0, cores, probe), 3, 1, cores)
        line["cpu_baseline_all_cores"] = {
            "value": va, "unit": UNIT, "cores": used, "host_cores": cores, "kind": "oracle",
            "sample": "first %d of %d parameters, M=%d, 3 steps, %d threads on disjoint 32-aligned slices, "
                      "unmodified oracle" % (na, d, M, used)}
    print(json.dumps(line), flush=True)
    multi.finish()


def run_workers(args, torch, B, multi, dev, rank, local_rank, world):
    """Algorithm 3 with one worker per GPU: rank r is worker r, M = world size."""
    cfg = get_workload(args.workload, args.seed)
    d, ld, ldw, W = cfg.d, cfg.ld, cfg.ldw, cfg.words
    momentum = cfg.momentum_buffer
    one = cfg.prefix(d)
    one.M = 1
    one.seed = args.seed * 1000003 + rank            # every worker draws its own gradient noise
    shared = cfg.shared(dev)                         # ... around the same mean
    x = cfg.x0(dev)                                  # replicas of x start (and stay) identical
    g = one.g(0, dev, shared)
    m = one.m0(dev) if momentum else None
    del shared
    ws = multi.WorkerStep(d, dev, exchange=args.exchange)
    stream = torch.cuda.current_stream()
    K, Wm = args.steps, args.warmup
    small = 2 * ld * 4 <= (256 << 20)       # one rank's g + m would stay in L2 from step to step
    flush = L2Flush(torch, dev) if small else None
    step = lambda ev=None: ws.step(x, g, m, cfg.beta, cfg.delta, events=ev)
    for _ in range(Wm):
        step()

    def block():
        """K steps, each with its four events; returns a reader of (step, pack, exchange, vote + apply) ms sums."""
        marks = []
        for _ in range(K):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            step(ev)
            if flush is not None:
                flush()
            marks.append(ev)
        return lambda: [sum(e[i].elapsed_time(e[j]) for e in marks) for i, j in ((0, 3), (0, 1), (1, 2), (2, 3))]

    sampler = ClockSampler(local_rank)
    multi.barrier(dev)
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    read = block()
    t1.record(stream)
    multi.barrier(dev)
    step_sum, pack_sum, xchg_sum, rest_sum = read()
    # without a flush the K steps are timed as one region; with it, as the sum of the per-step event pairs
    elapsed_ms = step_sum if flush is not None else t0.elapsed_time(t1)
    pack_ms, xchg_ms, rest_ms = pack_sum / K, xchg_sum / K, rest_sum / K
    elapsed_ms, pack_ms, xchg_ms, rest_ms = multi.max_over_ranks([elapsed_ms, pack_ms, xchg_ms, rest_ms], dev)
    # Clock samples must be of timed work: a short region is repeated under the sampler.  Every block holds
    # collectives, so all ranks must run the same number of them: it is derived from the reduced time.
    extra = min(2000, max(0, int(150.0 / max(elapsed_ms, 1e-3))))
    for _ in range(extra):
        block()
    multi.barrier(dev)
    sampler.stop()
    same = multi.all_ranks_equal(ws.vote)
    if rank == 0:
        peak, peak_kind = measured_peak()
        Mw = world
        pack_bytes = worker_bpp(1, momentum) * d
        line = {
            "metric": METRIC, "value": d * K / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": Wm, "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(cfg, world, "workers"),
                           l2=L2Flush.NOTE if small else "g + m per step exceed L2 (no flush needed)"),
            "wire_bits_per_step_table1": 2 * Mw * d,
            "wire_bytes_sent_per_rank_per_step": ws.ldw * 4 * (world - 1),
            "exchange": {"transport": "all_gather_into_tensor of ceil(d/32)-word rows (NCCL)" if args.exchange == "allgather"
                         else "peer stores from the worker kernel (symmetric memory) + one barrier", "ms": xchg_ms,
                         "share_of_step": xchg_ms / (elapsed_ms / K)},
            "kernels": [
                {"kernel": "worker_pack_kernel" if args.exchange == "allgather" else "pack_scatter_kernel",
                 "ms_per_launch": pack_ms, "bytes_per_launch": pack_bytes,
                 "achieved_gbs": pack_bytes / (pack_ms * 1e-3) / 1e9,
                 "frac": pack_bytes / (pack_ms * 1e-3) / 1e9 / peak},
                {"kernel": "vote_kernel + apply_kernel", "ms_per_launch": rest_ms,
                 "bytes_per_launch": (vote_bpp(Mw) + APPLY_BPP) * d,
                 "achieved_gbs": (vote_bpp(Mw) + APPLY_BPP) * d / (rest_ms * 1e-3) / 1e9,
                 "frac": (vote_bpp(Mw) + APPLY_BPP) * d / (rest_ms * 1e-3) / 1e9 / peak}],
            "roofline": {"kernel": "worker_pack_kernel" if args.exchange == "allgather" else "pack_scatter_kernel",
                         "bound": "hbm", "achieved": pack_bytes / (pack_ms * 1e-3) / 1e9, "peak": peak, "peak_kind": "of " + peak_kind,
                         "unit": "GB/s", "frac": pack_bytes / (pack_ms * 1e-3) / 1e9 / peak, "traffic": None},
            "votes_identical_on_all_ranks": bool(same),
            "gpu_launches": 3 * K,
            "clocks": sampler.summary("the %d-step block was repeated %d more times inside the sampling window"
                                      % (K, extra) if extra else None),
        }
        print(json.dumps(line), flush=True)
    multi.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="bert",
                    help="bert (default, the largest single-GPU configuration) | resnet50 | small | tie | sweep:<d>x<M>")
    ap.add_argument("--mode", choices=["shards", "workers"], default="shards",
                    help="shards: every GPU simulates all M workers on its own shard of parameters (no collective); "
                         "workers: one worker per GPU, sign rows all-gathered (Algorithm 3 as a distributed step)")
    ap.add_argument("--exchange", choices=["allgather", "p2p"], default="allgather",
                    help="--mode workers: how the sign rows travel (a collective, or peer stores from the worker kernel)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=3, help="timed end-to-end steps (0: skip the end-to-end leg)")
    ap.add_argument("--e2e-warmup", type=int, default=3)
    ap.add_argument("--ref-threads", type=int, default=0, help="threads of the oracle arm (0 = all host cores)")
    ap.add_argument("--ref-sample", type=int, default=0,
                    help="parameters per step of the oracle arm (0 = sized from a probe of its speed)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-kernels", action="store_true",
                    help="skip the extra fused-kernel entry on the Resnet-50-sized workload")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
