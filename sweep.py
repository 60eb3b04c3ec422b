"""Per-kernel bandwidth sweep: d = 2^10 .. 2^28, M in {1, 3, 7, 15, 31}, Signum beta = 0.9.

    python sweep.py [--min-log2 10] [--max-log2 28] [--workers 1,3,7,15,31]
                    [--reps 20] [--out sweep.tsv]

For every point and every kernel of the step (worker momentum + pack, majority vote, apply) and for
the whole step (and, beside the vote kernel, for its shared-memory-staged alternative and for a plain
device copy of the vote's byte volume as a yardstick), prints the time per launch, the algorithmic GB/s and its fraction of the measured
copy peak.  Launches are replayed from a CUDA graph between two CUDA events.  When
one launch touches less than twice the L2 size, the launches rotate over several buffer sets so that
the combined footprint exceeds it (column `cold` = 1); for the smallest sizes that would need more
sets than are allowed and the figures are launch-latency numbers, not bandwidth (cold = 0).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_1802_04434_b200 import binding as B

L2_BYTES = 126 << 20
MAX_SETS = 48


def peak_gbs() -> float:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"])
    except Exception:
        return 6650.0


PLAIN_LAUNCHES = False     # --plain: no CUDA graph, every launch issued from the host (for use under a profiler)


def time_launches(fn, n_sets: int, reps: int) -> float:
    """Average milliseconds per launch of fn(set_index).

    The launches are captured once into a CUDA graph (at least 32 per replay, cycling over the
    buffer sets) and the graph is replayed `reps` times between two events, so that the host's
    per-call cost does not limit short kernels."""
    for s in range(n_sets):
        fn(s)
    torch.cuda.synchronize()
    inner = max(1, -(-32 // n_sets))
    if PLAIN_LAUNCHES:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            for s in range(n_sets):
                fn(s)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * n_sets)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(inner):
            for s in range(n_sets):
                fn(s)
    graph.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        graph.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / (reps * inner * n_sets)


def run_point(d: int, M: int, reps: int, dev) -> list:
    ld = (d + 3) // 4 * 4
    W = (d + 31) // 32
    ldw = (W + 3) // 4 * 4
    beta, delta = 0.9, 1e-4
    bytes_worker = 12.125 * M * d
    bytes_vote = (M + 1) / 8.0 * d
    bytes_apply = 8.125 * d
    n_sets = int(min(MAX_SETS, max(1, -(-2 * L2_BYTES // int(bytes_vote + 1)))))
    n_sets_big = int(min(MAX_SETS, max(1, -(-2 * L2_BYTES // int(bytes_worker + 1)))))
    g = [torch.randn(M, ld, device=dev) for _ in range(n_sets_big)]
    m = [torch.zeros(M, ld, device=dev) for _ in range(n_sets_big)]
    n_x = int(min(MAX_SETS, max(1, -(-2 * L2_BYTES // int(bytes_apply + 1)))))
    x = [torch.randn(d, device=dev) for _ in range(n_x)]
    bits = [torch.zeros(M, ldw, dtype=torch.int32, device=dev) for _ in range(n_sets)]
    vote = [torch.zeros(W, dtype=torch.int32, device=dev) for _ in range(max(n_sets, n_x))]
    for s in range(n_sets):                                  # realistic bit rows for the vote
        B.sign_pack(g[s % n_sets_big], M, d, ld, bits[s], ldw)
    rows = []

    def rec(name, ms, nbytes, cold):
        gbs = nbytes / (ms * 1e-3) / 1e9
        rows.append((d, M, name, ms * 1e3, gbs, gbs / peak_gbs(), int(cold)))

    ms = time_launches(lambda s: B.signum_momentum_pack(g[s % n_sets_big], m[s % n_sets_big], M, d, ld, beta,
                                                        bits[s % n_sets], ldw), n_sets_big, reps)
    rec("momentum_pack", ms, bytes_worker, n_sets_big * bytes_worker >= 2 * L2_BYTES)
    ms = time_launches(lambda s: B.majority_vote(bits[s], M, d, ldw, vote[s]), n_sets, reps)
    rec("majority_vote", ms, bytes_vote, n_sets * bytes_vote >= 2 * L2_BYTES)
    # the other vote kernel design: rows staged through shared memory by bulk copies
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ms = time_launches(lambda s: B.majority_vote_staged(bits[s], M, d, ldw, vote[s], status), n_sets, reps)
    rec("majority_vote_staged", ms, bytes_vote, n_sets * bytes_vote >= 2 * L2_BYTES)
    if int(status.item()) != 0:
        raise SystemExit("a bounded wait of the staged vote kernel ran out")
    # yardstick for the short vote kernel: a plain device copy that moves the same number of bytes.
    # Sources and destinations are separate buffers and both rotate, so no launch reads what an
    # earlier one left in L2.
    half = max(1, int(bytes_vote / 2) // 4)
    if n_sets > 1:
        src = [torch.randint(0, 1 << 30, (half,), dtype=torch.int32, device=dev) for _ in range(2 * n_sets)]
        dst = [torch.empty(half, dtype=torch.int32, device=dev) for _ in range(2 * n_sets)]
        ms = time_launches(lambda s: dst[s].copy_(src[s]), 2 * n_sets, reps)
        rec("copy_of_vote_bytes", ms, 2.0 * half * 4, 2 * n_sets * half * 4 >= 2 * L2_BYTES)
        del src, dst
    ms = time_launches(lambda s: B.sign_apply(x[s], vote[s], d, delta), n_x, reps)
    rec("sign_apply", ms, bytes_apply, n_x * bytes_apply >= 2 * L2_BYTES)
    ms = time_launches(lambda s: B.signsgd_step(x[s % n_x], g[s % n_sets_big], m[s % n_sets_big], M, d, ld, beta,
                                                delta, bits[s % n_sets], ldw, vote[s % n_sets]),
                       n_sets_big, reps)
    rec("signsgd_step", ms, bytes_worker + bytes_apply, n_sets_big * bytes_worker >= 2 * L2_BYTES)
    return rows


def run_variants(d: int, M: int, reps: int, dev) -> list:
    """The calls beside the main path (warm-up, count planes, abstention, statistics) at one size."""
    ld = (d + 3) // 4 * 4
    W = (d + 31) // 32
    ldw = (W + 3) // 4 * 4
    NPc = B.count_planes(M)
    g = torch.randn(M, ld, device=dev)
    m = torch.zeros(M, ld, device=dev)
    x = torch.randn(d, device=dev)
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=dev)
    act = torch.zeros(M, ldw, dtype=torch.int32, device=dev)
    counts = torch.zeros(NPc, ldw, dtype=torch.int32, device=dev)
    vs = torch.zeros(W, dtype=torch.int32, device=dev)
    va = torch.zeros(W, dtype=torch.int32, device=dev)
    mean, m2 = torch.zeros(d, device=dev), torch.zeros(d, device=dev)
    sums = torch.zeros(2, dtype=torch.float64, device=dev)
    B.sign_pack(g, M, d, ld, bits, ldw)
    rows = []

    def rec(name, ms, nbytes):
        gbs = nbytes / (ms * 1e-3) / 1e9
        rows.append((d, M, name, ms * 1e3, gbs, gbs / peak_gbs(), int(nbytes >= 2 * L2_BYTES)))

    # Algorithm 3 as printed (no momentum): one fused kernel up to 8 workers, and up to 32 on long vectors
    sign_only_bytes = (4.125 * M + 8.125 + (0.0 if B.step_is_fused(M, d, False) else (M + 1) / 8.0)) * d
    rec("signsgd_step_sign_only", time_launches(lambda s: B.signsgd_step(x, g, None, M, d, ld, 0.0, 1e-4, bits, ldw, vs),
                                                1, reps), sign_only_bytes)
    B.sign_pack(g, M, d, ld, bits, ldw)
    rec("signum_warmup_pack", time_launches(lambda s: B.signum_warmup_pack(g, m, M, d, ld, 0.9, bits, ldw), 1, reps),
        12.125 * M * d)
    rec("vote_counts", time_launches(lambda s: B.vote_counts(bits, M, d, ldw, counts, ldw), 1, reps),
        (M + NPc) / 8.0 * d)
    rec("sum_apply", time_launches(lambda s: B.sum_apply(x, counts, M, d, ldw, 1e-4), 1, reps), (8 + NPc / 8.0) * d)
    rec("ternary_pack", time_launches(lambda s: B.ternary_pack(g, m, M, d, ld, 0.9, 0.1, bits, act, ldw), 1, reps),
        12.25 * M * d)
    rec("quorum_vote", time_launches(lambda s: B.quorum_vote(bits, act, M, d, ldw, 2, vs, va), 1, reps),
        (2 * M + 2) / 8.0 * d)
    rec("ternary_apply", time_launches(lambda s: B.ternary_apply(x, vs, va, d, 1e-4), 1, reps), 8.25 * d)
    rec("welford_update", time_launches(lambda s: B.welford_update(g[0], 3, mean, m2, d), 1, reps), 20.0 * d)
    lib = B.lib()
    sp, xp, st = sums.data_ptr(), x.data_ptr(), None
    rec("density_sums", time_launches(lambda s: lib.ssgd_density_sums(xp, d, 0, sp, torch.cuda.current_stream().cuda_stream),
                                      1, reps), 4.0 * d)
    return rows


def run_yardsticks(log2n: int, reps: int, dev) -> list:
    """Plain streaming library kernels over 2^log2n floats, as yardsticks for what this board's HBM gives to
    each read : write mix (nothing here is part of the step): (name, us, GB/s) rows."""
    n = 1 << log2n
    a, b = torch.randn(n, device=dev), torch.randn(n, device=dev)
    c = torch.empty(n, device=dev)
    g = torch.randn(4, n // 4, device=dev)
    m = torch.zeros(4, n // 4, device=dev)
    bits = torch.zeros(4, n // 128, dtype=torch.int32, device=dev)
    cases = [
        ("torch add c <- a + b (2 reads : 1 write)", lambda: torch.add(a, b, out=c), 12 * n),
        ("torch add_ a <- a + b in place (2 : 1)", lambda: a.add_(b, alpha=1e-6), 12 * n),
        ("torch lerp_ a <- a + w (b - a) in place (2 : 1)", lambda: a.lerp_(b, 0.1), 12 * n),
        ("ssgd_signum_momentum_pack, M = 4 (2 : 1 + 1/8)", lambda: B.signum_momentum_pack(g, m, 4, n // 4, n // 4, 0.9, bits, n // 128), 12.125 * n),
        ("torch mul_ a <- 0.999 a in place (1 : 1)", lambda: a.mul_(0.999), 8 * n),
        ("ssgd_sign_apply (1 : 1 + 1/8)", lambda: B.sign_apply(a, bits.view(-1), n, 1e-7), 8.125 * n),
        ("torch sum(a) (read only)", lambda: torch.sum(a), 4 * n),
        ("ssgd_sign_pack, M = 4 (read only + 1/8)", lambda: B.sign_pack(g, 4, n // 4, n // 4, bits, n // 128), 4.125 * n),
        ("torch fill_ (write only)", lambda: c.fill_(1.0), 4 * n),
    ]
    rows = []
    for name, fn, nbytes in cases:
        ms = time_launches(lambda s: fn(), 1, reps)
        rows.append((name, ms * 1e3, nbytes / (ms * 1e-3) / 1e9))
    return rows


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--min-log2", type=int, default=10)
    ap.add_argument("--max-log2", type=int, default=28)
    ap.add_argument("--workers", default="1,3,7,15,31")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--out", default=None)
    ap.add_argument("--plain", action="store_true",
                    help="issue every launch from the host instead of replaying a CUDA graph (times then include "
                         "the host's per-call cost; meant for runs under a profiler)")
    ap.add_argument("--yardsticks", type=int, default=None, metavar="LOG2N",
                    help="instead of the sweep, time plain streaming library kernels (and this library's) over 2^LOG2N floats")
    ap.add_argument("--variants", default=None, metavar="LOG2D,M",
                    help="instead of the sweep, time the calls beside the main path at d = 2^LOG2D with M workers")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device")
    global PLAIN_LAUNCHES
    PLAIN_LAUNCHES = args.plain
    dev = torch.device("cuda", 0)
    B.lib()
    if args.yardsticks is not None:
        print("kernel\tus_per_launch\tGBps\tfrac_of_measured_peak")
        for name, us, gbs in run_yardsticks(args.yardsticks, max(2, args.reps // 4), dev):
            print("%s\t%.1f\t%.0f\t%.3f" % (name, us, gbs, gbs / peak_gbs()), flush=True)
        return 0
    out = open(args.out, "w") if args.out else None
    header = "d\tM\tkernel\tus_per_launch\talgorithmic_GBps\tfrac_of_measured_peak\tcold"
    print(header)
    if out:
        out.write(header + "\n")
    if args.variants:
        k, M = [int(t) for t in args.variants.split(",")]
        for r in run_variants(1 << k, M, max(2, args.reps // 4), dev):
            line = "%d\t%d\t%s\t%.2f\t%.1f\t%.3f\t%d" % r
            print(line, flush=True)
            if out:
                out.write(line + "\n")
        if out:
            out.close()
        return 0
    for M in [int(t) for t in args.workers.split(",")]:
        for k in range(args.min_log2, args.max_log2 + 1):
            reps = args.reps if k < 24 else max(2, args.reps // 8)
            for r in run_point(1 << k, M, reps, dev):
                line = "%d\t%d\t%s\t%.2f\t%.1f\t%.3f\t%d" % r
                print(line, flush=True)
                if out:
                    out.write(line + "\n")
            torch.cuda.empty_cache()
    if out:
        out.close()


if __name__ == "__main__":
    sys.exit(main())
