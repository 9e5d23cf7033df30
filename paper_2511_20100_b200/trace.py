"""Device-side timeline of one call, from the trace build of the library.

    python -m paper_2511_20100_b200.trace C2                  # a benchmark configuration (C1..C5, X1..)
    python -m paper_2511_20100_b200.trace 4096 4096 4096      # mtmc_fused_linear, GELU-tanh, bf16 out
    options: --cta-pair N  --split-k N  --stream-k N  --repeat R  --csv FILE

Builds libmtmcfused_trace.so (-DMTMC_TRACE) on first use, runs the call a few times to warm up, then once
more with a trace buffer and prints, over the CTAs of the launch: when each role started and ended
(microseconds from the first CTA's entry), the SM clock the CTAs ran at, how many cycles the producer waited for a
free ring stage, the MMA issuer for data (in all, on the first k-blocks of its work items, longest single wait) and for a
drained accumulator, how long it took to issue a stage's tensor-core work, the epilogue for an accumulator, and
nanoseconds per k-block.
The figures describe the kernels' pipelines; they are taken with the instrumented build and are not
benchmark results.
"""
from __future__ import annotations

import argparse
import os
import sys

os.environ["MTMC_LIB_VARIANT"] = "trace"

import torch  # noqa: E402

from . import binding as B  # noqa: E402
from . import inputs  # noqa: E402

WORDS = 32
NAMES = ["start_ns", "setup_ns", "prod_first_ns", "prod_last_ns", "prod_stall", "mma_first_ns", "mma_last_ns", "mma_stall_data",
         "mma_stall_acc", "mma_kblocks", "epi_first_ns", "epi_end_ns", "epi_stall", "epi_busy", "epi_items", "epi_handover", "end_ns",
         "xchg_ready", "xchg_send", "xchg_recv", "xchg_sum", "start_clk", "end_clk", "mma_stall_head", "mma_stall_max", "mma_issue"]


def _problem(args):
    if len(args.what) == 1:
        c = inputs.CONFIGS.get(args.what[0]) or inputs.EXTRA_CONFIGS[args.what[0]]
    else:
        M, N, K = (int(v) for v in args.what)
        c = dict(op="fused_linear", M=M, N=N, K=K, act="gelu_tanh", out_dtype="bf16", seed=1)
    if c["op"] == "fused_linear_mxfp8":
        mi = inputs.mx_linear_inputs(c["M"], c["N"], c["K"], c["seed"])
        d = [mi.X.cuda(), mi.SX.cuda(), mi.W.cuda(), mi.SW.cuda(), mi.b.cuda()]
        return c, lambda: B.mtmc_fused_linear_mxfp8(d[0], d[1], d[2], d[3], d[4], c["act"], c["out_dtype"])
    if c["op"] == "fused_linear_fp8":
        fi = inputs.fp8_linear_inputs(c["M"], c["N"], c["K"], c["seed"])
        d = [fi.X.cuda(), fi.W.cuda(), fi.b.cuda()]
        return c, lambda: B.mtmc_fused_linear_fp8(d[0], d[1], d[2], fi.scale_x, fi.scale_w, c["act"], c["out_dtype"])
    if c["op"] == "swiglu":
        si = inputs.swiglu_inputs(c["M"], c["N"], c["K"], c["seed"])
        d = [si.X.cuda(), si.Wg.cuda(), si.Wu.cuda()]
        return c, lambda: B.mtmc_swiglu(d[0], d[1], d[2])
    li = inputs.linear_inputs(c["M"], c["N"], c["K"], c["seed"])
    d = [li.X.cuda(), li.W.cuda(), li.b.cuda()]
    if c["op"] == "linear_lse":
        return c, lambda: B.mtmc_linear_lse(d[0], d[1], d[2])
    if c["op"] == "linear_rowmax":
        return c, lambda: B.mtmc_linear_rowmax(d[0], d[1], d[2])
    if c["op"] == "linear_cross_entropy":
        tgt = inputs.targets(c["M"], c["N"], c["seed"]).cuda()
        return c, lambda: B.mtmc_linear_cross_entropy(d[0], d[1], d[2], tgt)
    if c["op"] == "linear_softmax":
        return c, lambda: B.mtmc_linear_softmax(d[0], d[1], d[2], c["out_dtype"])
    if c["op"] == "fused_linear_residual":
        R = inputs.residual(c["M"], c["N"], c["seed"]).cuda()
        return c, lambda: B.mtmc_fused_linear_residual(d[0], d[1], d[2], R, c["act"], c["out_dtype"])
    if c["op"] != "fused_linear":
        raise SystemExit("no trace driver for %s" % c["op"])
    return c, lambda: B.mtmc_fused_linear(d[0], d[1], d[2], c["act"], c["out_dtype"])


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", nargs="+", help="a configuration name, or M N K")
    ap.add_argument("--cta-pair", type=int, default=0)
    ap.add_argument("--split-k", type=int, default=0)
    ap.add_argument("--stream-k", type=int, default=0)
    ap.add_argument("--repeat", type=int, default=3, help="untraced calls before the traced one")
    ap.add_argument("--csv", default="", help="write the raw per-CTA records here")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    B.load()
    assert B.mtmc_trace_enabled()
    B.mtmc_set_tuning(split_k=args.split_k, cta_pair=args.cta_pair)
    B.mtmc_set_schedule(args.stream_k)
    c, call = _problem(args)
    for _ in range(args.repeat):
        call()
    torch.cuda.synchronize()
    buf = torch.zeros(1024 * WORDS, dtype=torch.int64, device="cuda")
    B.mtmc_set_trace(buf)
    call()
    torch.cuda.synchronize()
    B.mtmc_set_trace(None)
    B.mtmc_check_status()
    kernel = B.mtmc_last_kernel_name()
    rec = buf.cpu().view(-1, WORDS).numpy()
    rec = rec[rec[:, 0] != 0]
    if len(rec) == 0:
        raise SystemExit("%s wrote no trace (the single-CTA tiled kernels are not instrumented)" % kernel)
    t0 = rec[:, 0].min()
    print("%s  M=%d N=%d K=%d  kernel %s  %d CTAs traced" % (" ".join(args.what), c["M"], c["N"], c["K"], kernel, len(rec)))

    def us(col, only=None):
        v = rec[:, col]
        v = v[v != 0] if only is None else v[only]
        return (float("nan"),) * 3 if len(v) == 0 else ((v.min() - t0) / 1e3, (float(v.mean()) - t0) / 1e3, (v.max() - t0) / 1e3)

    for label, col in (("entry", 0), ("set-up done", 1), ("first load", 2), ("last load", 3), ("first MMA", 5), ("last MMA commit", 6),
                       ("first accumulator ready", 10), ("last epilogue done", 11), ("teardown", 16)):
        lo, mean, hi = us(col)
        print("  %-26s min %9.2f  mean %9.2f  max %9.2f us" % (label, lo, mean, hi))
    timed = (rec[:, 16] > rec[:, 0] + 100000) & (rec[:, 22] > rec[:, 21])      # %globaltimer ticks are too coarse for CTAs shorter than 0.1 ms
    if timed.any():
        mhz = (rec[timed, 22] - rec[timed, 21]).astype(float) / (rec[timed, 16] - rec[timed, 0]).astype(float) * 1e3
        print("  SM clock over the CTAs' lifetimes: %.0f MHz (min %.0f, max %.0f)" % (mhz.mean(), mhz.min(), mhz.max()))
    issuers = rec[:, 9] > 0
    if issuers.any():
        kb = rec[issuers, 9].astype(float)
        span = (rec[issuers, 6] - rec[issuers, 5]).astype(float)      # ns from first MMA to last commit
        print("  MMA issuers: %d, k-blocks each %.1f (min %d, max %d); first MMA to last commit %.2f us mean = %.1f ns per k-block" % (
            int(issuers.sum()), kb.mean(), kb.min(), kb.max(), span.mean() / 1e3, (span / kb).mean()))
        print("  MMA issuer waits, cycles per CTA: for data %.0f (%.0f per k-block; %.0f of it on the first ring-depth k-blocks of the work items; longest wait %.0f), "
              "for a drained accumulator %.0f" % (rec[issuers, 7].mean(), (rec[issuers, 7] / kb).mean(), rec[issuers, 23].mean(), rec[issuers, 24].max(),
                                                  rec[issuers, 8].mean()))
    if issuers.any() and rec[issuers, 25].any():
        print("  MMA issuer, from a stage's data being there to its commit issued: %.0f cycles per k-block" % (rec[issuers, 25] / kb).mean())
    print("  producer waits for a free stage: %.0f cycles per CTA" % rec[:, 4].mean())
    items = rec[:, 14].astype(float)
    has = items > 0
    if has.any():
        print("  epilogue (first warp): %.1f items per CTA, busy %.0f cycles per item, waiting %.0f cycles per CTA, hand-overs %.0f cycles per CTA" % (
            items[has].mean(), (rec[has, 13] / items[has]).mean(), rec[has, 12].mean(), rec[has, 15].mean()))
    if rec[:, 18].any():
        print("  cluster split-K exchange (first warp), cycles per CTA: peers ready %.0f, send %.0f, wait for the peers' parts %.0f, sum %.0f" % (
            rec[:, 17].mean(), rec[:, 18].mean(), rec[:, 19].mean(), rec[:, 20].mean()))
    if args.csv:
        with open(args.csv, "w") as f:
            f.write("cta," + ",".join(NAMES) + "\n")
            for i, r in enumerate(rec):
                f.write("%d," % i + ",".join(str(int(v) - int(t0) if n.endswith("_ns") and v else int(v)) for n, v in zip(NAMES, r)) + "\n")


if __name__ == "__main__":
    sys.exit(main())
