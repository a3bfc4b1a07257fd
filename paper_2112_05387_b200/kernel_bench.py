"""Time one stand-alone convolution through the C ABI (lp_conv2d) and print its throughput.

  python -m paper_2112_05387_b200.kernel_bench --op fwd --N 128 --H 32 --W 32 --Cin 160 --Cout 160 [--R 3]
      [--stride 1] [--impl 2] [--reps 20]

Used for kernel-level measurements and as the small, single-kernel command that profiler captures
are taken on.  Inputs are seeded N(0,1) tensors; the result is not checked here (tests do that).
"""
import argparse
import json

import numpy as np


def main():
    import torch
    import paper_2112_05387_b200 as lp
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="fwd", choices=["fwd", "dgrad", "wgrad"])
    ap.add_argument("--N", type=int, default=128)
    ap.add_argument("--H", type=int, default=32)
    ap.add_argument("--W", type=int, default=32)
    ap.add_argument("--Cin", type=int, default=160)
    ap.add_argument("--Cout", type=int, default=160)
    ap.add_argument("--R", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--impl", type=int, default=2)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--stats", action="store_true")
    ap.add_argument("--sustain", type=float, default=0.0, help="also run back to back for this many seconds "
                    "and report the sustained rate with the clocks and power seen (the part is power-capped)")
    a = ap.parse_args()
    pad = 1 if a.R == 3 else (0 if a.R == 1 else a.R // 2)
    OH = (a.H + 2 * pad - a.R) // a.stride + 1
    OW = (a.W + 2 * pad - a.R) // a.stride + 1
    dev = "cuda:0"
    g = torch.Generator(device=dev).manual_seed(0)
    x = torch.randn(a.N, a.H, a.W, a.Cin, device=dev, generator=g).to(torch.bfloat16)
    dy = torch.randn(a.N, OH, OW, a.Cout, device=dev, generator=g).to(torch.bfloat16)
    w = (torch.randn(a.Cout, a.R, a.R, a.Cin, device=dev, generator=g) * (2.0 / (a.R * a.R * a.Cin)) ** 0.5).float()
    op = {"fwd": lp.LP_CONV_FWD, "dgrad": lp.LP_CONV_DGRAD, "wgrad": lp.LP_CONV_WGRAD}[a.op]
    if a.op == "fwd":
        ta, tb, out = x, w, torch.empty(a.N, OH, OW, a.Cout, device=dev, dtype=torch.bfloat16)
    elif a.op == "dgrad":
        ta, tb, out = dy, w, torch.empty(a.N, a.H, a.W, a.Cin, device=dev, dtype=torch.bfloat16)
    else:
        ta, tb, out = x, dy, torch.empty(a.Cout, a.R, a.R, a.Cin, device=dev, dtype=torch.float32)
    nbytes = lp.lp_conv2d_scratch_bytes(a.Cin, a.Cout, a.R)
    scratch = torch.zeros(nbytes + 256, dtype=torch.uint8, device=dev)
    base = (scratch.data_ptr() + 255) // 256 * 256
    stats = torch.zeros(2 * a.Cout, dtype=torch.float64, device=dev) if (a.stats and a.op == "fwd") else None
    times = []
    for i in range(a.reps + 3):
        st, ms = lp.lp_conv2d(op, lp.LP_BF16, a.impl, a.N, a.H, a.W, a.Cin, a.Cout, a.R, a.stride, pad, ta, tb, out,
                              stats, base, nbytes, timed=True)
        if st != 0:
            raise SystemExit("lp_conv2d: " + lp.lp_status_string(st))
        if i >= 3:
            times.append(ms)
    flops = 2.0 * a.N * OH * OW * a.Cout * a.R * a.R * a.Cin
    med = float(np.median(times))
    out_line = {"op": a.op, "shape": [a.N, a.H, a.W, a.Cin, a.Cout, a.R, a.stride], "ms_median": med,
                "ms_min": float(min(times)), "tflops_median": flops / med / 1e9,
                "tflops_best": flops / min(times) / 1e9}
    if a.sustain > 0:
        import subprocess
        import time
        q = subprocess.Popen(["nvidia-smi", "-i", "0", "--query-gpu=clocks.sm,power.draw", "--format=csv,noheader,nounits",
                              "-lms", "100"], stdout=subprocess.PIPE, text=True)
        t0 = time.time()
        sus = []
        while time.time() - t0 < a.sustain:
            for _ in range(50):
                st, ms = lp.lp_conv2d(op, lp.LP_BF16, a.impl, a.N, a.H, a.W, a.Cin, a.Cout, a.R, a.stride, pad, ta, tb,
                                      out, stats, base, nbytes, timed=True)
                sus.append(ms)
        q.terminate()
        rows = [r.split(",") for r in q.stdout.read().strip().splitlines() if "," in r]
        tail_ms = float(np.median(sus[len(sus) // 2:]))
        out_line.update({"sustained_tflops": flops / tail_ms / 1e9,
                         "sm_mhz_median": float(np.median([float(r[0]) for r in rows[len(rows) // 2:]])) if rows else None,
                         "power_w_median": float(np.median([float(r[1]) for r in rows[len(rows) // 2:]])) if rows else None})
    print(json.dumps(out_line))


if __name__ == "__main__":
    main()
