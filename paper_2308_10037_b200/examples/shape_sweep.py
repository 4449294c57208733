"""Which kernel serves a row length, and how fast one fused pass runs on it.

    python -m paper_2308_10037_b200.examples.shape_sweep 28 30 100 256 1001 4096 12000
    python -m paper_2308_10037_b200.examples.shape_sweep --bf16 --mb 256 64 100 4096

For every row length n it builds a random m x n matrix of about ``--mb`` megabytes (larger than the L2, so the pass
streams from HBM), asks the library for its launch plan (``lr_plan_query``), times ``lr_loss_grad`` with CUDA events
(3 untimed calls, then 20 timed ones) and prints the plan and the algorithmic bytes per second, (elem_bytes*m*n + 4*m) per
call -- the figures of the shape-coverage table in the design doc section 6.  ``--shift K`` starts the matrix K elements
into its allocation (a view that is aligned to its element size only).
"""
from __future__ import annotations

import argparse

import torch

from paper_2308_10037_b200 import api, build


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("n", type=int, nargs="+", help="row lengths (columns)")
    ap.add_argument("--mb", type=int, default=512, help="size of X in MiB (default 512)")
    ap.add_argument("--bf16", action="store_true", help="store X as bfloat16")
    ap.add_argument("--shift", type=int, default=0, help="offset of the matrix into its allocation, in elements")
    ap.add_argument("--device", type=int, default=0)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: the library has no CPU path")
    build.build()
    torch.cuda.set_device(args.device)
    eb = 2 if args.bf16 else 4
    ctx = api.Context(n_max=max(args.n), device=args.device)
    names = {0: "k_stream_rows", 1: "k_stream_split", 2: "k_generic", 3: "k_stream_rows (element-wise)", 4: "k_stream_wide"}
    for n in args.n:
        m = max(1, (args.mb << 20) // (eb * n))
        buf = torch.randn(m * n + args.shift, device="cuda")
        if args.bf16:
            buf = buf.to(torch.bfloat16)
        X = buf[args.shift:args.shift + m * n].view(m, n)
        y = (torch.rand(m, device="cuda") < 0.5).float()
        w = torch.randn(n, device="cuda") / n ** 0.5
        b = torch.zeros(1, device="cuda")
        for _ in range(3):
            ctx.loss_grad(X, y, w, b)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            ctx.loss_grad(X, y, w, b)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 20
        p = api.plan_query(m, n, x_aligned16=X.data_ptr() % 16 == 0, bf16=args.bf16,
                           sm_count=torch.cuda.get_device_properties(args.device).multi_processor_count)
        print(f"n={n:6d} m={m:10d} {names[p['variant']]:30s} warps={p['threads'] // 32:2d} lanes/row={p['lanes_per_row']:3d} "
              f"per-lane={p['vec_per_lane']:2d} rows/batch={p['rows_per_batch']:2d} stages={p['stages']} "
              f"{ms:8.4f} ms {(eb * m * n + 4 * m) / ms / 1e6:7.0f} GB/s", flush=True)
        del buf, X, y
    status = ctx.device_status()
    if status:
        raise SystemExit(f"device status {status}: {api.status_string(status)}")


if __name__ == "__main__":
    main()
