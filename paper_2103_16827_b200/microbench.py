"""Times one operation of the library on synthetic int8 data (seeded), through the C ABI.

  python -m paper_2103_16827_b200.microbench conv B C_in C_out T [--iters N]
  python -m paper_2103_16827_b200.microbench dw   B C T K [--stride S] [--dilation D]
  python -m paper_2103_16827_b200.microbench tcs  B C_in C_out T K
  python -m paper_2103_16827_b200.microbench add  B C T N_TERMS
  python -m paper_2103_16827_b200.microbench peak [KBLOCKS]      (int8 tensor-core rate of this GPU)

The launches are queued behind a short device-side delay so that they run back to back and the
figure is device time per launch, not host launch latency.  Prints one JSON line.  This is also
the small, single-kernel program used for profiler captures.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import Context


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["conv", "dw", "tcs", "add", "peak"])
    ap.add_argument("dims", type=int, nargs="*")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--dilation", type=int, default=1)
    ap.add_argument("--shift", type=int, default=24)
    ap.add_argument("--no-scratch", action="store_true", help="conv: lend no scratch (K-tap convolutions then use the generic kernel)")
    ap.add_argument("--no-delay", action="store_true", help="do not queue the launches behind a device delay")
    ap.add_argument("--residual", type=int, default=0,
                    help="conv: number of residual tensors added in the epilogue (each rescaled on its own)")
    args = ap.parse_args()
    rng = np.random.Generator(np.random.PCG64(0))
    ctx = Context(0)
    if args.op == "peak":      # the int8 tensor-core rate of this GPU: dims = [K blocks per SM], default 2000 (~0.5 ms)
        kb = args.dims[0] if args.dims else 2000
        runs = [ctx.measure_int8_tensor_peak(kb) for _ in range(max(1, args.iters))]
        print(json.dumps({"op": "peak", "kblocks": kb, "tops_best": max(r[0] for r in runs),
                          "tops_median": sorted(r[0] for r in runs)[len(runs) // 2], "ms": runs[-1][1]}))
        return

    def rq(C):
        return (_dev(rng.integers(1 << 14, 1 << 15, size=C).astype(np.int32)),
                _dev(np.full(C, args.shift, np.uint8)))

    if args.op == "conv":
        B, Ci, Co, T = args.dims[:4]
        K = args.dims[4] if len(args.dims) > 4 else 1          # conv B C_in C_out T [K]
        T_out = (T - 1) // args.stride + 1
        x = _dev(rng.integers(-128, 128, size=(B, Ci, T), dtype=np.int8))
        w = _dev(rng.integers(-127, 128, size=(Co, Ci, K), dtype=np.int8))
        bias = _dev(rng.integers(-4096, 4097, size=Co).astype(np.int32))
        m, s = rq(Co)
        y = torch.empty((B, Co, T_out), dtype=torch.int8, device="cuda")
        if not args.no_scratch:
            ctx.set_conv_scratch(torch.empty(max(256, ctx.conv_scratch_bytes(B, Ci, Co, T, K, args.stride)),
                                             dtype=torch.uint8, device="cuda"))
        res = [_dev(rng.integers(-128, 128, size=(B, Co, T_out), dtype=np.int8)) for _ in range(args.residual)]
        tm = [int(v) for v in rng.integers(1 << 13, 1 << 14, size=args.residual + 1)]
        ts = [15] * (args.residual + 1)
        if args.residual:
            fn = lambda: ctx.conv(x, w, bias, 4096, m, s, True, stride=args.stride, dilation=args.dilation,
                                  terms=[None] + res, term_mult=tm, term_shift=ts, y=y)
        else:
            fn = lambda: ctx.conv(x, w, bias, 4096, m, s, True, stride=args.stride, dilation=args.dilation, y=y)
        macs, nbytes = B * Ci * Co * T_out * K, B * (T * Ci + T_out * Co * (1 + args.residual)) + Ci * Co * K
    elif args.op == "dw":
        B, C, T, K = args.dims
        x = _dev(rng.integers(-128, 128, size=(B, C, T), dtype=np.int8))
        w = _dev(rng.integers(-127, 128, size=(C, K), dtype=np.int8))
        m, s = rq(C)
        T_out = (T - 1) // args.stride + 1
        y = torch.empty((B, C, T_out), dtype=torch.int8, device="cuda")
        fn = lambda: ctx.dw_conv(x, w, args.stride, args.dilation, m, s, y=y)
        macs, nbytes = B * C * T_out * K, B * C * (T + T_out)
    elif args.op == "tcs":
        B, Ci, Co, T, K = args.dims
        x = _dev(rng.integers(-128, 128, size=(B, Ci, T), dtype=np.int8))
        wd = _dev(rng.integers(-127, 128, size=(Ci, K), dtype=np.int8))
        wp = _dev(rng.integers(-127, 128, size=(Co, Ci), dtype=np.int8))
        bias = _dev(rng.integers(-4096, 4097, size=Co).astype(np.int32))
        md, sd = rq(Ci)
        mp, sp = rq(Co)
        T_out = (T - 1) // args.stride + 1
        y = torch.empty((B, Co, T_out), dtype=torch.int8, device="cuda")
        ws = torch.empty(max(256, ctx.tcs_block_workspace_bytes(B, Ci, Co, T, K, args.stride, args.dilation)),
                         dtype=torch.uint8, device="cuda")
        fn = lambda: ctx.tcs_block(x, wd, args.stride, args.dilation, md, sd, wp, bias, 4096, mp, sp, True, y=y,
                                   workspace=ws)
        macs, nbytes = B * T_out * Ci * (K + Co), B * (Ci * T + Co * T_out)
    else:
        B, C, T, n = args.dims
        terms = [_dev(rng.integers(-128, 128, size=(B, C, T), dtype=np.int8)) for _ in range(n)]
        mult = rng.integers(1 << 14, 1 << 15, size=n)
        shift = np.full(n, 15)
        y = torch.empty((B, C, T), dtype=torch.int8, device="cuda")
        fn = lambda: ctx.residual_requant_add(terms, mult, shift, True, y=y)
        macs, nbytes = 0, B * C * T * (n + 1)

    for _ in range(args.warmup):
        fn()
    ctx.poll_status()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    if not args.no_delay:
        torch.cuda._sleep(10_000_000)
    e0.record()
    for _ in range(args.iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ctx.poll_status()
    us = e0.elapsed_time(e1) / args.iters * 1e3
    print(json.dumps({"op": args.op, "dims": args.dims, "us_per_launch": us,
                      "tops": 2 * macs / us / 1e6 if macs else None, "gbs_algorithmic": nbytes / us / 1e3,
                      "launches": ctx.launch_count()}))


if __name__ == "__main__":
    main()
