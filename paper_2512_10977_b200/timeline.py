"""Where one decode_attn call spends its time on the device.

    python -m paper_2512_10977_b200.timeline [--workload c2] [--kv fp8] [--calls 5]
    python -m paper_2512_10977_b200.timeline --workload c5a --cascade      (the prefix kernel's phases)
    python -m paper_2512_10977_b200.timeline --workload c2 --extend 512    (the same kernel in extend mode)

Builds the timeline variant of the library (the same sources with -DDA_TIMELINE: the plan, partition and
merge kernels keep %globaltimer stamps of their phases), runs the workload through it and prints the
phases of the last call in ns, relative to the plan kernel's start.  The stamps cost a few stores per
tile, so the call is 1-3 % slower than with the normal library; use bench.py for throughput.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "c5a", "c5b"])
    ap.add_argument("--kv", default="bf16", choices=["bf16", "fp8"])
    ap.add_argument("--calls", type=int, default=5, help="calls before the one that is reported")
    ap.add_argument("--cascade", action="store_true", help="c5a: decode_attn_cascade; report the prefix kernel")
    ap.add_argument("--extend", type=int, default=0, metavar="LQ", help="decode_attn_extend with LQ new tokens")
    args = ap.parse_args()

    from . import binding, build
    binding.use_library(build.build_diag())
    import torch
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import workloads
    case = workloads.RECIPES[args.workload]("cuda", kv_dtype=args.kv)
    out = torch.empty(case.q.shape, dtype=torch.float32, device="cuda")
    lse = torch.empty(case.q.shape[:2], dtype=torch.float32, device="cuda")

    if args.cascade or args.extend:
        return prefix_report(args, binding, case, out, lse)

    def call():
        if args.kv == "fp8":
            binding.decode_attn_fp8kv(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table,
                                      case.seq_lens, case.window, case.scale, out=out, lse=lse)
        else:
            binding.decode_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, case.window,
                                case.scale, out=out, lse=lse)

    for _ in range(max(args.calls, 1)):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(20):
        call()
    e1.record()
    torch.cuda.synchronize()
    period_ns = e0.elapsed_time(e1) / 20 * 1e6
    binding.timeline(clear=True)
    call()
    tl = binding.timeline()

    R, MERGE, PLAN = 1024, 1024, 1036
    blocks = tl[:R]
    used = blocks[:, 4] > 0
    part = blocks[used]
    t0 = tl[PLAN:PLAN + 8, 0]
    t0 = int(t0[t0 > 0].min())
    rel = lambda x: int(x) - t0
    q = lambda col, f: rel(f(part[:, col]))
    print(f"workload {args.workload}, cache {args.kv}: {used.sum()} partition blocks, {int(part[:, 5].sum())} tiles, "
          f"{int(part[:, 6].sum())} (sequence, KV head) items; back-to-back calls every {period_ns:.0f} ns")
    print(f"plan kernel        : first block enters 0, last passes the wait for the kernel before it "
          f"{rel(tl[PLAN:PLAN + 8, 2].max())}, last block done {rel(tl[PLAN:PLAN + 8, 1].max())}")
    pl = tl[PLAN:PLAN + 8]
    print(f"  plan block 0     : lengths scanned {rel(pl[0, 3])}, cut made {rel(pl[0, 4])}, units written {rel(pl[0, 5])}, exit {rel(pl[0, 1])}")
    print(f"partition kernel   : first block enters {q(0, np.min)}, last passes the wait for the plan {q(1, np.max)}")
    print(f"  first tile ready : min {q(2, np.min)}  median {q(2, np.median)}  max {q(2, np.max)}")
    print(f"  last tile done   : min {q(3, np.min)}  median {q(3, np.median)}  max {q(3, np.max)}")
    print(f"  block exits      : min {q(4, np.min)}  median {q(4, np.median)}  max {q(4, np.max)}")
    end = part[:, 4].max()
    left = ", ".join(f"{(part[:, 4] > end - back).sum()} at -{back // 1000} us" for back in (15000, 10000, 7500, 5000, 2500, 1000))
    print(f"  blocks still running before the last exit: {left}")
    m = tl[MERGE:MERGE + 8]
    print(f"merge kernel       : first blocks resident {rel(m[:, 0].min())}, released {rel(m[:, 1].max())}, "
          f"their exit {rel(m[:, 2].max())}, last block of the grid done {rel(tl[MERGE + 8, 2])}")


def prefix_report(args, binding, case, out, lse) -> None:
    """Cycles per 128-token tile that one warp of each role of the prefix kernel's thread block 0 spent in
    its phases (the diagnostic build's clock64 counters), for a cascade or an extend call."""
    import torch
    if args.extend:
        q = torch.randn((case.B, args.extend) + tuple(case.q.shape[1:]), device="cuda",
                        generator=torch.Generator(device="cuda").manual_seed(7)).to(torch.bfloat16)
        out = torch.empty(q.shape, dtype=torch.float32, device="cuda")
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
        call = lambda: binding.decode_attn_extend(q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                                                  case.scale, out=out, lse=lse)
    else:
        call = lambda: binding.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                                                   16384, case.scale, out=out, lse=lse)
    binding.set_option("cascade_overlap", 0)   # the prefix kernel alone on all SMs
    for _ in range(max(args.calls, 1)):
        call()
    torch.cuda.synchronize()
    binding.timeline(clear=True)
    call()
    tl = binding.timeline()[1052:1058]
    tiles = max(int(tl[0, 5]), 1)
    ghz = tl[0, 6] / max(tl[0, 7], 1)
    per = lambda x: f"{x / tiles:7.0f}"
    print(f"prefix kernel, thread block 0: {tiles} tiles of 128 tokens, {tl[0, 6]} cycles = {tl[0, 7]} ns "
          f"({ghz:.2f} GHz), {tl[0, 6] / tiles:.0f} cycles per tile")
    print("cycles per tile        :   wait-1  wait-2    work   store")
    print(f"  softmax warp 0       : {per(tl[0, 0])} {per(tl[0, 1])} {per(tl[0, 2])} {per(tl[0, 3])}"
          f"   (scores ready; load + row maximum; exp2 + high/low parts; store P + arrive)  after the last tile {tl[0, 4]}")
    print(f"  score MMA warp       : {per(tl[1, 0])} {per(tl[1, 1])} {per(tl[1, 2])}           (PV products done; K landed; issue 8 MMAs)")
    print(f"  P_hi V MMA warp      : {per(tl[2, 0])} {per(tl[2, 1])} {per(tl[2, 2])}           (P written; V landed; issue 8 MMAs)")
    print(f"  P_lo V MMA warp      : {per(tl[3, 0])} {per(tl[3, 1])} {per(tl[3, 2])}")
    print(f"  K loader warp        : {per(tl[4, 0])}         {per(tl[4, 1])}           (buffer free; issue the tile's copies)")
    print(f"  V loader warp        : {per(tl[5, 0])}         {per(tl[5, 1])}")


if __name__ == "__main__":
    main()
