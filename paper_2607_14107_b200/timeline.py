"""Kernel timeline of real forwards (debugging / profiling aid).

A library built with -DPOLESTAR_TRACE (`python -m paper_2607_14107_b200.build --trace`, built here on
demand) and run with POLESTAR_KERNEL_TRACE=1 records, for every kernel of a forward, the time at which
block 0 had its dependencies resolved (and, for the GEMM, when its CTA 0 finished).  Consecutive
stamps give what each kernel really costs inside the pipeline, launch gaps included -- something
neither CUDA events (too coarse) nor ncu (serialised, idle clocks) show.

    python -m paper_2607_14107_b200.timeline [--config c2] [--forwards 6]
"""
from __future__ import annotations

import argparse
import collections
import ctypes as C
import os

import numpy as np

NAMES = {1: "build_rows", 2: "embed", 3: "prep_qkv", 4: "prep_rows", 5: "prep_head", 7: "attention/select",
         10: "head_list", 11: "conf_partial", 12: "conf_final", 13: "commit", 14: "delta", 15: "keep_hidden",
         100: "gemm_qkv", 101: "gemm_o", 102: "gemm_gate_up", 103: "gemm_down", 104: "gemm_lm_head",
         200: "gemm_qkv:cta0_done", 201: "gemm_o:cta0_done", 202: "gemm_gate_up:cta0_done",
         203: "gemm_down:cta0_done", 204: "gemm_lm_head:cta0_done",
         311: "attn:end"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c2")
    ap.add_argument("--forwards", type=int, default=6)
    ap.add_argument("--max-steps", type=int, default=0, help="override the step budget (fewer steps: more tokens per step, blocks turn over sooner)")
    ap.add_argument("--attn-cycles", action="store_true", help="print the cycle counters of the last attention launch")
    ap.add_argument("--entry", action="store_true", help="also print forward 0, the block-entry forward of the first block")
    a = ap.parse_args()
    os.environ["POLESTAR_KERNEL_TRACE"] = "1"
    from . import build as Bu
    os.environ["POLESTAR_LIB"] = Bu.build(trace=True)
    import torch
    from . import binding as Bd, inputs as I
    m, p = I.config(a.config)
    if a.max_steps:
        import dataclasses
        p = dataclasses.replace(p, max_steps=a.max_steps)
    dec = Bd.Polestar(m, Bd.make_packed_weights(m), p, I.make_prompt(m, p).numpy())
    dec.commit()
    for _ in range(a.forwards):
        dec.step()
        dec.commit()
    torch.cuda.synchronize()
    out = np.zeros(8192, np.int64)
    Bd._check(Bd.load().polestar_read(dec.ctx, Bd.READ_TRACE_KERNELS, 0, out.ctypes.data_as(C.c_void_p), 65536))
    if a.attn_cycles:
        # cycle counters of the last attention launch (attn_tc.cuh dbg_clock): per thread, relative to its point 0
        for name, base in (("epilogue rows 64..", 0), ("epilogue rows 0..", 20), ("producer", 40), ("mma", 50)):
            v = out[8100 + base:8100 + base + 20]
            t0 = min(x for x in out[8100:8160] if x > 0)
            print(f"  {name:20s}", [int(x - t0) if x > 0 else None for x in v])
    n = min(int(out[0]), 4000)
    ids, ts = out[1:1 + 2 * n:2], out[2:2 + 2 * n:2].astype(np.float64) / 1000.0
    order = np.argsort(ts, kind="stable")
    ids, ts = ids[order], ts[order]
    starts = [i for i in range(n) if ids[i] == 1]
    for f in range(0 if a.entry else 1, len(starts) - 1):
        lo, hi = starts[f], starts[f + 1]
        agg = collections.OrderedDict()
        for i in range(lo, hi):
            x = agg.setdefault(NAMES.get(int(ids[i]), str(int(ids[i]))), [0, 0.0])
            x[0] += 1
            x[1] += ts[i + 1] - ts[i]
        print(f"forward {f}: {ts[hi] - ts[lo]:.0f} us, {hi - lo} stamps")
        for k, v in agg.items():
            print(f"    {k:24s} x{v[0]:3d}  avg {v[1] / v[0]:7.1f} us  total {v[1]:8.0f} us")


if __name__ == "__main__":
    main()
