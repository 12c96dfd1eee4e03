"""Throughput sweeps of the decoding path over the method's knobs (Sec. 5.3 / Appendix D ablation axes): history
length h, drift threshold scale alpha, update threshold tau_upd, local-window size, clusters refreshed.

    python -m paper_2607_14107_b200.sweep [--config c2] [--logit-scale 30] [--max-steps 0] [--axes h,alpha,tau_upd,window,cluster_k]

Every point is the fastest of three decodes on synthetic weights (seeded), timed with CUDA events after one warm-up decode.  The
columns are what the kernels' cost depends on: tokens per second, tokens per forward (TPF), forwards, refresh
steps and rows refreshed.  Accuracy columns of the paper's figures need its trained weights and datasets and are
not reproduced; with random weights the commit behaviour is driven by `logit_scale` (sharper logits, more
confident rows), which is printed with the table.  Prints a markdown table.
"""
from __future__ import annotations

import argparse
import dataclasses

import torch

from . import binding as Bd
from . import inputs as I


def run_point(m, packed, p, prompt_dev):
    def once():
        dec = Bd.Polestar(m, packed, p, prompt_dev)
        info = dec.commit()
        refresh_steps = rows = 0
        while not info.all_done:
            dec.step()
            info = dec.commit()
            if info.rows_refreshed > 0:
                refresh_steps += 1
                rows += info.rows_refreshed
        dec.destroy()
        return info, refresh_steps, rows
    once()
    times = []
    for _ in range(3):                  # fastest of three timed decodes (a decode is only ~0.1-1 s: host hiccups show)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        info, refresh_steps, rows = once()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = min(times)
    return {"tokens_per_s": info.generated_non_eos / (ms / 1e3), "tpf": info.generated_non_eos / max(1, info.forwards),
            "forwards": info.forwards, "refresh_steps": refresh_steps, "rows_refreshed": rows, "ms": ms, "all_ms": times}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c2")
    ap.add_argument("--logit-scale", type=float, default=30.0)
    ap.add_argument("--max-steps", type=int, default=0)
    ap.add_argument("--axes", default="h,alpha,tau_upd,window,cluster_k")
    ap.add_argument("--show-all", action="store_true", help="append the three timings of every point")
    a = ap.parse_args()
    m, p0 = I.config(a.config)
    p0 = dataclasses.replace(p0, logit_scale=a.logit_scale, flags=p0.flags | Bd.FLAG_PROMPT_DEVICE)
    if a.max_steps:
        p0 = dataclasses.replace(p0, max_steps=a.max_steps)
    packed = Bd.make_packed_weights(m, seed=0, device="cuda")
    prompt_dev = I.make_prompt(m, p0).cuda()
    axes = {
        "h": [("hist", v) for v in (0, 1, 2, 5, 8)],
        "alpha": [("alpha", v) for v in (0.1, 1.0, 10.0, 100.0)],
        "tau_upd": [("tau_upd", v) for v in (-1, 1, 3, 7, 15, 10 ** 9)],
        "window": [(("win_prefix_blocks", "win_suffix_blocks"), v) for v in ((1, 0), (1, 1), (2, 1), (3, 1), (2, 2))],
        "cluster_k": [(("select_mode", "cluster_k"), (I.SELECT_CLUSTER_TOPK, v)) for v in (2, 4, 6, 8)],
    }
    print(f"workload {a.config} ({I.SHAPES.get(a.config, '?')}), batch {p0.batch}, prompt {p0.prompt_len} + gen {p0.gen_len}, "
          f"block {p0.block}, {p0.max_steps} steps, logit_scale {p0.logit_scale}; defaults: h {p0.hist}, alpha {p0.alpha}, "
          f"tau_upd {p0.tau_upd}, window ({p0.win_prefix_blocks}B, {p0.win_suffix_blocks}B)\n")
    print("| axis | value | tokens/s | TPF | forwards | refresh steps | rows refreshed | ms per decode |")
    print("|---|---|---|---|---|---|---|---|")
    for axis in a.axes.split(","):
        for key, val in axes[axis]:
            kw = dict(zip(key, val)) if isinstance(key, tuple) else {key: val}
            r = run_point(m, packed, dataclasses.replace(p0, **kw), prompt_dev)
            shown = "inf" if val == 10 ** 9 else (val[1] if axis == "cluster_k" else val)
            print(f"| {axis} | {shown} | {r['tokens_per_s']:.1f} | {r['tpf']:.2f} | {r['forwards']} | {r['refresh_steps']} | "
                  f"{r['rows_refreshed']} | {r['ms']:.0f} |" + (f"  <!-- {[round(t) for t in r['all_ms']]} -->" if a.show_all else ""), flush=True)


if __name__ == "__main__":
    main()
