"""Single-kernel timings through the C ABI: the refresh micro-benchmark (select -> gathered QKV
refresh -> scatter, 4096 cache positions x 4096 hidden, refresh fraction 1..100 %, batch 1 and 8),
the hidden-delta stream, the drift kernel at the 8B shapes and the confidence kernel.

    python -m paper_2607_14107_b200.kernel_bench [--quick] [--only select,refresh,...]

Every line printed is one JSON record: time per call (CUDA events around a loop over rotating
buffer copies, so that no call finds its inputs in L2), algorithmic bytes / flops, and the
fractions of the measured HBM and bf16 peaks (MEASURED_PEAKS.json, else the machine's fallback).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys

import torch

from . import binding as Bd
from . import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return d["hbm_gbs"], d["bf16_tflops_sustained"], "measured"
    return 6650.0, 1590.0, "fallback"


def timed(fn, n_iter, warmup=3):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n_iter):
        fn(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / n_iter      # microseconds per call


def emit(name, us, bytes_, flops, extra):
    hbm, tf, src = peaks()
    rec = {"kernel": name, "us": round(us, 2), "GBps": round(bytes_ / us / 1e3, 1), "hbm_frac": round(bytes_ / us / 1e3 / hbm, 3),
           "TFLOPs": round(flops / us / 1e6, 1), "tensor_frac": round(flops / us / 1e6 / tf, 3), "peaks": src}
    rec.update(extra)
    print(json.dumps(rec), flush=True)


def bench_select(quick):
    for bs in (1, 8):
        _, drift = I.make_refresh_inputs(1, 4096, 8)
        drift = drift.repeat(bs, 1).cuda() * torch.linspace(1.0, 2.0, bs, device="cuda")[:, None]
        idx = torch.zeros((bs, 4096), dtype=torch.int32, device="cuda")
        cnt = torch.zeros(bs, dtype=torch.int32, device="cuda")
        for frac in (0.01, 0.25, 1.0):
            k = I.refresh_count(frac)
            us = timed(lambda i: Bd.polestar_k_select(drift, I.SELECT_TOPK_COUNT, k, 0.0, 0.0, idx, cnt), 50)
            emit("select", us, bs * 4096 * 4 + bs * k * 4, 0, {"batch": bs, "frac": frac, "k": k})


def bench_refresh(quick):
    d, nh, nkv, dh, P = 4096, 32, 32, 128, 4096
    m = I.ModelCfg(1, d, nh, nkv, dh, 64, 1024, I.DTYPE_BF16, 1e-5, 500000.0)
    n_w = 4                                        # rotating weight copies: 4 x 100 MB > L2
    wq = []
    for c in range(n_w):
        w = I.make_weights(m, seed=10 + c, device="cuda", with_globals=False)["layers"][0]
        perm = Bd.rope_interleave_index(dh).cuda()
        q = w["wq"].view(nh, dh, d)[:, perm].reshape(nh * dh, d)
        k = w["wk"].view(nkv, dh, d)[:, perm].reshape(nkv * dh, d)
        wq.append(Bd.tile_major(torch.cat([q, k, w["wv"]], 0)))
        del w
    norm = torch.ones(d, device="cuda")
    for bs in (1, 8):
        for clustered in (False, True):
            h, drift = I.make_refresh_inputs(bs, P, d, clustered=clustered, device="cuda")
            kc = torch.zeros((bs, P, nkv * dh), dtype=torch.bfloat16, device="cuda")
            vc = torch.zeros_like(kc)
            full_idx = torch.zeros((bs, P), dtype=torch.int32, device="cuda")
            cnt = torch.zeros(bs, dtype=torch.int32, device="cuda")
            fracs = (0.01, 0.25, 1.0) if quick else (0.01, 0.05, 0.10, 0.25, 0.50, 1.0)
            if clustered:
                fracs = (0.25,)
            for frac in fracs:
                k = I.refresh_count(frac)
                idx = torch.zeros((bs, k), dtype=torch.int32, device="cuda")
                scratch = torch.empty(Bd.polestar_k_refresh_scratch_bytes(bs, k, d, nh, nkv, dh) + 1024,
                                      dtype=torch.uint8, device="cuda")
                scratch = scratch[(-scratch.data_ptr()) % 1024:]

                def chain(i):
                    Bd.polestar_k_select(drift, I.SELECT_TOPK_COUNT, k, 0.0, 0.0, full_idx, cnt)
                    idx.copy_(full_idx[:, :k])
                    Bd.polestar_k_refresh(h, idx, cnt, wq[i % n_w], norm, kc, vc, None, k, nh, nkv, dh, 1e-5, 500000.0, scratch)

                def only_refresh(i):
                    Bd.polestar_k_refresh(h, idx, cnt, wq[i % n_w], norm, kc, vc, None, k, nh, nkv, dh, 1e-5, 500000.0, scratch)

                M = bs * k
                nq = (nh + 2 * nkv) * dh
                by = nq * d * 2 + M * d * 2 + M * 2 * nkv * dh * 2
                fl = 2.0 * M * nq * d
                us_chain = timed(chain, 8 if M > 8192 else 20)
                us_ref = timed(only_refresh, 8 if M > 8192 else 20)
                emit("refresh (gather+norm, QKV GEMM, RoPE, scatter)", us_ref, by, fl,
                     {"batch": bs, "frac": frac, "rows": M, "clustered": clustered,
                      "chain_us_with_select": round(us_chain, 2),
                      "bound": "hbm" if M <= 215 else "tensor"})
            del h, kc, vc


def bench_hidden_delta(quick):
    for bs in (1, 8):
        rows, d = bs * 4096, 4096
        n = 4 if bs == 1 else 2
        a = [I.normal_tensor(I.tensor_key(3, c, I.T_HCACHE), (rows, d), 1.0, torch.bfloat16, "cuda") for c in range(n)]
        b = [x.clone() for x in a]
        out = torch.empty(rows, device="cuda")
        us = timed(lambda i: Bd.polestar_k_hidden_delta(a[i % n], b[i % n], out), 20)
        emit("hidden_delta", us, 2 * rows * d * 2, 0, {"batch": bs, "rows": rows})


def bench_drift(quick):
    # window rows of one layer of the 8B shape (W = 96, N = 512) and of the long config (W = 192, N = 2048);
    # --quick: the 8B-shape cases only (a small case for profiler captures)
    for name, R, N, nh, n_copy in (("c2", 96, 512, 32, 24), ("c2 window+block", 128, 512, 32, 24), ("c2 block entry", 512, 512, 32, 8),
                                   ("c4 per sequence", 192, 2048, 32, 4), ("c4 block entry", 2048, 2048, 32, 2)):
        if quick and not name.startswith("c2"):
            continue
        dh = 128
        q = [I.normal_tensor(I.tensor_key(5, c, 1), (R, nh * dh), 1.0, torch.bfloat16, "cuda") for c in range(n_copy)]
        k = [I.normal_tensor(I.tensor_key(5, c, 2), (N, nh * dh), 1.0, torch.bfloat16, "cuda") for c in range(n_copy)]
        v = [I.normal_tensor(I.tensor_key(5, c, 3), (N, nh * dh), 1.0, torch.bfloat16, "cuda") for c in range(n_copy)]
        prev = [torch.full((R, nh, N), -math.log(N), device="cuda") for _ in range(n_copy)]
        lse = [torch.zeros((R, nh), device="cuda") for _ in range(n_copy)]
        kl = torch.empty((R, nh), device="cuda")
        out = torch.empty((R, nh * dh), dtype=torch.bfloat16, device="cuda")
        us = timed(lambda i: Bd.polestar_k_attention(q[i % n_copy], k[i % n_copy], v[i % n_copy], prev[i % n_copy], lse[i % n_copy], kl, out,
                                                     nh, nh, dh), 48)
        by = 2 * N * nh * dh * 2 + 2 * R * nh * N * 4 + 2 * R * nh * dh * 2
        emit("drift+attention rows", us, by, 4.0 * R * N * nh * dh, {"shape": name, "rows": R, "keys": N})
        us = timed(lambda i: Bd.polestar_k_attention(q[i % n_copy], k[i % n_copy], v[i % n_copy], None, None, None, out,
                                                     nh, nh, dh), 48)
        emit("attention rows (no drift)", us, 2 * N * nh * dh * 2 + 2 * R * nh * dh * 2, 4.0 * R * N * nh * dh,
             {"shape": name, "rows": R, "keys": N})


def bench_confidence(quick):
    V = 126464
    for rows in (32, 512):
        n = 8 if rows == 32 else 2
        lg = [I.normal_tensor(I.tensor_key(7, c, 1), (rows, V), 3.0, torch.float32, "cuda") for c in range(n)]
        yh = torch.zeros(rows, dtype=torch.int32, device="cuda")
        cf = torch.zeros(rows, device="cuda")
        sc = torch.empty(rows * 512, dtype=torch.uint8, device="cuda")
        us = timed(lambda i: Bd.polestar_k_confidence(lg[i % n], V - 1, yh, cf, sc), 30)
        emit("confidence", us, rows * V * 4, 0, {"rows": rows, "vocab": V})


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--only", default="select,refresh,hidden_delta,drift,confidence")
    a = ap.parse_args()
    fns = {"select": bench_select, "refresh": bench_refresh, "hidden_delta": bench_hidden_delta, "drift": bench_drift,
           "confidence": bench_confidence}
    for name in a.only.split(","):
        fns[name](a.quick)


if __name__ == "__main__":
    main()
