"""Parity at the benchmark's sizes: the LLaDA-8B shape in the launch configuration bench.py times.

The oracle cannot run 32 layers of this width in reasonable time, so
  * at reduced depth (2 layers, full widths, full vocabulary, full sequence) every logit, hidden
    state, drift value and selected index of an entry forward and of a refresh step is compared
    with the oracle;
  * at full depth the library is checked against itself through a property that holds at any
    size: with every window row refreshed at every step the cached decode must reproduce the
    full-recompute decode (Sec. 4.1 / Sec. 3.1), plus the invariants of drift, selection and commit.
"""
import dataclasses
import re

import numpy as np
import pytest
import torch

from oracle import polestar_oracle as O
from paper_2607_14107_b200 import binding as Bd
from paper_2607_14107_b200 import inputs as I

from parity import check_commit_quantities, new_stats, outside_fraction
from test_gpu_decode import impose_codes

pytestmark = pytest.mark.gpu
TOL = 2e-2
# Largest share of elements of any compared tensor that may fall outside the plain abs/rel 2e-2 rule (they are
# inside the RMS-scaled rule of close()); the measured shares are printed at the end of the module (-s).
OUTSIDE_MAX = 5e-2
OUTSIDE = {}


@pytest.fixture(scope="module", autouse=True)
def _report_outside_fraction():
    yield
    worst = sorted(OUTSIDE.items(), key=lambda kv: -kv[1])[:8]
    print("\nshare of elements outside the plain abs/rel 2e-2 rule (worst tensors):", worst)


def close(a, b, tol, what="", scale=1.0, depth=1, bound=OUTSIDE_MAX):
    """|a - b| <= tol * sqrt(depth) * (s + |b|), s = max(1, rms(b)).

    At these widths hidden states have an RMS of ~2 (14 after 32 layers) and dot products run over
    4096..12288 bf16 terms, so the absolute part of the tolerance is taken relative to the tensor's own
    scale (the plain 2e-2 for tensors of RMS <= 1).  The bf16 rounding perturbations of successive layers
    are independent and add in quadrature, hence the sqrt(depth) for values `depth` layers deep."""
    tol = tol * max(1.0, float(depth)) ** 0.5
    a, b = np.asarray(a, np.float64) / scale, np.asarray(b, np.float64) / scale
    assert a.shape == b.shape, (what, a.shape, b.shape)
    assert np.isfinite(a).all(), what
    s = max(1.0, float(np.sqrt(np.mean(b * b)))) if b.size else 1.0
    err = np.abs(a - b) - tol * np.abs(b)
    assert err.max(initial=0.0) <= tol * s, f"{what}: max abs err {np.abs(a - b).max():.3e} (tol {tol}, scale {s:.2f})"
    # what the scaled tolerance hides: the share of elements outside the plain rule |a - b| <= 2e-2 (1 + |b|)
    frac = outside_fraction(a, b, TOL)
    key = re.sub(r"(step|seq) \d+ ?", "", what)
    OUTSIDE[key] = max(frac, OUTSIDE.get(key, 0.0))
    if bound is not None:       # (None: the 32-layer self-consistency check, where the share is only reported)
        assert frac <= bound, f"{what}: {frac:.2e} of the elements outside the plain abs/rel {TOL} rule"


def forced_commit(gpu, ora, infos, p, m=None, y_before=None, stats=None):
    forced = np.full((p.batch, p.block + gpu.W_max), -1, np.int32)
    ftok = np.zeros_like(forced)
    for s, i in enumerate(infos):
        pos = [int(ora.seqs[s].act[j]) for j in np.nonzero(i["commit"] & i["masked"])[0]] + i["suffix_committed"]
        forced[s, :len(pos)] = pos
        ftok[s, :len(pos)] = ora.tokens()[s, pos]
    gpu.force_commit(forced, ftok)
    ci = gpu.commit()
    if stats is not None:
        check_commit_quantities(gpu, ora, infos, y_before, p, m, TOL, stats)
    return ci


def compare_step(gpu, ora, m, p, step):
    L = m.n_layers
    for s in range(p.batch):
        tr = ora.seqs[s].trace
        for l in range(L + 1):
            close(gpu.read(Bd.READ_HIDDEN, l)[s], tr["x_act"][l], TOL, f"step {step} seq {s} hidden l{l}", depth=l)
        # (the LM head is one more normalisation + projection on top of the L layers; measured at the 8B widths:
        # RMS error 0.0046, so the largest of 8.1 million logits sits at ~5.5 sigma = 0.025)
        close(gpu.read(Bd.READ_LOGITS)[s], tr["logits"], TOL, f"step {step} seq {s} logits", p.logit_scale, depth=L + 1)
        W = len(ora.seqs[s].win)
        if tr["kind"] == "within":
            close(gpu.read(Bd.READ_DELTA)[s], tr["delta"], TOL, f"step {step} delta")
            if tr["refresh"]:
                for l in range(L):
                    nD = len(tr["D"][l])            # window rows, or clusters (centroid proxies)
                    close(gpu.read(Bd.READ_DRIFT, l)[s, :nD], tr["D"][l], TOL, f"step {step} drift l{l}")
                    n = gpu.read(Bd.READ_SEL_COUNT, l)[s]
                    assert list(gpu.read(Bd.READ_SEL_IDX, l)[s, :n]) == list(tr["sel"][l])
        for l in range(L):
            Kc = gpu.read(Bd.READ_KCACHE, l)[s].reshape(ora.seqs[s].Kc[l].shape)
            Vc = gpu.read(Bd.READ_VCACHE, l)[s].reshape(ora.seqs[s].Vc[l].shape)
            # K / V of layer l: the layer's input (l layers deep) through one more normalisation + projection
            close(Kc, ora.seqs[s].Kc[l], TOL, f"step {step} K l{l}", depth=l + 1)
            close(Vc, ora.seqs[s].Vc[l], TOL, f"step {step} V l{l}", depth=l + 1)
            close(gpu.read(Bd.READ_HCACHE, l)[s, :W], ora.seqs[s].Hc[l], TOL, f"step {step} H l{l}", depth=l)


def run_reduced_depth(m, p, n_within):
    w = I.make_weights(m, seed=0, device="cuda")
    packed = Bd.pack_weights(m, w)
    wn = I.weights_to_numpy(w)
    del w
    prompt = I.make_prompt(m, p).numpy()
    gpu = Bd.Polestar(m, packed, p, prompt)
    ora = O.PolestarOracle(m, wn, p, prompt)
    ora.step()
    cluster = p.select_mode == I.SELECT_CLUSTER_TOPK
    quant = bool(p.flags & I.FLAG_NVFP4_HCACHE)
    if cluster:
        for s in range(p.batch):        # the library's own K-means of the first block entry (inside polestar_init)
            for l in range(m.n_layers):
                W = len(ora.seqs[s].win)
                assert np.array_equal(gpu.read(Bd.READ_LABELS, l)[s, :W], ora.seqs[s].labels[l]), f"labels l{l}"
    if quant:
        impose_codes(gpu, ora, p, m)    # a value next to a code boundary may have fallen the other way: same codes from here on
    compare_step(gpu, ora, m, p, 0)
    kinds = [ora.seqs[0].trace["kind"]]
    stats = new_stats()
    for step in range(1, n_within + 1):
        y_before = ora.tokens().copy()
        forced_commit(gpu, ora, ora.commit(), p, m, y_before, stats)
        assert np.array_equal(gpu.tokens(), ora.tokens())
        ora.step()
        tr = ora.seqs[0].trace
        if cluster and tr["kind"] != "within":
            for l in range(m.n_layers):
                lab = np.zeros((p.batch, len(ora.seqs[0].labels[l])), np.int32)
                for s in range(p.batch):
                    lab[s] = ora.seqs[s].labels[l]
                gpu.force_labels(l, lab)
        if quant:
            impose_codes(gpu, ora, p, m)
        if tr["kind"] == "within" and tr["refresh"]:
            for l in range(m.n_layers):
                sel = np.full((p.batch, gpu.W_max), -1, np.int32)
                for s in range(p.batch):
                    sl = ora.seqs[s].trace["sel"][l]
                    sel[s, :len(sl)] = sl
                gpu.force_select(l, sel)
        gpu.step()
        compare_step(gpu, ora, m, p, step)
        kinds.append(tr["kind"] + ("_refresh" if tr["kind"] == "within" and tr["refresh"] else ""))
    gpu.destroy()
    return kinds


def test_c2_shape_reduced_depth_matches_oracle():
    m, p = I.config("c2")
    m = I.reduced_depth(m, 2)
    p = dataclasses.replace(p, tau_upd=-1, flags=p.flags | I.FLAG_KEEP_HIDDEN)
    run_reduced_depth(m, p, n_within=1)


def test_c3_widths_gqa_batch_matches_oracle():
    # Dream-7B widths (28 query heads on 4 kv heads, d 3584, FFN 18944, vocab 152064), batch 4 as in the
    # workload, short sequences
    m, _ = I.config("c3")
    m = I.reduced_depth(m, 1)
    p = I.Params(batch=4, prompt_len=64, gen_len=64, block=32, max_steps=64, tau_upd=-1,
                 flags=I.FLAG_DEFAULT | I.FLAG_KEEP_HIDDEN)
    run_reduced_depth(m, p, n_within=2)


def test_c4_shape_reduced_depth_matches_oracle():
    # The long-generation workload's shape at depth 1: LLaDA-8B widths and vocabulary, 1024 + 1024 positions,
    # block 64 (window 192), batch 2.  With 3 steps per block and tau_upd = 25 the first forwards are: a
    # full-sequence entry (2048 rows per sequence: multi-token-tile GEMMs, the 64-row attention kernel with
    # recorded rows), a plain step, a refresh step (192 window rows per sequence through drift, select and the
    # sparse forward) and the window entry of the next block.
    m, p = I.config("c4")
    m = I.reduced_depth(m, 1)
    p = dataclasses.replace(p, batch=2, max_steps=48, tau_upd=25, flags=p.flags | I.FLAG_KEEP_HIDDEN)
    kinds = run_reduced_depth(m, p, n_within=3)
    assert kinds == ["entry_full", "within", "within_refresh", "entry_window"], kinds


def test_c2_shape_centroid_proxies_and_nvfp4_cache_match_oracle():
    # Sec. 4.1 default policy at the LLaDA-8B widths, depth 2: K-means over 4096-wide rows (the library's own labels
    # against the oracle's at the first entry), proxy rows through the staging kernel and the attention kernels, cluster
    # top-k, the hidden cache as NVFP4 residuals (the library's own codes replaced by the oracle's after every encode)
    m, p = I.config("c2")
    m = I.reduced_depth(m, 2)
    p = dataclasses.replace(p, tau_upd=-1, select_mode=I.SELECT_CLUSTER_TOPK,
                            flags=p.flags | I.FLAG_KEEP_HIDDEN | I.FLAG_NVFP4_HCACHE)
    kinds = run_reduced_depth(m, p, n_within=2)
    assert kinds == ["entry_full", "within_refresh", "within_refresh"], kinds


def test_c3_widths_centroid_proxies_and_nvfp4_cache_match_oracle():
    # the same policy at the Dream-7B widths (d 3584 = 28 x 128: not a power of two; GQA 28 / 4), batch 2, short
    # sequences: K-means, proxy staging and the codec with 3584-wide rows, proxy rows of two sequences in one forward
    m, _ = I.config("c3")
    m = I.reduced_depth(m, 1)
    p = I.Params(batch=2, prompt_len=64, gen_len=64, block=32, max_steps=64, tau_upd=-1, select_mode=I.SELECT_CLUSTER_TOPK,
                 n_clusters=6, cluster_k=3, flags=I.FLAG_DEFAULT | I.FLAG_KEEP_HIDDEN | I.FLAG_NVFP4_HCACHE)
    kinds = run_reduced_depth(m, p, n_within=2)
    assert kinds == ["entry_full", "within_refresh", "within_refresh"], kinds


def test_c6_short_generation_shape_matches_oracle():
    # Sec. 5.2 (hard-to-parallelise tasks): generation length 32 with block 8 at the LLaDA-8B widths, depth 2: a
    # window of 16 + 8 rows, eight active rows per step, a block entry every few forwards
    m, p = I.config("c6")
    m = I.reduced_depth(m, 2)
    p = dataclasses.replace(p, tau_upd=-1, flags=p.flags | I.FLAG_KEEP_HIDDEN)
    kinds = run_reduced_depth(m, p, n_within=9)
    assert kinds[0] == "entry_full" and "entry_window" in kinds and "within_refresh" in kinds, kinds


@pytest.fixture(scope="module")
def c2_full():
    m, p = I.config("c2")
    packed = Bd.make_packed_weights(m, seed=0, device="cuda")
    return m, p, packed


@pytest.mark.parametrize("mode", ["every row", "every cluster"])
def test_c2_full_depth_full_refresh_equals_nocache(c2_full, mode):
    # Sec. 4.1 / Sec. 3.1: refreshing everything (all window rows; or, with centroid proxies, all eight clusters of a
    # window that spans the sequence) reproduces decoding without a cache, here over the full 32 layers
    m, p, packed = c2_full
    if mode == "every cluster":          # (the cluster mode takes windows of up to 256 rows: a 128 + 128 sequence)
        p = dataclasses.replace(p, prompt_len=128, gen_len=128)
    prompt = I.make_prompt(m, p).numpy()
    sel = dict(select_mode=I.SELECT_ALL) if mode == "every row" else dict(select_mode=I.SELECT_CLUSTER_TOPK, n_clusters=8, cluster_k=8)
    pa = dataclasses.replace(p, tau_upd=-1, win_prefix_blocks=16, win_suffix_blocks=16,
                             flags=(I.FLAG_DEFAULT | I.FLAG_KEEP_HIDDEN) & ~I.FLAG_SUFFIX_COMMIT, max_steps=64, **sel)
    pb = dataclasses.replace(pa, flags=pa.flags | I.FLAG_NOCACHE)
    a, b = Bd.Polestar(m, packed, pa, prompt), Bd.Polestar(m, packed, pb, prompt)
    for step in range(5):
        if step:
            a.step(); b.step()
        ha, hb = a.read(Bd.READ_HIDDEN, m.n_layers), b.read(Bd.READ_HIDDEN, m.n_layers)
        close(a.read(Bd.READ_HIDDEN, 1), b.read(Bd.READ_HIDDEN, 1), TOL, f"step {step} hidden after layer 0")
        close(ha, hb, TOL, f"step {step} final hidden (32 layers, self-consistency)", depth=m.n_layers, bound=None)
        close(a.read(Bd.READ_LOGITS), b.read(Bd.READ_LOGITS), TOL, f"step {step} logits (32 layers, self-consistency)",
              depth=m.n_layers, bound=None)
        if step:
            close(a.read(Bd.READ_DELTA), b.read(Bd.READ_DELTA), TOL, f"step {step} delta", depth=m.n_layers)
        # keep the two decoders on one trajectory: b commits what a commits
        a.commit()
        flags = a.read(Bd.READ_COMMIT)[0]
        pos = [p.prompt_len + j for j in np.nonzero(flags & 1)[0]]
        forced = np.full((1, p.block + b.W_max), -1, np.int32)
        forced[0, :len(pos)] = pos
        ftok = np.zeros_like(forced)
        ftok[0, :len(pos)] = a.tokens()[0, pos]
        b.force_commit(forced, ftok)
        b.commit()
        assert np.array_equal(a.tokens(), b.tokens())
    a.destroy(); b.destroy()


def test_c2_full_depth_default_mode_invariants(c2_full):
    m, p, packed = c2_full
    prompt = I.make_prompt(m, p).numpy()
    p = dataclasses.replace(p, max_steps=64, logit_scale=30.0)      # quota 4: refresh after every step
    gpu = Bd.Polestar(m, packed, p, prompt)
    prev = gpu.tokens().copy()
    n_refresh = 0
    for step in range(10):
        if step:
            info = gpu.step()
            if info.kind == 2:
                assert (gpu.read(Bd.READ_DELTA) > -1e-4).all()          # KL >= 0
            if info.kind == 2 and info.n_refreshing:
                n_refresh += 1
                for l in (0, m.n_layers // 2, m.n_layers - 1):
                    D = gpu.read(Bd.READ_DRIFT, l)[0, :96]
                    n = int(gpu.read(Bd.READ_SEL_COUNT, l)[0])
                    idx = gpu.read(Bd.READ_SEL_IDX, l)[0, :n]
                    assert (D > -1e-4).all() and np.isfinite(D).all()
                    assert n == min(24, int((D > 0).sum()))               # k = floor(0.25 * 96 + 1/2)
                    assert list(idx) == sorted(idx)
                    if n:                                                   # the selected rows are the k largest
                        rest = np.delete(D, idx)
                        assert D[idx].min() >= rest.max() - 1e-6
        conf = gpu.read(Bd.READ_CONF)
        assert ((conf > 0) & (conf <= 1 + 1e-5)).all()
        ci = gpu.commit()
        cur = gpu.tokens()
        was = prev != m.mask_id
        assert np.array_equal(cur[was], prev[was])                          # committed tokens never change
        assert (cur != prev).sum() == ci.n_committed and ci.n_committed >= 1
        assert ci.n_committed == ci.n_by_conf + ci.n_by_drift + ci.n_by_quota + ci.n_suffix
        prev = cur.copy()
    assert n_refresh >= 3
    gpu.destroy()


def test_c2_full_depth_decode_is_bitwise_reproducible(c2_full, monkeypatch):
    # with the ordered reduction (POLESTAR_GEMM_ACCUMULATE=0) split tiles are reduced in a fixed order and no kernel
    # uses floating-point atomics: two runs of the same decode give the same bits (also a guard against races in
    # the partial-tile exchange)
    monkeypatch.setenv("POLESTAR_GEMM_ACCUMULATE", "0")
    m, p, packed = c2_full
    prompt = I.make_prompt(m, p).numpy()
    p = dataclasses.replace(p, max_steps=64, logit_scale=30.0, tau_upd=-1)
    runs = []
    for _ in range(2):
        gpu = Bd.Polestar(m, packed, p, prompt)
        trace = []
        for step in range(6):
            if step:
                gpu.step()
            trace.append((gpu.read(Bd.READ_LOGITS).copy(), gpu.read(Bd.READ_CONF).copy(), gpu.read(Bd.READ_DELTA).copy()))
            gpu.commit()
            trace.append((gpu.tokens().copy(),))
        runs.append(trace)
        gpu.destroy()
    for a, b in zip(*runs):
        for x, y in zip(a, b):
            assert np.array_equal(x, y)


def test_c2_chained_projections_equal_separate_launches(monkeypatch):
    # the persistent O -> RMSNorm -> gate/up -> down kernel does the arithmetic of the four separate launches in the
    # same order: same bits (2 layers at full widths, an entry forward, plain and refresh steps)
    m, p = I.config("c2")
    m = I.reduced_depth(m, 2)
    p = dataclasses.replace(p, max_steps=64, logit_scale=30.0, flags=p.flags | I.FLAG_KEEP_HIDDEN)
    packed = Bd.make_packed_weights(m, seed=0, device="cuda")
    prompt = I.make_prompt(m, p).numpy()
    runs = []
    monkeypatch.setenv("POLESTAR_GEMM_ACCUMULATE", "0")
    for chain in ("1", "0"):
        monkeypatch.setenv("POLESTAR_CHAIN", chain)
        gpu = Bd.Polestar(m, packed, p, prompt)
        trace = []
        for step in range(8):
            if step:
                gpu.step()
            trace.append((gpu.read(Bd.READ_LOGITS).copy(), gpu.read(Bd.READ_HIDDEN, m.n_layers).copy(),
                          gpu.read(Bd.READ_KCACHE, 1).copy(), gpu.read(Bd.READ_HCACHE, 1).copy()))
            gpu.commit()
            trace.append((gpu.tokens().copy(),))
        runs.append(trace)
        gpu.destroy()
    for a, b in zip(*runs):
        for x, y in zip(a, b):
            assert np.array_equal(x, y)


def test_c2_accumulating_projections_match_the_ordered_reduction(monkeypatch):
    # O / down projections that add their parts onto the residual rows in L2 (arrival order) against the ordered
    # reduction of published partial tiles: same numbers up to the rounding of a different summation order
    m, p = I.config("c2")
    m = I.reduced_depth(m, 2)
    p = dataclasses.replace(p, max_steps=64, logit_scale=30.0, flags=p.flags | I.FLAG_KEEP_HIDDEN)
    packed = Bd.make_packed_weights(m, seed=0, device="cuda")
    prompt = I.make_prompt(m, p).numpy()
    runs, committed = [], []
    for acc in ("1", "0"):
        monkeypatch.setenv("POLESTAR_GEMM_ACCUMULATE", acc)
        gpu = Bd.Polestar(m, packed, p, prompt)
        trace = []
        for step in range(8):
            if step:
                gpu.step()
            trace.append((gpu.read(Bd.READ_LOGITS).copy() / p.logit_scale, gpu.read(Bd.READ_HIDDEN, m.n_layers).copy(),
                          gpu.read(Bd.READ_KCACHE, 1).copy().astype(np.float32), gpu.read(Bd.READ_HCACHE, 1).copy()))
            before = gpu.tokens().copy()
            if acc == "0":          # the second run replays the first run's commits (a near-tie may fall either way)
                after = committed[step]
                forced = np.full((p.batch, p.block + gpu.W_max), -1, np.int32)
                ftok = np.zeros_like(forced)
                pos = np.nonzero(after[0] != before[0])[0]
                forced[0, :len(pos)] = pos
                ftok[0, :len(pos)] = after[0][pos]
                gpu.force_commit(forced, ftok)
            gpu.commit()
            if acc == "1":
                committed.append(gpu.tokens().copy())
            else:
                assert np.array_equal(gpu.tokens(), committed[step])
        runs.append(trace)
        gpu.destroy()
    worst = 0.0
    for a, b in zip(*runs):
        for x, y in zip(a, b):
            x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
            worst = max(worst, float(np.abs(x - y).max() / max(1.0, np.sqrt(np.mean(y * y)))))
    # fp32 sums in another order differ in the last places; where that flips the bf16 rounding of an operand of the
    # next projection the difference grows to bf16 size: the bound is the oracle-parity rule for values L + 1 = 3
    # projections deep, TOL * sqrt(3) relative to the tensor's RMS (measured: 0.024)
    assert worst < TOL * 3 ** 0.5, worst
