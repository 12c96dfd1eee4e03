"""Helpers shared by the GPU parity tests: tolerance checks, margin rules for decisions, and the
comparison of the commit rule's quantities (Sec. 4.2; Algorithm 1 after the layer loop) with the oracle."""
import numpy as np

from oracle import polestar_oracle as O
from paper_2607_14107_b200 import binding as Bd
from paper_2607_14107_b200 import inputs as I

TOL = {I.DTYPE_F32: 1e-4, I.DTYPE_BF16: 2e-2}     # abs/rel tolerance on hidden states and logits


def close(a, b, tol, what=""):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    assert a.shape == b.shape, (what, a.shape, b.shape)
    err = np.abs(a - b) - tol * np.abs(b)
    assert np.isfinite(a).all(), what
    assert err.max(initial=0.0) <= tol, f"{what}: max abs err {np.abs(a - b).max():.3e} (tol {tol})"


def close_scaled(a, b, tol, what="", depth=1):
    """The same rule with the absolute part taken relative to the tensor's RMS when that exceeds one:
    |a - b| <= tol * sqrt(depth) * (max(1, rms(b)) + |b|).  For activations whose scale is well above one
    (larger initialisations, wide models), where bf16 rounding errors scale with the values; the rounding
    perturbations of successive layers are independent and add in quadrature, hence sqrt(depth) for a value
    `depth` layers deep."""
    tol = tol * max(1.0, float(depth)) ** 0.5
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    assert a.shape == b.shape, (what, a.shape, b.shape)
    assert np.isfinite(a).all(), what
    s = max(1.0, float(np.sqrt(np.mean(b * b)))) if b.size else 1.0
    err = np.abs(a - b) - tol * np.abs(b)
    assert err.max(initial=0.0) <= tol * s, f"{what}: max abs err {np.abs(a - b).max():.3e} (tol {tol}, scale {s:.2f})"


def outside_fraction(a, b, tol):
    """Share of elements outside the plain rule |a - b| <= tol + tol * |b|."""
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.mean(np.abs(a - b) > tol + tol * np.abs(b))) if a.size else 0.0


def topk_margin_ok(D, sel, tol):
    """True if every decision of the top-k cut is farther than tol from the cut value."""
    D = np.asarray(D, np.float64)
    if len(sel) == 0 or len(sel) == len(D):
        return True
    inside = D[sel].min()
    outside = np.delete(D, sel)
    outside = outside[outside > 0].max() if (outside > 0).any() else 0.0
    cut = 0.5 * (inside + outside)
    return (inside - outside) > 2 * (tol + tol * abs(cut))


def argmax_margin_ok(logits, yhat, mask_id, tol_logit):
    """True where the best non-[MASK] logit of a row beats the runner-up by more than 2 * tol_logit."""
    l = np.array(logits, np.float64, copy=True)
    l[:, mask_id] = -np.inf
    best = l[np.arange(len(yhat)), yhat].copy()
    l[np.arange(len(yhat)), yhat] = -np.inf
    return (best - l.max(axis=1)) > 2 * tol_logit


def commit_margins(info, p, tol, within):
    """Which of the oracle's commit decisions are decidable at tolerance `tol`: a row is decidable if its
    confidence is farther than tol(c) from tau_s and (within-block steps with the drift clause) its drift delta is
    farther than tol(Delta) + 2 alpha |tau_s - c| tol(c) from its threshold.  Returns (decidable [B], quota_ok)."""
    conf, masked = np.asarray(info["conf"], np.float64), np.asarray(info["masked"], bool)
    tol_c = tol * (1 + np.abs(conf))
    dec = np.abs(conf - p.tau_s) > tol_c
    if within and (p.flags & I.FLAG_DRIFT_COMMIT):
        Dl, td = np.asarray(info["Delta"], np.float64), np.asarray(info["tau_d"], np.float64)
        d_ok = np.abs(Dl - td) > tol * (1 + np.abs(Dl)) + 2 * p.alpha * np.abs(p.tau_s - conf) * tol_c
        dec &= d_ok | (conf >= p.tau_s + tol_c)          # the confidence clause already decides those rows
    dec |= ~masked
    quota_ok = bool(dec.all())
    if quota_ok:
        first = np.asarray(info["by_conf"], bool) | np.asarray(info["by_drift"], bool)
        need = info["quota"] - int(first.sum())
        rest = sorted((j for j in range(len(conf)) if masked[j] and not first[j]), key=lambda j: (-conf[j], j))
        if 0 < need < len(rest):
            a, b = conf[rest[need - 1]], conf[rest[need]]
            quota_ok = (a - b) > 2 * tol * (1 + abs(a))
    return dec, quota_ok


def check_commit_quantities(gpu, ora, infos, y_before, p, m, tol, stats):
    """After both sides committed: the GPU's Delta, tau_d, drift history and its rule's OWN decisions (taken before
    any forced decision replaced them) against the oracle's commit_rule, every sequence."""
    B = p.block
    Delta, taud = gpu.read(Bd.READ_DRIFT_DELTA), gpu.read(Bd.READ_TAU_D)
    ring, cnt = gpu.read(Bd.READ_THETA), gpu.read(Bd.READ_THETA_COUNT)
    own, conf_g = gpu.read(Bd.READ_OWN_COMMIT), gpu.read(Bd.READ_CONF)
    suf = gpu.read(Bd.READ_SUFFIX)
    for s, info in enumerate(infos):
        seq = ora.seqs[s]
        within = bool(seq.within)
        conf = np.asarray(info["conf"], np.float64)
        tol_c = tol * (1 + np.abs(conf))
        # tau_d = alpha (tau_s - c)^2 inherits the confidence's tolerance through its derivative
        td_tol = 2 * p.alpha * np.abs(p.tau_s - conf) * tol_c + p.alpha * tol_c ** 2 + tol * np.abs(info["tau_d"]) + 1e-7
        assert (np.abs(taud[s] - info["tau_d"]) <= td_tol).all(), f"tau_d seq {s}"
        if within:
            close(Delta[s], info["Delta"], tol, f"Delta seq {s}")
            stats["delta_rows"] += B
        # drift history: the oracle's list, oldest first, against the ring
        n_h = min(int(cnt[s]), p.hist)
        assert n_h == len(seq.theta), (n_h, len(seq.theta))
        for u in range(n_h):
            close(ring[s, (int(cnt[s]) - n_h + u) % p.hist], seq.theta[u], tol, f"theta[{u}] seq {s}")
        stats["theta_vectors"] += n_h
        # the rule's own decisions on decidable rows
        dec, quota_ok = commit_margins(info, p, tol, within)
        masked = np.asarray(info["masked"], bool)
        rows = dec & masked
        g_conf, g_drift, g_quota = (own[s] & 2) != 0, (own[s] & 4) != 0, (own[s] & 8) != 0
        assert np.array_equal(g_conf[rows], np.asarray(info["by_conf"], bool)[rows]), f"by_conf seq {s}"
        assert np.array_equal(g_drift[rows], np.asarray(info["by_drift"], bool)[rows]), f"by_drift seq {s}"
        assert not (own[s][~masked] & 1).any()
        stats["own_by_conf"] += int((g_conf & rows).sum())
        stats["own_by_drift"] += int((g_drift & rows).sum())
        if quota_ok:
            assert np.array_equal(g_quota, np.asarray(info["by_quota"], bool)), f"by_quota seq {s}"
            stats["own_by_quota"] += int(g_quota.sum())
        # suffix rows: eligibility comes from the last layer's selection, the decision from confidence alone
        if within and (p.flags & I.FLAG_SUFFIX_COMMIT):
            elig = sorted(int(w) for w in seq.suffix_rows if y_before[s, seq.win[w]] == m.mask_id)
            assert sorted(np.nonzero(suf[s] & 1)[0].tolist()) == elig, f"suffix eligibility seq {s}"
            if "suffix_conf" in info:
                for t, w in enumerate(seq.suffix_rows):
                    if int(w) not in elig:
                        continue
                    sc = float(info["suffix_conf"][t])
                    if abs(sc - p.tau_suffix) > tol * (1 + abs(sc)):
                        assert bool(suf[s, w] & 4) == (sc >= p.tau_suffix), f"suffix decision seq {s} row {w}"
                        stats["own_suffix"] += int(bool(suf[s, w] & 4))
            stats["suffix_eligible"] += len(elig)


def new_stats():
    return dict(delta_rows=0, theta_vectors=0, own_by_conf=0, own_by_drift=0, own_by_quota=0, own_suffix=0,
                suffix_eligible=0)
