"""Pins for the CPU oracle's building blocks: library special cases, closed forms,
and the theory appendix's propositions used as invariants (no GPU needed)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import polestar_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def _read(name):
    rows = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append(line)
    return rows


# ---------------------------------------------------------------- storage rounding
def test_bf16_round_matches_library_cast():
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, 1e-40]])
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.bf16_round(x), ref)


# ---------------------------------------------------------------- model pieces
def test_rmsnorm_silu_match_torch():
    x = rng.standard_normal((7, 48))
    g = rng.standard_normal(48)
    ref = torch.nn.functional.rms_norm(torch.tensor(x), (48,), torch.tensor(g), eps=1e-5).numpy()
    assert np.allclose(O.rmsnorm(x, g, 1e-5), ref, rtol=1e-13, atol=1e-13)
    assert np.allclose(O.silu(x), torch.nn.functional.silu(torch.tensor(x)).numpy(), rtol=1e-13)


def test_rope_is_a_rotation_by_complex_multiplication():
    R, H, dh, theta = 5, 3, 16, 10000.0
    x = rng.standard_normal((R, H, dh))
    pos = np.array([0, 1, 7, 100, 4095])
    y = O.rope(x, pos, theta)
    half = dh // 2
    z = x[..., :half] + 1j * x[..., half:]
    ang = pos[:, None] * theta ** (-2.0 * np.arange(half) / dh)[None, :]
    zr = z * np.exp(1j * ang)[:, None, :]
    assert np.allclose(y[..., :half], zr.real, atol=1e-12)
    assert np.allclose(y[..., half:], zr.imag, atol=1e-12)
    assert np.array_equal(y[0], x[0])                       # position 0: identity
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))


def test_rope_scores_depend_on_relative_position_only():
    dh, theta = 32, 500000.0
    q = rng.standard_normal((1, 1, dh))
    k = rng.standard_normal((1, 1, dh))
    a = (O.rope(q, [10], theta) * O.rope(k, [3], theta)).sum()
    b = (O.rope(q, [1010], theta) * O.rope(k, [1003], theta)).sum()
    assert abs(a - b) < 1e-9


def test_linear_rowwise_equals_matmul():
    x, w = rng.standard_normal((6, 20)), rng.standard_normal((9, 20))
    assert np.allclose(O.linear(x, w, True), x @ w.T, atol=1e-13)
    assert np.allclose(O.linear(x, w, False), x @ w.T, atol=1e-13)


@pytest.mark.parametrize("nh,nkv", [(4, 4), (8, 2), (7, 1)])
def test_attention_matches_noncausal_sdpa(nh, nkv):
    R, N, dh = 5, 37, 16
    q = rng.standard_normal((R, nh, dh))
    K = rng.standard_normal((N, nkv, dh))
    V = rng.standard_normal((N, nkv, dh))
    for rowwise in (False, True):
        logp = O.attn_logp_rows(q, K, rowwise)
        out = O.attn_out_rows(logp, V, rowwise=rowwise)
        rep = nh // nkv
        tq = torch.tensor(q).permute(1, 0, 2)[None]                       # [1, nh, R, dh]
        tk = torch.tensor(K).permute(1, 0, 2).repeat_interleave(rep, 0)[None]
        tv = torch.tensor(V).permute(1, 0, 2).repeat_interleave(rep, 0)[None]
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=False)
        ref = ref[0].permute(1, 0, 2).reshape(R, nh * dh).numpy()
        assert np.allclose(out, ref, rtol=1e-10, atol=1e-12)
        assert np.allclose(np.exp(logp).sum(-1), 1.0, atol=1e-12)


def test_attention_transposed_operand_would_fail():
    # a q/k swap or a missing 1/sqrt(dh) changes the distribution: check one row by hand
    q = np.array([[[1.0, 2.0, 0.0, -1.0]]])
    K = np.array([[[1.0, 0.0, 0.0, 0.0]], [[0.0, 1.0, 0.0, 0.0]], [[0.0, 0.0, 0.0, 1.0]]])
    s = np.array([1.0, 2.0, -1.0]) / 2.0
    ref = s - np.log(np.exp(s).sum())
    assert np.allclose(O.attn_logp_rows(q, K)[0, 0], ref, atol=1e-14)


# ---------------------------------------------------------------- KL drift (Eq. 4)
def test_kl_closed_forms():
    for line in _read("kl.txt"):
        a, b, v = [t.strip() for t in line.split(";")]
        a = np.array([float(t) for t in a.split()])
        b = np.array([float(t) for t in b.split()])
        with np.errstate(divide="ignore"):
            la, lb = np.log(a), np.log(b)
        la = np.where(a > 0, la, -1e300)     # 0 ln 0 = 0: p = exp(-1e300) = 0
        got = O.kl_rows(la[None, None, :], lb[None, None, :])[0]
        assert abs(got - float(v)) < 1e-12, line


def test_kl_against_uniform_is_logN_minus_entropy():
    N = 512
    s = rng.standard_normal(N) * 3
    lp = s - np.log(np.exp(s).sum())
    lu = np.full(N, -math.log(N))
    H = -(np.exp(lp) * lp).sum()
    assert abs(O.kl_rows(lp[None, None], lu[None, None])[0] - (math.log(N) - H)) < 1e-12
    onehot = np.full(N, -1e300)
    onehot[17] = 0.0
    assert abs(O.kl_rows(onehot[None, None], lu[None, None])[0] - math.log(512)) < 1e-12


def test_kl_matches_library_and_head_mean_and_is_not_symmetric():
    R, nh, N = 4, 3, 50
    a = rng.standard_normal((R, nh, N))
    b = rng.standard_normal((R, nh, N))
    la = a - np.log(np.exp(a).sum(-1, keepdims=True))
    lb = b - np.log(np.exp(b).sum(-1, keepdims=True))
    import scipy.stats
    ref = scipy.stats.entropy(np.exp(la), np.exp(lb), axis=-1).mean(-1)
    got = O.kl_rows(la, lb)
    assert np.allclose(got, ref, rtol=1e-12)
    tref = torch.nn.functional.kl_div(torch.tensor(lb), torch.tensor(la), log_target=True,
                                      reduction="none").sum(-1).mean(-1).numpy()
    assert np.allclose(got, tref, rtol=1e-12)
    assert not np.allclose(got, O.kl_rows(lb, la))          # argument order matters
    assert (got >= 0).all()
    assert np.array_equal(O.kl_rows(la, la), np.zeros(R))   # identical rows: exactly zero


def test_pinsker_bound_on_attention_output_change():
    # Appendix B, Prop. 2: ||sum_j (a_j - a'_j) v_j|| <= M ||a - a'||_1 <= M sqrt(2 KL(a||a'))
    N, dh = 64, 16
    V = rng.standard_normal((N, 1, dh))
    M = np.linalg.norm(V[:, 0], axis=-1).max()
    for _ in range(20):
        s1 = rng.standard_normal((1, 1, N)) * 2
        s2 = s1 + rng.standard_normal((1, 1, N)) * rng.uniform(0.01, 1.0)
        l1 = s1 - np.log(np.exp(s1).sum(-1, keepdims=True))
        l2 = s2 - np.log(np.exp(s2).sum(-1, keepdims=True))
        kl = O.kl_rows(l1, l2)[0]
        d_out = np.linalg.norm(O.attn_out_rows(l1, V) - O.attn_out_rows(l2, V))
        l1n = np.abs(np.exp(l1) - np.exp(l2)).sum()
        assert d_out <= M * l1n + 1e-12
        assert l1n <= math.sqrt(2 * kl) + 1e-12


def test_first_order_attention_perturbation():
    # Appendix B, Prop. 1: o_i(x_s + eta) - o_i(x_s) = a_is W_V eta
    #   + a_is (q_i^T W_K eta / sqrt(dh)) (v_s - o_i) + O(|eta|^2)   (single head, no norm / RoPE)
    d, dh, N = 12, 8, 9
    X = rng.standard_normal((N, d))
    WQ, WK, WV = (rng.standard_normal((dh, d)) * 0.3 for _ in range(3))
    i, s = 2, 6

    def out(Xm):
        q = (Xm[i] @ WQ.T)[None, None, :]
        K = (Xm @ WK.T)[:, None, :]
        Vm = (Xm @ WV.T)[:, None, :]
        lp = O.attn_logp_rows(q, K)
        return O.attn_out_rows(lp, Vm)[0], np.exp(lp[0, 0]), Vm[:, 0]

    o0, a, Vm = out(X)
    eta = rng.standard_normal(d)
    for eps in (1e-4, 1e-5):
        X2 = X.copy()
        X2[s] += eps * eta
        o1, _, _ = out(X2)
        q = X[i] @ WQ.T
        pred = a[s] * (WV @ (eps * eta)) + a[s] * (q @ (WK @ (eps * eta)) / math.sqrt(dh)) * (Vm[s] - o0)
        assert np.linalg.norm((o1 - o0) - pred) < 50 * eps ** 2 * np.linalg.norm(eta) ** 2
        assert np.linalg.norm(o1 - o0) > 1e-3 * eps           # the drift itself is not zero


# ---------------------------------------------------------------- selection
def test_select_budget_table():
    for line in _read("select_k.txt"):
        rho, W, k = line.split()
        D = rng.random(int(W)) + 0.1
        got = O.select_rows(D, O.SELECT_TOPK_FRAC, frac=float(rho))
        assert len(got) == int(k), line


def test_select_equals_stable_argsort_bruteforce():
    for W in (1, 7, 96, 257):
        D = np.round(rng.random(W), 1)          # many ties
        D[rng.random(W) < 0.2] = 0.0
        k = max(1, W // 4)
        order = np.argsort(-D, kind="stable")   # descending value, ascending index on ties
        ref = sorted(int(i) for i in order[:k] if D[i] > 0.0)
        got = O.select_rows(D, O.SELECT_TOPK_COUNT, k=k, floor=0.0)
        assert list(got) == ref
        assert list(got) == sorted(got)


def test_select_modes_and_zero_drift():
    D = np.array([0.0, 0.5, 0.0, 0.2, 0.9])
    assert list(O.select_rows(D, O.SELECT_ALL)) == [0, 1, 2, 3, 4]
    assert list(O.select_rows(D, O.SELECT_NONE)) == []
    assert list(O.select_rows(D, O.SELECT_THRESHOLD, thresh=0.3)) == [1, 4]
    assert list(O.select_rows(D, O.SELECT_THRESHOLD, thresh=np.inf)) == []
    assert list(O.select_rows(D, O.SELECT_TOPK_COUNT, k=4)) == [1, 3, 4]      # floor removes zeros
    assert list(O.select_rows(np.zeros(96), O.SELECT_TOPK_FRAC, frac=0.25)) == []
    assert list(O.select_rows(D, O.SELECT_TOPK_COUNT, k=2)) == [1, 4]


# ---------------------------------------------------------------- confidence / commit
def test_confidence_is_softmax_of_argmax_excluding_mask():
    V, mask_id = 50, 49
    l = rng.standard_normal((6, V)) * 3
    l[0, mask_id] = 100.0              # MASK has the largest logit: must not be chosen
    l[1, 5] = l[1, 9] = 50.0           # tie: lowest id
    yhat, c = O.confidence_rows(l, mask_id)
    p = torch.softmax(torch.tensor(l), -1).numpy()
    for r in range(6):
        cand = [v for v in range(V) if v != mask_id]
        best = max(cand, key=lambda v: (l[r, v], -v))
        assert yhat[r] == best
        assert abs(c[r] - p[r, best]) < 1e-13
    assert yhat[1] == 5 and c[0] < 1e-20


def test_tau_d_table():
    for line in _read("tau_d.txt"):
        alpha, tau_s, c, want = (float(t) for t in line.split())
        r = O.commit_rule(np.array([c]), np.array([0]), np.array([True]), np.array([0.0]), [],
                          within=True, tau_s=tau_s, alpha=alpha, ge=True, drift_commit=True, quota=0)
        assert abs(r["tau_d"][0] - want) < 1e-12, line


def _scalar_commit(conf, masked, delta, hist, tau_s, alpha, ge, drift, quota, within):
    B = len(conf)
    out = set()
    for j in range(B):
        if not masked[j]:
            continue
        mean = sum(h[j] for h in hist) / len(hist) if hist else 0.0
        Dl = (delta[j] - mean) if within else 0.0
        td = alpha * (tau_s - conf[j]) * (tau_s - conf[j])
        c_ok = conf[j] >= tau_s if ge else conf[j] > tau_s
        d_ok = within and drift and (Dl >= td if ge else Dl > td)
        if c_ok or d_ok:
            out.add(j)
    rest = sorted((j for j in range(B) if masked[j] and j not in out), key=lambda j: (-conf[j], j))
    while len(out) < quota and rest:
        out.add(rest.pop(0))
    return out


def test_commit_rule_bruteforce_and_invariants():
    B = 32
    for trial in range(200):
        conf = rng.random(B)
        masked = rng.random(B) < 0.7
        delta = rng.random(B) * 4
        hist = [rng.random(B) for _ in range(rng.integers(0, 6))]
        alpha = float(rng.choice([2.5, 10.0, 40.0]))
        tau_s = float(rng.choice([0.7, 0.9]))
        ge = bool(rng.integers(0, 2))
        drift = bool(rng.integers(0, 2))
        within = bool(rng.integers(0, 2))
        quota = int(rng.integers(0, 5))
        quota = min(quota, int(masked.sum()))
        r = O.commit_rule(conf, np.zeros(B, int), masked, delta, hist, within=within, tau_s=tau_s,
                          alpha=alpha, ge=ge, drift_commit=drift, quota=quota)
        got = set(np.nonzero(r["commit"])[0].tolist())
        assert got == _scalar_commit(conf, masked, delta, hist, tau_s, alpha, ge, drift, quota, within)
        assert got <= set(np.nonzero(masked)[0].tolist())                 # only masked rows commit
        assert len(got) >= quota                                          # progress
        hi = {j for j in range(B) if masked[j] and conf[j] > tau_s}
        assert hi <= got                                                  # confident rows always commit
        assert not (r["by_conf"] & r["by_drift"]).any()


def test_commit_reductions():
    B = 16
    conf = np.linspace(0.05, 0.99, B)
    masked = np.ones(B, bool)
    delta = rng.random(B) * 3
    kw = dict(within=True, tau_s=0.9, ge=True, drift_commit=True, quota=0)
    # alpha -> infinity: confidence-only commit (Sec. 4.2)
    r = O.commit_rule(conf, np.zeros(B, int), masked, delta, [], alpha=1e30, **kw)
    assert set(np.nonzero(r["commit"])[0]) == {j for j in range(B) if conf[j] >= 0.9}
    # empty history (h = 0): Delta is the raw drift (Appendix D, "Drift history size")
    r = O.commit_rule(conf, np.zeros(B, int), masked, delta, [], alpha=10.0, **kw)
    assert np.array_equal(r["Delta"], delta)
    # history mean is subtracted
    hist = [np.full(B, 1.0), np.full(B, 3.0)]
    r = O.commit_rule(conf, np.zeros(B, int), masked, delta, hist, alpha=10.0, **kw)
    assert np.allclose(r["Delta"], delta - 2.0)
    # tau_d is symmetric around tau_s and zero at c = tau_s
    r2 = O.commit_rule(np.array([0.8, 1.0, 0.9]), np.zeros(3, int), np.ones(3, bool), np.zeros(3), [],
                       alpha=10.0, **kw)
    assert abs(r2["tau_d"][0] - r2["tau_d"][1]) < 1e-12 and r2["tau_d"][2] == 0.0
    # entry steps never use the drift clause
    r = O.commit_rule(conf, np.zeros(B, int), masked, delta + 100, [], alpha=10.0, within=False,
                      tau_s=0.9, ge=True, drift_commit=True, quota=0)
    assert not r["by_drift"].any()


# ---------------------------------------------------------------- staleness metric
def test_staleness_metric():
    K = rng.standard_normal((5, 2, 8))
    V = rng.standard_normal((5, 2, 8))
    assert np.allclose(O.staleness(K, K, V, V), 0.0, atol=1e-15)
    assert np.allclose(O.staleness(K, -K, V, -V), 2.0)
    assert np.allclose(O.staleness(K, 3.0 * K, V, V), 0.0, atol=1e-15)     # scale-free
    assert np.allclose(O.staleness(K, -K, V, V), 1.0)


# ---------------------------------------------------------------- K/V refresh (Cor. 1)
def test_refresh_delta_bounded_by_projection_norm():
    # Appendix B, Cor. 1: ||[dK; dV]|| <= ||[W_K; W_V]||_2 ||dH||, and dH = 0 => dK = dV = 0.
    # With RMSNorm in front the hidden difference is that of the normed rows; RoPE is orthogonal.
    d, nkv, dh = 32, 2, 8
    wk, wv = rng.standard_normal((nkv * dh, d)), rng.standard_normal((nkv * dh, d))
    g = np.ones(d)
    h0 = rng.standard_normal((6, d))
    h1 = h0 + rng.standard_normal((6, d)) * 0.1
    h1[3] = h0[3]
    pos = np.arange(6) * 11

    def kv(h):
        a = O.rmsnorm(h, g, 1e-5)
        k = O.rope((a @ wk.T).reshape(6, nkv, dh), pos, 10000.0).reshape(6, -1)
        return a, k, a @ wv.T
    a0, k0, v0 = kv(h0)
    a1, k1, v1 = kv(h1)
    lhs = np.sqrt(((k1 - k0) ** 2).sum(-1) + ((v1 - v0) ** 2).sum(-1))
    sig = np.linalg.norm(np.concatenate([wk, wv], 0), 2)
    assert (lhs <= sig * np.linalg.norm(a1 - a0, axis=-1) + 1e-12).all()
    assert lhs[3] == 0.0


def test_refresh_chain_rows_equal_full_recompute():
    # Sec. 4.1 "Measuring Drift and Layer-wise KV Updates": a refreshed K/V row is what a full recompute of the
    # same hidden row gives; rows that were not selected keep their old contents.  The full recompute here is
    # written with an independent rotary formula (complex rotation at the row's absolute position) and with
    # per-row matrix-vector products, so a wrong position, a wrong gain or a scatter to the wrong row shows.
    P, d, nh, nkv, dh, k = 23, 32, 4, 2, 8, 7
    H = rng.standard_normal((P, d))
    drift = np.exp(rng.standard_normal(P))
    drift[5] = 0.0                                       # never a candidate
    wq, wk, wv = (rng.standard_normal((n * dh, d)) for n in (nh, nkv, nkv))
    gain = 1.0 + 0.3 * rng.standard_normal(d)
    theta = 500.0
    Kc, Vc = rng.standard_normal((P, nkv, dh)), rng.standard_normal((P, nkv, dh))
    idx, q, K2, V2 = O.refresh_chain(H, drift, k, wq, wk, wv, gain, 1e-5, theta, nh, nkv, dh, Kc, Vc, emulate_bf16=False)
    assert idx.tolist() == sorted(np.argsort(-drift, kind="stable")[:k].tolist())       # brute-force top-k, ascending
    half = dh // 2
    inv = theta ** (-2.0 * np.arange(half) / dh)

    def rot(x, pos):        # half-split pairs (i, i + dh/2) rotated by pos * theta^(-2i/dh)
        z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * pos * inv)
        return np.concatenate([z.real, z.imag], -1)
    for t, r in enumerate(idx):
        a = H[r] / np.sqrt(np.mean(H[r] ** 2) + 1e-5) * gain
        assert np.allclose(K2[r], rot((wk @ a).reshape(nkv, dh), r), rtol=1e-12, atol=1e-12)
        assert np.allclose(V2[r], (wv @ a).reshape(nkv, dh), rtol=1e-12, atol=1e-12)
        assert np.allclose(q[t], rot((wq @ a).reshape(nh, dh), r), rtol=1e-12, atol=1e-12)
    rest = np.setdiff1d(np.arange(P), idx)
    assert np.array_equal(K2[rest], Kc[rest]) and np.array_equal(V2[rest], Vc[rest])
    assert 5 not in idx
    # unchanged hidden row => unchanged K/V (Cor. 1 with dH = 0): refreshing twice changes nothing
    _, _, K3, V3 = O.refresh_chain(H, drift, k, wq, wk, wv, gain, 1e-5, theta, nh, nkv, dh, K2, V2, emulate_bf16=False)
    assert np.array_equal(K3, K2) and np.array_equal(V3, V2)


# ---------------------------------------------------------------- centroid proxies (Sec. 4.1)
def test_spherical_kmeans_pins():
    # well separated directions are recovered whatever the rows' lengths (cosine similarity: "spherical")
    d, K = 16, 4
    dirs = np.linalg.qr(rng.standard_normal((d, d)))[0][:K]              # orthonormal centres
    truth = np.array([0, 1, 2, 3] * 6)                                     # evenly spread, so every start row differs
    H = dirs[truth] + 0.05 * rng.standard_normal((len(truth), d))
    scale = 10.0 ** rng.uniform(-3, 3, size=(len(truth), 1))
    lab = O.spherical_kmeans(H * scale, K, 4)
    assert np.array_equal(lab, O.spherical_kmeans(H, K, 4))                # row scale does not matter
    # same partition as the truth (cluster ids are a permutation)
    assert len(set(zip(lab.tolist(), truth.tolist()))) == K
    # no more rows than clusters: every row its own cluster
    assert sorted(O.spherical_kmeans(H[:3], 8, 4).tolist()) == [0, 1, 2]
    assert O.spherical_kmeans(np.zeros((0, d)), 8, 4).shape == (0,)
    # brute force on random data: the returned labels are the nearest centres of the centres that the
    # previous iteration produced, and the objective (sum of cosines to the own centre) never decreases
    X = rng.standard_normal((40, 6))
    U = X / np.linalg.norm(X, axis=1, keepdims=True)
    Ke = 5
    C = np.stack([U[int(np.floor((j + 0.5) * 40 / Ke))] for j in range(Ke)])
    obj_prev = -np.inf
    for it in range(1, 5):
        lab_it = np.array([int(np.argmax([U[i] @ C[j] for j in range(Ke)])) for i in range(40)])
        assert np.array_equal(lab_it, O.spherical_kmeans(X, Ke, it))
        for j in range(Ke):
            mem = U[lab_it == j]
            if len(mem):
                C[j] = mem.sum(0) / np.linalg.norm(mem.sum(0))
        obj = sum(U[i] @ C[lab_it[i]] for i in range(40))
        assert obj >= obj_prev - 1e-12
        obj_prev = obj


def test_cluster_proxies_pins():
    H = rng.standard_normal((7, 5))
    pos = np.array([3, 4, 5, 6, 20, 21, 22])
    lab = np.array([0, 0, 2, 2, 2, 4, 0])
    Z, zp, cnt = O.cluster_proxies(H, pos, lab, 6)
    assert cnt.tolist() == [3, 0, 3, 0, 1, 0]
    assert np.allclose(Z[0], (H[0] + H[1] + H[6]) / 3) and np.allclose(Z[2], H[2:5].mean(0))
    assert np.array_equal(Z[4], H[5]) and zp[4] == 21                      # a cluster of one row is that row
    assert zp[0] == int(np.floor((3 + 4 + 22) / 3 + 0.5)) and zp[2] == 10   # rounded mean position
    assert not Z[1].any() and not Z[3].any()


# ---------------------------------------------------------------- NVFP4 residual codec (Appendix "Quantization Format")
def test_e4m3_scale_rounding_matches_library_cast():
    x = np.abs(rng.standard_normal(200000)).astype(np.float32) * np.float32(10.0) ** rng.integers(-5, 3, 200000).astype(np.float32)
    x = np.concatenate([x, np.float32([0.0, 2.0 ** -9, 2.0 ** -10, 1.5 * 2.0 ** -9, 448.0, 1000.0, 0.0625 * 1.0625])])
    ref = torch.tensor(np.minimum(x, np.float32(448.0))).to(torch.float8_e4m3fn).float().numpy()     # library: RNE; saturation by the clamp
    assert np.array_equal(O.e4m3_round(x), ref)


def test_e2m1_grid_is_the_formats_value_set():
    # 1 sign, 2 exponent (bias 1), 1 mantissa bit: subnormals m/2, normals (1 + m/2) 2^(e-1)
    vals = sorted({(m / 2.0) if e == 0 else (1 + m / 2.0) * 2.0 ** (e - 1) for e in range(4) for m in range(2)})
    assert vals == O.E2M1_GRID.tolist() == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def test_nvfp4_quantize_pins():
    r = (rng.standard_normal((64, 128)) * 10.0 ** rng.integers(-3, 2, (64, 1))).astype(np.float32)
    r[3, 16:32] = 0.0                                            # an all-zero group
    r[5, 0] = 1e4                                                # an outlier: the rest of its group rounds to zero
    codes, scale = O.nvfp4_quantize(r)
    dq = O.nvfp4_dequantize(codes, scale)
    g, gq = r.reshape(64, 8, 16), dq.reshape(64, 8, 16)
    amax = np.abs(g).max(-1)
    assert np.array_equal(scale, O.e4m3_round(amax / np.float32(6.0))) and (scale[3, 1] == 0) and not gq[3, 1].any()
    # brute force: every code is a nearest grid point of |x| / s (saturating), sign kept
    for i, j, k in [(a, b, c) for a in range(0, 64, 7) for b in range(8) for c in range(16)]:
        if scale[i, j] == 0:
            continue
        y = abs(g[i, j, k]) / scale[i, j]
        best = np.abs(O.E2M1_GRID - min(y, np.float32(6.0))).min()
        assert abs(abs(gq[i, j, k]) / scale[i, j] - min(y, 6.0)) <= best + 1e-6
        assert gq[i, j, k] == 0 or np.sign(gq[i, j, k]) == np.sign(g[i, j, k])
    # ties go to the even code: 0.25 -> 0, 0.75 -> 1, 1.25 -> 1, 1.75 -> 2, 2.5 -> 2, 3.5 -> 4, 5 -> 4 (scale 1: amax 6)
    t = np.zeros((1, 16), np.float32)
    t[0, :8] = [6.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    c, s1 = O.nvfp4_quantize(t)
    assert s1[0, 0] == 1.0 and O.nvfp4_dequantize(c, s1)[0, :8].tolist() == [6.0, 0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0]
    # error bound: half the coarsest grid step (2) times the scale, plus what saturation at 6 s cuts off
    assert (np.abs(g - gq) <= scale[..., None] * 1.0 + np.maximum(np.abs(g) - 6 * scale[..., None], 0) + 1e-12).all()
    # a group whose largest code is 6 keeps its scale, so its grid points stay put when quantised again
    top = np.abs(gq).max(-1) == 6 * scale
    c2, s2 = O.nvfp4_quantize(dq)
    assert top.any() and np.array_equal(O.nvfp4_dequantize(c2, s2).reshape(64, 8, 16)[top], gq[top])
    # the residual round trip keeps the reference exactly when the row equals it
    ref = rng.standard_normal((4, 32)).astype(np.float32)
    assert np.array_equal(O.residual_nvfp4_roundtrip(ref, ref), ref.astype(np.float64))
