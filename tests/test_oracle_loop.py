"""Whole-loop pins for the CPU oracle on tiny models: brute force against no-cache
decoding, schedule reductions, commit invariants (no GPU needed)."""
import dataclasses

import numpy as np
import pytest

from oracle import polestar_oracle as O
from paper_2607_14107_b200 import inputs as I


def tiny(nkv=1, **kw):
    m = I.ModelCfg(2, 64, 2, nkv, 32, 128, 96, I.DTYPE_F32, 1e-5, 10000.0)
    p = I.Params(batch=1, prompt_len=16, gen_len=24, block=8, max_steps=12)
    p = dataclasses.replace(p, **kw)
    w = I.weights_to_numpy(I.make_weights(m, seed=0, std=0.2))
    prompt = I.make_prompt(m, p).numpy()
    return m, p, w, prompt


def test_full_refresh_equals_nocache_bitwise():
    # Sec. 4.1: layer-wise packets keep the cache aligned with the evolving context; when every
    # non-active row is refreshed at every step the result is the full-recompute baseline of
    # Sec. 3.1 ("Setup").  Row-independent arithmetic makes this exact.
    m, p, w, prompt = tiny(select_mode=I.SELECT_ALL, tau_upd=-1, win_prefix_blocks=100,
                           win_suffix_blocks=100, logit_scale=1.0, tau_suffix=0.4)
    a = O.PolestarOracle(m, w, p, prompt, rowwise=True)
    b = O.NoCacheOracle(m, w, p, prompt, rowwise=True)
    n_within = n_suffix = 0
    while not a.done:
        a.step()
        b.step()
        ta, tb = a.seqs[0].trace, b.seqs[0].trace
        for xa, xb in zip(ta["x_act"], tb["x_act"]):
            assert np.array_equal(xa, xb)
        assert np.array_equal(ta["logits"], tb["logits"])
        if ta["kind"] == "within":
            n_within += 1
            assert np.array_equal(ta["delta"], tb["delta"])
            for l in range(m.n_layers):       # whole cache equals the full recompute
                assert np.array_equal(a.seqs[0].Kc[l], b.seqs[0].Kc[l])
                assert np.array_equal(a.seqs[0].Vc[l], b.seqs[0].Vc[l])
        ia, ib = a.commit(), b.commit()
        assert np.array_equal(ia[0]["commit"], ib[0]["commit"])
        # the no-cache decoder has no packets, hence no suffix commits: copy those over so both
        # decoders keep seeing the same tokens (this also drives the layer-0 packet path)
        n_suffix += ia[0]["n_suffix"]
        act = a.seqs[0].act
        assert np.array_equal(a.tokens()[0, act], b.tokens()[0, act])
        b.seqs[0].y[:] = a.seqs[0].y
        b.inner.b, b.inner.need_entry, b.inner.done = a.b, a.need_entry, a.done
        b.inner.steps_used = a.steps_used
    assert n_within > 3 and n_suffix > 0


def test_sparse_refresh_differs_from_nocache_but_stays_close():
    # the default sparse policy is an approximation: it must NOT be bit-identical (otherwise the
    # pin above could not detect a refresh that silently recomputes everything) ...
    m, p, w, prompt = tiny(tau_upd=-1, logit_scale=6.0)
    a = O.PolestarOracle(m, w, p, prompt)
    b = O.NoCacheOracle(m, w, p, prompt)
    errs = []
    for _ in range(3):
        a.step(); b.step()
        errs.append(np.abs(a.seqs[0].trace["x_act"][-1] - b.seqs[0].trace["x_act"][-1]).max())
        forced = [dict(commit=i["commit"], suffix=()) for i in b.commit()]
        a.commit(forced)
    assert errs[0] < 1e-12 and max(errs[1:]) > 1e-9
    # ... and the staleness metric (Appendix C.2) of the refreshed rows is zero-ish only under ALL
    E = O.staleness(a.seqs[0].Kc[1], b.seqs[0].Kc[1], a.seqs[0].Vc[1], b.seqs[0].Vc[1])
    assert np.isfinite(E).all() and E.max() > 0.0 and E.min() >= -1e-12


def test_zero_drift_refreshes_nothing():
    # nothing decoded between entry and the next step: every attention row is unchanged,
    # D = 0 exactly, top-k picks nothing, the cache is untouched.
    m, p, w, prompt = tiny(tau_upd=-1)
    a = O.PolestarOracle(m, w, p, prompt, rowwise=True)
    a.step()
    a.commit([dict(commit=np.zeros(p.block, bool), suffix=())])
    s = a.seqs[0]
    K0 = [k.copy() for k in s.Kc]
    V0 = [v.copy() for v in s.Vc]
    H0 = [h.copy() for h in s.Hc]
    a.step()
    tr = s.trace
    assert tr["kind"] == "within" and tr["refresh"]
    for l in range(m.n_layers):
        assert np.array_equal(tr["D"][l], np.zeros(len(s.win)))
        assert len(tr["sel"][l]) == 0
        assert np.array_equal(s.Kc[l], K0[l]) and np.array_equal(s.Vc[l], V0[l])
        assert np.array_equal(s.Hc[l], H0[l])
    assert np.array_equal(tr["delta"], np.zeros(p.block))


def test_no_refresh_schedule_is_a_static_block_cache():
    # tau_upd = infinity (Sec. 5.3 "Update Schedule"): rows outside the active block keep the
    # values written at block entry for the whole block.
    m, p, w, prompt = tiny(tau_upd=I.TAU_UPD_NEVER, logit_scale=6.0)
    a = O.PolestarOracle(m, w, p, prompt)
    a.step(); a.commit()
    s = a.seqs[0]
    other = np.setdiff1d(np.arange(s.N), s.act)
    K0 = s.Kc[1][other].copy()
    while not a.need_entry:
        a.step()
        assert not s.trace["refresh"]
        a.commit()
        assert np.array_equal(s.Kc[1][other], K0)


def test_update_schedule_counts_decoded_tokens():
    # Sec. 4.1 "Update Schedule": refresh once more than tau_upd tokens were decoded since the
    # last refresh (a single step decoding > tau_upd tokens is the same test).
    m, p, w, prompt = tiny(tau_upd=3, max_steps=24)          # quota 1: one token per step
    a = O.PolestarOracle(m, w, p, prompt)
    kinds = []
    while not a.done:
        a.step()
        tr = a.seqs[0].trace
        kinds.append(tr["kind"][0] + ("r" if tr.get("refresh") else ""))
        a.commit()
    # per block: entry (1 token, cum=1), w (2), w (3), w (4), then cum=4 > 3 -> refresh, ...
    assert kinds[:8] == ["e", "w", "w", "w", "wr", "w", "w", "w"]
    assert a.forwards == 24


def test_alternate_entries_are_full_sequence():
    m, p, w, prompt = tiny()
    a = O.PolestarOracle(m, w, p, prompt)
    kinds = []
    while not a.done:
        a.step()
        if a.seqs[0].trace["kind"].startswith("entry"):
            kinds.append((a.seqs[0].trace["kind"], len(a.seqs[0].trace["rows"])))
        a.commit()
    assert kinds == [("entry_full", 40), ("entry_window", 32), ("entry_full", 40)]


def test_window_geometry():
    p = I.Params(prompt_len=256, gen_len=256, block=32)
    pre, suf = O.window_positions(p, 0)
    assert pre == list(range(192, 256)) and suf == list(range(288, 320))
    pre, suf = O.window_positions(p, 7)                       # last block: suffix clipped away
    assert pre == list(range(416, 480)) and suf == []
    p = I.Params(prompt_len=16, gen_len=64, block=32)
    pre, suf = O.window_positions(p, 0)                       # prefix clipped at the sequence start
    assert pre == list(range(0, 16)) and suf == list(range(48, 80))


def test_decode_terminates_within_budget_and_never_rewrites_tokens():
    m, p, w, prompt = tiny(logit_scale=8.0, nkv=2)
    a = O.PolestarOracle(m, w, p, prompt)
    prev = a.tokens().copy()
    while not a.done:
        a.step()
        infos = a.commit()
        cur = a.tokens()
        was_unmasked = prev != m.mask_id
        assert np.array_equal(cur[was_unmasked], prev[was_unmasked])
        changed = np.nonzero(cur[0] != prev[0])[0]
        s = a.seqs[0]
        allowed = set(s.act.tolist()) | set(s.win[s.n_pre:].tolist())
        assert set(changed.tolist()) <= allowed
        assert len(changed) == infos[0]["n_committed"]
        prev = cur.copy()
    assert a.forwards <= p.max_steps
    assert not (a.tokens() == m.mask_id).any()
    assert np.array_equal(a.tokens()[0, :p.prompt_len], prompt[0])
    assert a.generated == p.gen_len
    assert abs(a.tpf - a.generated_non_eos / a.forwards) < 1e-15


def test_quota_gives_32_forwards_for_64_tokens():
    m, p = I.config("c1")
    m = dataclasses.replace(m, d_model=64, n_heads=2, n_kv_heads=2, head_dim=32, d_ffn=128, vocab=128,
                            mask_id=127, eos_id=126)
    w = I.weights_to_numpy(I.make_weights(m))
    a = O.PolestarOracle(m, w, p, I.make_prompt(m, p).numpy())
    a.decode()
    assert a.forwards == 32 and a.generated == 64


def test_commit_branches_fire_with_scaled_logits():
    m, p, w, prompt = tiny(logit_scale=3.0, tau_upd=-1, alpha=3.0, max_steps=24, tau_suffix=0.7)
    a = O.PolestarOracle(m, w, p, prompt)
    tot = dict(n_by_conf=0, n_by_drift=0, n_by_quota=0, n_suffix=0)
    while not a.done:
        a.step()
        for i in a.commit():
            for k in tot:
                tot[k] += i[k]
    assert min(tot.values()) > 0
    assert sum(tot.values()) == p.gen_len


def test_suffix_commit_goes_through_layer0_packet():
    # a suffix token committed early changes that position's embedding; the next refresh step
    # must carry it into the cache (otherwise full refresh could not equal no-cache decoding)
    m, p, w, prompt = tiny(logit_scale=3.0, tau_upd=-1, select_mode=I.SELECT_ALL, tau_suffix=0.7, max_steps=24)
    a = O.PolestarOracle(m, w, p, prompt)
    seen = False
    while not a.done and not seen:
        a.step()
        info = a.commit()[0]
        if info["n_suffix"] and not a.need_entry:
            pos = info["suffix_committed"][0]
            a.step()
            s = a.seqs[0]
            wi = int(np.nonzero(s.win == pos)[0][0])
            assert wi in s.trace["patched"][0].tolist()
            assert np.allclose(s.Hc[0][wi], w["embed"][s.y[pos]])
            a.commit()
            seen = True
    assert seen


def test_batch_sequences_are_independent():
    m, p, w, _ = tiny(logit_scale=8.0)
    p2 = dataclasses.replace(p, batch=2)
    prompt = I.make_prompt(m, p2).numpy()
    both = O.PolestarOracle(m, w, p2, prompt)
    both.decode()
    for s in range(2):
        one = O.PolestarOracle(m, w, p, prompt[s:s + 1])
        # alone, a sequence may finish blocks earlier than in lock-step; compare its tokens
        # under the lock-step schedule by replaying the batch decoder with the other row copied
        pair = O.PolestarOracle(m, w, p2, np.stack([prompt[s], prompt[s]]))
        pair.decode()
        one.decode()
        assert np.array_equal(pair.tokens()[0], pair.tokens()[1])
        assert np.array_equal(pair.tokens()[0], one.tokens()[0])
    assert both.tokens().shape == (2, p.seq_len)


def test_bf16_emulation_changes_little():
    m, p, w, prompt = tiny(logit_scale=6.0)
    wb = {k: (O.bf16_round(v) if not isinstance(v, list) else
              [{kk: O.bf16_round(vv) for kk, vv in l.items()} for l in v]) for k, v in w.items()}
    a = O.PolestarOracle(m, wb, p, prompt, emulate_bf16=False)
    b = O.PolestarOracle(m, wb, p, prompt, emulate_bf16=True)
    a.step(); b.step()
    xa, xb = a.seqs[0].trace["x_act"][-1], b.seqs[0].trace["x_act"][-1]
    assert 0 < np.abs(xa - xb).max() < 2e-2 * np.abs(xa).max()


# ---------------------------------------------------------------- centroid proxies (Sec. 4.1)
def test_singleton_clusters_equal_per_position_mode():
    # With at least as many clusters as window rows every cluster is one row: its proxy is the row itself at the
    # row's position, so cluster drift is row drift and "top-k clusters" is "top-k rows": the whole decode must be
    # that of the per-position mode with the same budget: the same refresh sets and tokens, and the same numbers
    # up to the rounding of the incremental centroid update (old + (new - old) instead of new).
    m, p, w, prompt = tiny(logit_scale=3.0, tau_upd=-1, tau_suffix=0.7)
    pa = dataclasses.replace(p, select_mode=I.SELECT_TOPK_COUNT, select_k=5)
    pb = dataclasses.replace(p, select_mode=I.SELECT_CLUSTER_TOPK, n_clusters=64, cluster_k=5)
    a, b = O.PolestarOracle(m, w, pa, prompt, rowwise=True), O.PolestarOracle(m, w, pb, prompt, rowwise=True)
    n_ref = 0
    while not a.done:
        a.step(); b.step()
        ta, tb = a.seqs[0].trace, b.seqs[0].trace
        assert np.allclose(ta["logits"], tb["logits"], rtol=1e-9, atol=1e-9)
        if ta["kind"] == "within" and ta["refresh"]:
            n_ref += 1
            W = len(a.seqs[0].win)
            for l in range(m.n_layers):
                assert np.array_equal(ta["sel"][l], tb["sel"][l])
                assert np.allclose(ta["D"][l], tb["D"][l][:W], rtol=1e-9, atol=1e-12)
                assert np.allclose(a.seqs[0].Kc[l], b.seqs[0].Kc[l], rtol=1e-9, atol=1e-9)
        a.commit(); b.commit()
        assert np.array_equal(a.tokens(), b.tokens())
    assert b.done and n_ref > 5


def test_all_clusters_selected_equals_nocache_bitwise():
    # every cluster chosen at every step = every window row refreshed: the full-recompute baseline again
    m, p, w, prompt = tiny(select_mode=I.SELECT_CLUSTER_TOPK, n_clusters=4, cluster_k=4, tau_upd=-1,
                           win_prefix_blocks=100, win_suffix_blocks=100, tau_suffix=0.4)
    a = O.PolestarOracle(m, w, p, prompt, rowwise=True)
    b = O.NoCacheOracle(m, w, dataclasses.replace(p, select_mode=I.SELECT_ALL), prompt, rowwise=True)
    n_within = 0
    while not a.done:
        a.step(); b.step()
        ta, tb = a.seqs[0].trace, b.seqs[0].trace
        assert np.array_equal(ta["logits"], tb["logits"])
        if ta["kind"] == "within":
            n_within += 1
            for l in range(m.n_layers):
                assert np.array_equal(a.seqs[0].Kc[l], b.seqs[0].Kc[l])
        ia, ib = a.commit(), b.commit()
        assert np.array_equal(ia[0]["commit"], ib[0]["commit"])
        # (the no-cache decoder has no packets, hence no suffix commits: copy those over)
        b.seqs[0].y[:] = a.seqs[0].y
        b.inner.b, b.inner.need_entry, b.inner.done = a.b, a.need_entry, a.done
        b.inner.steps_used = a.steps_used
    assert n_within > 3


def test_cluster_mode_invariants():
    m, p, w, prompt = tiny(select_mode=I.SELECT_CLUSTER_TOPK, n_clusters=4, cluster_k=2, tau_upd=-1, logit_scale=3.0)
    a = O.PolestarOracle(m, w, p, prompt)
    n_ref = 0
    while not a.done:
        a.step()
        s = a.seqs[0]
        tr = s.trace
        if tr["kind"] == "within" and tr["refresh"]:
            n_ref += 1
            for l in range(m.n_layers):
                D, S, chosen = tr["D"][l], tr["sel"][l], tr["clusters"][l]
                assert D.shape == (p.n_clusters,) and (D >= -1e-12).all()
                assert len(chosen) <= p.cluster_k
                # the refreshed rows are exactly the members of the chosen clusters, ascending
                assert S.tolist() == [i for i in range(len(s.win)) if s.labels[l][i] in chosen.tolist()]
                # the chosen clusters are the ones with the largest positive drift
                rest = [c for c in range(p.n_clusters) if c not in chosen.tolist() and D[c] > 0]
                if len(chosen) and rest:
                    assert D[chosen].min() >= max(D[c] for c in rest)
                # incremental centroid update == mean of the members' current hidden rows
                Z, _, cnt = O.cluster_proxies(s.Hc[l], s.win, s.labels[l], p.n_clusters)
                assert np.allclose(Z, s.Z[l], rtol=1e-11, atol=1e-12) and np.array_equal(cnt, s.zcnt[l])
        a.commit()
    assert n_ref > 5


def test_cluster_mode_zero_drift_refreshes_nothing():
    m, p, w, prompt = tiny(select_mode=I.SELECT_CLUSTER_TOPK, n_clusters=4, cluster_k=2, tau_upd=-1)
    a = O.PolestarOracle(m, w, p, prompt, rowwise=True)      # row-independent arithmetic: unchanged rows give the same bits
    a.step()
    a.commit(forced=[{"commit": np.zeros(p.block, bool), "suffix": ()}])      # nothing committed: nothing changes
    a.step()
    tr = a.seqs[0].trace
    assert tr["kind"] == "within" and tr["refresh"]
    for l in range(m.n_layers):
        assert not tr["D"][l].any() and len(tr["sel"][l]) == 0


def test_nvfp4_hidden_cache_is_lossy_but_close():
    # Sec. 4.1 "Cluster and Quantize Hidden States": the cached hidden rows are NVFP4 residuals against their
    # cluster's centroid.  Every cached row lies on the codec's grid around its reference, the decode still
    # terminates, and the logits stay close to the unquantised cluster mode (the paper's quantisation ablation
    # reports the same ordering: a small loss).
    kw = dict(select_mode=I.SELECT_CLUSTER_TOPK, n_clusters=4, cluster_k=2, tau_upd=-1, logit_scale=3.0)
    m, p, w, prompt = tiny(**kw)
    m = dataclasses.replace(m)            # (d_model 64: a multiple of the group size 16)
    pq = dataclasses.replace(p, flags=p.flags | O.FLAG_NVFP4_HCACHE)
    a, b = O.PolestarOracle(m, w, p, prompt), O.PolestarOracle(m, w, pq, prompt)
    a.step(); b.step()
    errs = []
    for _ in range(2):       # the entry forward and the first step (later steps may already take other decisions)
        sa, sb = a.seqs[0], b.seqs[0]
        for l in range(m.n_layers):
            # every cached row is its reference plus a float32 grid value, within the codec's error of the plain row
            assert np.array_equal(sb.Hc[l].astype(np.float32).astype(np.float64), sb.Hc[l])
            if _ == 0:
                res = np.abs(sa.Hc[l] - sb.Z0[l][sb.labels[l]]).reshape(len(sb.win), -1, 16).max(-1, keepdims=True)
                assert (np.abs(sa.Hc[l] - sb.Hc[l]).reshape(len(sb.win), -1, 16) <= res / 6 * 1.07 + 1e-6).all()
        errs.append(np.abs(a.seqs[0].trace["logits"] - b.seqs[0].trace["logits"]).max())
        forced = [dict(commit=i["commit"], suffix=tuple(i["suffix_committed"])) for i in a.commit()]
        b.commit(forced)
        a.step(); b.step()
    assert errs[0] == 0.0 and 0 < errs[1] < 0.1 * np.abs(a.seqs[0].trace["logits"]).max()
    b2 = O.PolestarOracle(m, w, pq, prompt)
    b2.decode()
    assert b2.done and not (b2.tokens() == m.mask_id).any()


@pytest.mark.parametrize("nkv", [1, 2])
def test_entry_forward_matches_a_transformer_built_from_library_primitives(nkv):
    # The composition of the pieces (pre-norm residual wiring, which gain goes where, GQA head mapping, the order of
    # gate and up in SwiGLU, rotary positions, final norm + LM head + logit scale) against the same model written
    # with the tensor library's own primitives: rms_norm, linear, non-causal scaled_dot_product_attention (Eq. 3), and
    # the rotation done as a complex multiplication.  The first forward of a decode is a full-sequence forward.
    import torch
    import torch.nn.functional as F
    m, p, w, prompt = tiny(nkv=nkv, logit_scale=3.0)
    ora = O.PolestarOracle(m, w, p, prompt)
    y = torch.from_numpy(ora.seqs[0].y.copy()).long()
    ora.step()
    tr = ora.seqs[0].trace
    assert tr["kind"] == "entry_full"
    act = torch.from_numpy(np.asarray(ora.seqs[0].act)).long()
    N, nh, dh = len(y), m.n_heads, m.head_dim
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    pos = torch.arange(N, dtype=torch.float64)
    inv = m.rope_theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    rot = torch.polar(torch.ones(N, dh // 2, dtype=torch.float64), pos[:, None] * inv[None, :])[:, None, :]

    def rotate(u):          # [N, H, dh]: pair i = (u[i], u[i + dh/2]) as one complex number
        c = torch.complex(u[..., :dh // 2], u[..., dh // 2:]) * rot
        return torch.cat([c.real, c.imag], -1)

    x = t(w["embed"])[y]
    hidden = [x[act]]
    for wl in w["layers"]:
        a = F.rms_norm(x, (m.d_model,), t(wl["norm1"]), m.rms_eps)
        q = rotate(F.linear(a, t(wl["wq"])).view(N, nh, dh))
        k = rotate(F.linear(a, t(wl["wk"])).view(N, nkv, dh)).repeat_interleave(nh // nkv, dim=1)
        v = F.linear(a, t(wl["wv"])).view(N, nkv, dh).repeat_interleave(nh // nkv, dim=1)
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None])[0]
        x1 = x + F.linear(o.transpose(0, 1).reshape(N, nh * dh), t(wl["wo"]))
        f = F.rms_norm(x1, (m.d_model,), t(wl["norm2"]), m.rms_eps)
        x = x1 + F.linear(F.silu(F.linear(f, t(wl["wg"]))) * F.linear(f, t(wl["wu"])), t(wl["wd"]))
        hidden.append(x[act])
    logits = F.linear(F.rms_norm(x[act], (m.d_model,), t(w["final_norm"]), m.rms_eps), t(w["lm_head"])) * p.logit_scale
    for l, h in enumerate(hidden):
        assert np.allclose(tr["x_act"][l], h.numpy(), atol=1e-10, rtol=1e-9), f"hidden l{l}"
    assert np.allclose(tr["logits"], logits.numpy(), atol=1e-9, rtol=1e-9)
    # a mistake in the wiring would show: swapping gate and up moves the logits far beyond that
    wl = w["layers"][0]
    f0 = F.rms_norm(hidden[0], (m.d_model,), t(wl["norm2"]), m.rms_eps)
    assert not np.allclose((F.silu(F.linear(f0, t(wl["wg"]))) * F.linear(f0, t(wl["wu"]))).numpy(),
                           (F.silu(F.linear(f0, t(wl["wu"]))) * F.linear(f0, t(wl["wg"]))).numpy(), atol=1e-3)
