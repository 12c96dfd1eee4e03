"""Each CUDA kernel of the path against the matching oracle function, through the C ABI."""
import math

import numpy as np
import pytest
import torch

from oracle import polestar_oracle as O
from paper_2607_14107_b200 import binding as Bd
from paper_2607_14107_b200 import inputs as I

pytestmark = pytest.mark.gpu


def bf16_np(t):
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def rnd(shape, key, std=1.0, dtype=torch.float32):
    return I.normal_tensor(I.tensor_key(77, -1, key), shape, std, dtype, "cpu")


# ------------------------------------------------------------------ attention + drift (a1, a5)
@pytest.mark.parametrize("dtype,R,N,nh,nkv,dh", [
    (torch.float32, 5, 37, 4, 4, 64),          # ragged everything
    (torch.float32, 33, 128, 4, 2, 64),
    (torch.bfloat16, 16, 512, 4, 4, 128),      # one tile
    (torch.bfloat16, 37, 200, 4, 2, 128),      # ragged rows and keys, GQA
    (torch.bfloat16, 128, 512, 2, 2, 128),     # window + block rows of the 8B shape
    (torch.bfloat16, 3, 31, 2, 1, 128),        # fewer keys than one warp tile
])
def test_attention_drift_matches_oracle(dtype, R, N, nh, nkv, dh):
    check_attention(dtype, R, N, nh, nkv, dh)


@pytest.mark.parametrize("variant,R,N,nh,nkv", [
    (1, 37, 200, 4, 2),            # two-pass kernel, ragged
    (1, 40, 1100, 2, 1),           # two-pass kernel beyond the single-pass key limit
    (2, 37, 200, 4, 2), (3, 37, 200, 4, 2), (4, 37, 1000, 2, 1),     # single-pass variants
    (5, 150, 1100, 2, 1),          # 64-row tiles: three row tiles (last ragged), 18 key tiles (last ragged)
    (5, 5, 37, 2, 2),              # 64-row tiles, fewer rows and keys than one tile
    (0, 200, 2048, 8, 8),          # automatic choice at a long sequence
    (6, 32, 512, 4, 4), (6, 21, 300, 4, 2), (6, 5, 37, 2, 2),        # keys split over a cluster of two CTAs
    (7, 32, 1000, 2, 1), (7, 16, 512, 2, 2),
    (0, 32, 512, 2, 2),            # automatic choice for one block of rows
    # tensor-core kernel (tcgen05, S and O in tensor memory, key ranges over a cluster)
    (8, 128, 512, 2, 2),           # one full row tile, four key ranges
    (8, 32, 512, 4, 4),            # a block of active rows
    (8, 5, 37, 2, 2),              # fewer rows and keys than one tile, no cluster
    (8, 37, 200, 4, 2),            # ragged rows and keys, GQA, two key ranges
    (8, 150, 1100, 2, 1),          # two row tiles, two S tiles per CTA, five key ranges (last one a single ragged tile)
    (8, 200, 2048, 8, 8),          # the long-sequence shape: 2 x 8 key tiles
    (8, 130, 1024, 2, 2),          # eight key ranges of one tile
    (8, 64, 402, 2, 1),            # key count not a multiple of four (scalar access to the stored rows)
    # streaming tensor-core kernel (one CTA per row tile and head walks the key tiles twice)
    (9, 5, 37, 2, 2),              # fewer rows and keys than one tile
    (9, 128, 512, 2, 2),           # one full row tile, four key tiles
    (9, 37, 200, 4, 2),            # ragged rows and keys, GQA
    (9, 150, 1100, 2, 1),          # two row tiles, nine key tiles (odd count: the accumulators swap roles between the passes)
    (9, 200, 2048, 8, 8),          # the long-sequence shape
    (9, 64, 402, 2, 1),            # key count not a multiple of four
    (9, 70, 3000, 2, 2),           # more keys than the cluster kernel takes
])
def test_attention_kernel_variants(monkeypatch, variant, R, N, nh, nkv):
    monkeypatch.setenv("POLESTAR_ATTN_KERNEL", str(variant))
    Bd.polestar_reload_env()           # the stand-alone calls read the switches once, not per launch
    check_attention(torch.bfloat16, R, N, nh, nkv, 128)


def check_attention(dtype, R, N, nh, nkv, dh):
    q = rnd((R, nh * dh), 1, 1.0, dtype).cuda()
    k = rnd((N, nkv * dh), 2, 1.0, dtype).cuda()
    v = rnd((N, nkv * dh), 3, 1.0, dtype).cuda()
    prev_s = rnd((R, nh, N), 4, 1.0).double()
    prev = (prev_s - torch.logsumexp(prev_s, -1, keepdim=True)).float()
    prev_dev = prev.clone().cuda()
    lse_dev = torch.zeros((R, nh), device="cuda")          # stored pair (row, lse): log-probability = row - lse
    kl = torch.full((R, nh), -1.0, device="cuda")
    out = torch.zeros((R, nh * dh), dtype=dtype, device="cuda")
    Bd.polestar_k_attention(q, k, v, prev_dev, lse_dev, kl, out, nh, nkv, dh)
    torch.cuda.synchronize()
    qn, kn, vn = bf16_np(q).reshape(R, nh, dh), bf16_np(k).reshape(N, nkv, dh), bf16_np(v).reshape(N, nkv, dh)
    logp = O.attn_logp_rows(qn, kn)
    tol = 1e-4 if dtype == torch.float32 else 2e-2
    rp = O.bf16_round if dtype == torch.bfloat16 else (lambda x: x)
    ref_out = O.attn_out_rows(logp, vn, rp)
    ref_kl = np.sum(np.exp(logp) * (logp - prev.double().numpy()), -1)
    stored = prev_dev.cpu().double().numpy() - lse_dev.cpu().double().numpy()[..., None]
    assert np.allclose(stored, logp, atol=2e-4, rtol=1e-5)       # stored rows = new log-probs
    assert np.allclose(kl.cpu().numpy(), ref_kl, atol=1e-3 * max(1.0, np.abs(ref_kl).max()), rtol=1e-3)
    assert np.allclose(bf16_np(out), ref_out, atol=tol, rtol=tol)
    # Eq. 4 invariants: drift against the rows just stored is zero, and KL >= 0
    kl2 = torch.full((R, nh), -1.0, device="cuda")
    Bd.polestar_k_attention(q, k, v, prev_dev, lse_dev, kl2, None, nh, nkv, dh)
    torch.cuda.synchronize()
    assert np.abs(kl2.cpu().numpy()).max() < 1e-5
    if dtype == torch.bfloat16:
        assert (kl2 == 0).all()            # unchanged rows: exactly zero drift (same bits in, same bits out)
    assert (kl.cpu().numpy() > -1e-4).all()
    # Pinsker bound of Appendix B, Prop. 2 with the current value rows
    M = np.linalg.norm(vn, axis=-1).max()
    p_old = np.exp(prev.double().numpy())
    for h in range(nh):
        g = (h * nkv) // nh
        d_out = np.linalg.norm((np.exp(logp[:, h]) - p_old[:, h]) @ vn[:, g], axis=-1)
        assert (d_out <= M * np.sqrt(2 * np.maximum(kl.cpu().numpy()[:, h], 0)) + 1e-3).all()


def test_attention_without_recording():
    R, N, nh, dh = 20, 96, 2, 128
    q = rnd((R, nh * dh), 1, 1.0, torch.bfloat16).cuda()
    k = rnd((N, nh * dh), 2, 1.0, torch.bfloat16).cuda()
    v = rnd((N, nh * dh), 3, 1.0, torch.bfloat16).cuda()
    out = torch.zeros((R, nh * dh), dtype=torch.bfloat16, device="cuda")
    Bd.polestar_k_attention(q, k, v, None, None, None, out, nh, nh, dh)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.float().view(R, nh, dh).permute(1, 0, 2)[None], k.float().view(N, nh, dh).permute(1, 0, 2)[None],
        v.float().view(N, nh, dh).permute(1, 0, 2)[None])[0].permute(1, 0, 2).reshape(R, nh * dh)
    assert torch.allclose(out.float(), ref, atol=2e-2, rtol=2e-2)


@pytest.mark.parametrize("variant,R,N,nh,nkv", [(5, 150, 1100, 2, 1), (5, 64, 2048, 4, 4), (5, 5, 37, 2, 2), (0, 300, 2048, 8, 2),
                                                (9, 150, 1100, 2, 1), (9, 300, 2048, 8, 2), (9, 5, 37, 2, 2), (9, 130, 3000, 2, 2)])
def test_attention_many_rows_single_pass(monkeypatch, variant, R, N, nh, nkv):
    # without stored rows the 64-row-tile kernel makes one pass with a running maximum (probabilities are rounded
    # to bf16 before the final normalisation): same tolerance against the oracle; the streaming kernel (9) normalises
    # before it rounds, with or without stored rows
    monkeypatch.setenv("POLESTAR_ATTN_KERNEL", str(variant))
    Bd.polestar_reload_env()           # the stand-alone calls read the switches once, not per launch
    dh = 128
    q = rnd((R, nh * dh), 1, 1.0, torch.bfloat16).cuda()
    k = rnd((N, nkv * dh), 2, 1.0, torch.bfloat16).cuda()
    v = rnd((N, nkv * dh), 3, 1.0, torch.bfloat16).cuda()
    out = torch.zeros((R, nh * dh), dtype=torch.bfloat16, device="cuda")
    Bd.polestar_k_attention(q, k, v, None, None, None, out, nh, nkv, dh)
    torch.cuda.synchronize()
    qn, kn, vn = bf16_np(q).reshape(R, nh, dh), bf16_np(k).reshape(N, nkv, dh), bf16_np(v).reshape(N, nkv, dh)
    ref = O.attn_out_rows(O.attn_logp_rows(qn, kn), vn, O.bf16_round)
    assert np.allclose(bf16_np(out), ref, atol=2e-2, rtol=2e-2)


# ------------------------------------------------------------------ hidden delta (a1b)
@pytest.mark.parametrize("dtype,rows,d", [(torch.bfloat16, 4096, 4096), (torch.float32, 77, 256), (torch.bfloat16, 1, 8)])
def test_hidden_delta(dtype, rows, d):
    a = rnd((rows, d), 5, 1.0, dtype).cuda()
    b = a.clone()
    b[::3] += rnd((rows, d), 6, 0.5, dtype).cuda()[::3]
    out = torch.empty(rows, device="cuda")
    Bd.polestar_k_hidden_delta(a, b, out)
    ref = ((a.double() - b.double()) ** 2).sum(-1)
    assert torch.allclose(out.double(), ref, rtol=1e-4, atol=1e-6)
    assert (out[1::3] == 0).all()                       # Cor. 1: unchanged rows give exactly zero


# ------------------------------------------------------------------ select + compaction (a2)
@pytest.mark.parametrize("W,batch", [(96, 1), (64, 3), (192, 8), (4096, 2), (1, 1), (1000, 1)])
def test_select_matches_bruteforce(W, batch):
    g = torch.Generator().manual_seed(W * 31 + batch)
    z = torch.randn(batch, W, generator=g)
    drift = torch.exp(z)
    drift[:, ::7] = 0.0                                  # zero-drift rows are never candidates
    if W > 8:
        drift[:, 5] = drift[:, 3]                        # ties: lower index first
    dd = drift.cuda()
    idx = torch.full((batch, W), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(batch, dtype=torch.int32, device="cuda")
    for mode, k, th in [(I.SELECT_TOPK_COUNT, max(1, W // 4), 0.0), (I.SELECT_TOPK_COUNT, W, 0.0),
                        (I.SELECT_TOPK_COUNT, 1, 0.0), (I.SELECT_THRESHOLD, 0, 1.0), (I.SELECT_ALL, 0, 0.0),
                        (I.SELECT_NONE, 0, 0.0), (I.SELECT_TOPK_COUNT, max(1, W // 100), 0.0)]:
        Bd.polestar_k_select(dd, mode, k, th, 0.0, idx, cnt)
        torch.cuda.synchronize()
        for s in range(batch):
            ref = O.select_rows(drift[s].numpy(), mode, k=k, thresh=th, floor=0.0)
            n = int(cnt[s])
            assert n == len(ref), (mode, k, s)
            assert idx[s, :n].cpu().tolist() == ref.tolist()


def test_select_zero_drift_and_nan():
    d = torch.zeros(2, 96, device="cuda")
    d[1, 10] = float("nan")
    idx = torch.zeros((2, 96), dtype=torch.int32, device="cuda")
    cnt = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    Bd.polestar_k_select(d, I.SELECT_TOPK_COUNT, 24, 0.0, 0.0, idx, cnt)
    assert cnt.cpu().tolist() == [0, 0]


# ------------------------------------------------------------------ gathered refresh (a3 + a4)
@pytest.mark.parametrize("P,d,nh,nkv,k,batch", [
    (256, 256, 2, 2, 37, 1), (512, 512, 4, 1, 128, 2), (300, 256, 2, 2, 300, 1),
    (3400, 256, 2, 2, 3300, 4),       # 13200 rows: 312 output tiles > SM count (whole tiles round-robin + stream-K tail)
    (2000, 256, 2, 2, 1700, 2),       # 3400 rows: 27 token tiles (two raster chunks), fewer tiles than SMs
    # the refresh micro-benchmark's own shape (LLaDA-8B layer: d 4096 = 64 k-blocks, 32 x 128 heads, 4096 positions)
    (4096, 4096, 32, 32, 41, 1), (4096, 4096, 32, 32, 1024, 1), (4096, 4096, 32, 32, 410, 8),
])
def test_refresh_chain_matches_oracle(P, d, nh, nkv, k, batch):
    check_refresh_chain(P, d, nh, nkv, k, batch)


@pytest.mark.parametrize("P,d,nh,nkv,k,batch", [
    (300, 256, 2, 2, 300, 1),          # 300 rows: the second pair tile's second half is empty
    (3400, 256, 2, 2, 3300, 4),        # more pair tiles than pairs: whole tiles round-robin + stream-K tail
    (4096, 4096, 32, 32, 410, 8),      # the micro-benchmark's shape, 3280 rows
])
def test_refresh_chain_on_cta_pairs(monkeypatch, P, d, nh, nkv, k, batch):
    # the same projection on CTA pairs (tcgen05 cta_group::2): each CTA of a pair loads half of the weight tile
    monkeypatch.setenv("POLESTAR_GEMM_PAIR_ROWS", "200")
    Bd.polestar_reload_env()           # the stand-alone calls read the switches once, not per launch
    check_refresh_chain(P, d, nh, nkv, k, batch)


def check_refresh_chain(P, d, nh, nkv, k, batch):
    dh = 128
    big = d >= 2048
    dev = "cuda" if big else "cpu"                      # large inputs are generated on the device (same values)
    h, drift = I.make_refresh_inputs(batch, P, d, device=dev)
    drift = drift.cpu()
    m = I.ModelCfg(1, d, nh, nkv, dh, 256 if big else 2 * d, 1024, I.DTYPE_BF16, 1e-5, 500000.0)
    w = I.make_weights(m, seed=5, device=dev)
    packed = Bd.pack_weights(m, w)
    kc0 = I.normal_tensor(I.tensor_key(77, -1, 8), (batch, P, nkv * dh), 1.0, torch.bfloat16, dev)
    vc0 = I.normal_tensor(I.tensor_key(77, -1, 9), (batch, P, nkv * dh), 1.0, torch.bfloat16, dev)
    kc, vc = kc0.clone().cuda(), vc0.clone().cuda()
    idx = torch.zeros((batch, k), dtype=torch.int32, device="cuda")
    cnt = torch.zeros(batch, dtype=torch.int32, device="cuda")
    full_idx = torch.zeros((batch, P), dtype=torch.int32, device="cuda")
    Bd.polestar_k_select(drift.cuda(), I.SELECT_TOPK_COUNT, k, 0.0, 0.0, full_idx, cnt)
    idx.copy_(full_idx[:, :k])
    q_out = torch.zeros((batch, k, nh * dh), dtype=torch.bfloat16, device="cuda")
    scratch = torch.empty(Bd.polestar_k_refresh_scratch_bytes(batch, k, d, nh, nkv, dh) + 1024, dtype=torch.uint8, device="cuda")
    off = (-scratch.data_ptr()) % 1024
    Bd.polestar_k_refresh(h.cuda(), idx, cnt, packed["wqkv"][0], packed["norm1"][0], kc, vc, q_out, k, nh, nkv, dh,
                          m.rms_eps, m.rope_theta, scratch[off:])
    assert Bd.polestar_k_refresh_status(scratch[off:], batch, k, d, dh) == Bd.OK      # synchronises
    assert cnt.cpu().tolist() == [k] * batch
    wl = {n: t.detach().to("cpu", torch.float32).numpy() for n, t in w["layers"][0].items() if n in ("wq", "wk", "wv", "norm1")}
    inv = np.argsort(Bd.rope_interleave_index(dh).numpy())
    kc_h, vc_h, kc0_h, vc0_h = kc.cpu(), vc.cpu(), kc0.cpu(), vc0.cpu()
    for s in range(batch):
        ridx, q_ref, K_ref, V_ref = O.refresh_chain(bf16_np(h[s]), drift[s].numpy(), k, wl["wq"], wl["wk"], wl["wv"],
                                                    wl["norm1"], m.rms_eps, m.rope_theta, nh, nkv, dh,
                                                    bf16_np(kc0_h[s]).reshape(P, nkv, dh), bf16_np(vc0_h[s]).reshape(P, nkv, dh))
        assert idx[s, :int(cnt[s])].cpu().tolist() == ridx.tolist()
        Kg = bf16_np(kc_h[s]).reshape(P, nkv, dh)
        Vg = bf16_np(vc_h[s]).reshape(P, nkv, dh)
        Kg_log = Kg[..., inv]
        assert np.allclose(Kg_log[ridx], K_ref[ridx], atol=2e-2, rtol=2e-2)
        assert np.allclose(Vg[ridx], V_ref[ridx], atol=2e-2, rtol=2e-2)
        qg = bf16_np(q_out[s]).reshape(k, nh, dh)[..., inv]
        assert np.allclose(qg[:len(ridx)], q_ref, atol=2e-2, rtol=2e-2)
        rest = np.setdiff1d(np.arange(P), ridx)          # rows not selected keep their bits
        assert torch.equal(kc_h[s][rest], kc0_h[s][rest]) and torch.equal(vc_h[s][rest], vc0_h[s][rest])


# ------------------------------------------------------------------ confidence (a6, first half)
@pytest.mark.parametrize("rows,V", [(32, 126464), (7, 1024), (1, 50)])
def test_confidence_matches_oracle(rows, V):
    logits = rnd((rows, V), 11, 3.0)
    mask_id = V - 1
    logits[0, mask_id] = 50.0                            # [MASK] must never be predicted
    if rows > 1:
        logits[1, 3] = logits[1, 9] = 40.0               # tie: lowest id
    yhat = torch.zeros(rows, dtype=torch.int32, device="cuda")
    conf = torch.zeros(rows, device="cuda")
    scratch = torch.empty(rows * 512, dtype=torch.uint8, device="cuda")
    Bd.polestar_k_confidence(logits.cuda(), mask_id, yhat, conf, scratch)
    ry, rc = O.confidence_rows(logits.numpy(), mask_id)
    assert yhat.cpu().tolist() == ry.tolist()
    assert np.allclose(conf.cpu().numpy(), rc, rtol=1e-4, atol=1e-7)


# ------------------------------------------------------------------ empty inputs
def test_empty_inputs_are_noops():
    dev = "cuda"
    cnt = torch.full((2,), -7, dtype=torch.int32, device=dev)
    Bd.polestar_k_select(torch.zeros((2, 0), device=dev), I.SELECT_TOPK_COUNT, 3, 0.0, 0.0,
                         torch.zeros((2, 0), dtype=torch.int32, device=dev), cnt)
    assert cnt.tolist() == [0, 0]
    drift = torch.rand(2, 100, device=dev)
    idx = torch.full((2, 100), -7, dtype=torch.int32, device=dev)
    Bd.polestar_k_select(drift, I.SELECT_TOPK_COUNT, 0, 0.0, 0.0, idx, cnt)          # budget 0
    assert cnt.tolist() == [0, 0]
    e = torch.zeros((0, 256), dtype=torch.bfloat16, device=dev)
    Bd.polestar_k_hidden_delta(e, e, torch.zeros(0, device=dev))
    Bd.polestar_k_confidence(torch.zeros((0, 1024), device=dev), 1023, torch.zeros(0, dtype=torch.int32, device=dev),
                             torch.zeros(0, device=dev), torch.empty(4096, dtype=torch.uint8, device=dev))
    k = torch.zeros((10, 256), dtype=torch.bfloat16, device=dev)
    Bd.polestar_k_attention(e, k, k, None, None, None, torch.zeros((0, 256), dtype=torch.bfloat16, device=dev), 2, 2, 128)
    with pytest.raises(Bd.PolestarError):                                             # no keys: softmax over nothing
        Bd.polestar_k_attention(torch.zeros((4, 256), dtype=torch.bfloat16, device=dev), e, e, None, None, None,
                                torch.zeros((4, 256), dtype=torch.bfloat16, device=dev), 2, 2, 128)
    torch.cuda.synchronize()


def test_refresh_with_zero_selected_rows_touches_nothing():
    P, d, nh, nkv, dh, batch, k = 256, 256, 2, 2, 128, 2, 16
    m = I.ModelCfg(1, d, nh, nkv, dh, 2 * d, 1024, I.DTYPE_BF16, 1e-5, 500000.0)
    packed = Bd.pack_weights(m, I.make_weights(m, seed=5))
    h, _ = I.make_refresh_inputs(batch, P, d)
    kc0 = rnd((batch, P, nkv * dh), 8, 1.0, torch.bfloat16)
    kc, vc = kc0.clone().cuda(), kc0.clone().cuda()
    idx = torch.zeros((batch, k), dtype=torch.int32, device="cuda")
    cnt = torch.zeros(batch, dtype=torch.int32, device="cuda")                        # nothing selected
    scratch = torch.empty(Bd.polestar_k_refresh_scratch_bytes(batch, k, d, nh, nkv, dh) + 1024, dtype=torch.uint8, device="cuda")
    off = (-scratch.data_ptr()) % 1024
    Bd.polestar_k_refresh(h.cuda(), idx, cnt, packed["wqkv"][0], packed["norm1"][0], kc, vc, None, k, nh, nkv, dh,
                          m.rms_eps, m.rope_theta, scratch[off:])
    torch.cuda.synchronize()
    assert torch.equal(kc.cpu(), kc0) and torch.equal(vc.cpu(), kc0)


@pytest.mark.parametrize("rows,d", [(1, 128), (37, 256), (300, 4096)])
def test_nvfp4_residual_codec_bit_exact(rows, d):
    # Appendix "Quantization Format": E2M1 codes with one E4M3 scale per 16 channels, float32 arithmetic on both
    # sides, identical inputs -> identical codes, scales and stored values
    g = torch.Generator().manual_seed(rows * 131 + d)
    ref = torch.randn(rows, d, generator=g)
    mag = torch.exp(torch.randn(rows, d // 16, 1, generator=g) * 3.0).expand(rows, d // 16, 16).reshape(rows, d)
    x = ref + torch.randn(rows, d, generator=g) * mag * 0.05
    x[0, :16] = ref[0, :16]                                   # an all-zero group
    x[0, 16:32] = ref[0, 16:32] + 1e-7                         # below the smallest subnormal scale
    x[0, 32:48] = ref[0, 32:48] + 1e5                          # saturates the E4M3 scale at 448
    grid = torch.tensor([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    mids = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0])
    ref[0, 48:64] = 0.0                                        # exact grid points and midpoints at scale 1
    x[0, 48:56], x[0, 56:64] = grid, -mids
    xd, rd = x.cuda(), ref.cuda()
    codes = torch.empty(rows, d // 2, dtype=torch.uint8, device="cuda")
    scales = torch.empty(rows, d // 16, dtype=torch.uint8, device="cuda")
    deq = torch.empty(rows, d, device="cuda")
    Bd.polestar_k_nvfp4_residual(xd, rd, codes, scales, deq)
    torch.cuda.synchronize()
    res = (x - ref).numpy()
    o_codes, o_scale = O.nvfp4_quantize(res)
    c = codes.cpu().numpy()
    got = np.stack([c & 15, c >> 4], axis=-1).reshape(rows, d)
    o_mag = (o_codes & 7)
    # the sign bit of a zero magnitude carries no information
    assert np.array_equal(got & 7, o_mag)
    nz = o_mag > 0
    assert np.array_equal((got & 8)[nz], (o_codes & 8)[nz])
    sc = scales.cpu().view(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(sc, o_scale)
    assert np.array_equal(deq.cpu().numpy().astype(np.float64), O.residual_nvfp4_roundtrip(x.numpy(), ref.numpy()))


def test_bounded_wait_gives_up_with_an_error_code():
    # every device-side wait of the library is bounded; this is that wait alone, on a counter nobody advances: it
    # ends after its limit (~1 ms here) with E_TIMEOUT, and the context goes on working
    counter = torch.zeros(1, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert Bd.polestar_k_wait_probe(counter, 1, 2_000_000, status) == Bd.E_TIMEOUT
    assert int(status.item()) == 1
    counter += 1
    assert Bd.polestar_k_wait_probe(counter, 1, 2_000_000, status) == Bd.OK
    assert int(status.item()) == 0
    x = torch.arange(8, device="cuda").sum().item()              # the context is intact
    assert x == 28
