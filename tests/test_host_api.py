"""Host-side checks that need no GPU: the C-ABI library loads, exports every declared symbol,
sizes workspaces sensibly and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from oracle import polestar_oracle as O
from paper_2607_14107_b200 import binding as Bd
from paper_2607_14107_b200 import build as build_mod
from paper_2607_14107_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return Bd.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "polestar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(polestar_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(Bd.EXPORTS) == names


def test_workspace_bytes(lib):
    for name, lo, hi in [("c1", 1e6, 5e8), ("c2", 1e8, 5e9), ("c3", 5e8, 2e10), ("c4", 1e10, 6e10)]:
        m, p = I.config(name)
        n = Bd.polestar_workspace_bytes(m, p)
        assert lo < n < hi, (name, n)
    m, p = I.config("c1")
    p.gen_len = 65                      # not a multiple of the block
    assert Bd.polestar_workspace_bytes(m, p) == 0
    m, p = I.config("c1")
    m.n_heads = 3                       # not a multiple of the kv heads
    assert Bd.polestar_workspace_bytes(m, p) == 0


def test_workspace_shrinks_with_centroid_proxies_and_the_nvfp4_cache(lib):
    # Sec. 4.1: stored attention rows per cluster instead of per window row, hidden rows as 4-bit residuals with one
    # scale byte per 16 channels (9/64 of the fp32 bytes)
    import dataclasses
    m, p = I.config("c4")
    plain = Bd.polestar_workspace_bytes(m, p)
    pc = dataclasses.replace(p, select_mode=I.SELECT_CLUSTER_TOPK)
    proxies = Bd.polestar_workspace_bytes(m, pc)
    assert plain - proxies > 10e9, (plain, proxies)
    pq = dataclasses.replace(pc, flags=pc.flags | I.FLAG_NVFP4_HCACHE)
    quantised = Bd.polestar_workspace_bytes(m, pq)
    W_max = max(sum(len(part) for part in O.window_positions(p, b)) for b in range(p.gen_len // p.block))
    rows = m.n_layers * p.batch * W_max
    saved = rows * m.d_model * 4 * (1 - 9 / 64) - m.n_layers * p.batch * pc.n_clusters * m.d_model * 4
    assert abs((proxies - quantised) - saved) < 0.02 * saved + 4096, (proxies - quantised, saved)
    # the flag needs the cluster mode (the residuals' reference rows are the centroids)
    assert Bd.polestar_workspace_bytes(m, dataclasses.replace(p, flags=p.flags | I.FLAG_NVFP4_HCACHE)) == 0


def test_init_rejects_bad_arguments_before_using_the_device(lib):
    m, p = I.config("c1")
    cm, cp = Bd.c_model(m), Bd.c_params(p)
    ctx = C.c_void_p(123)
    assert lib.polestar_init(C.byref(ctx), C.byref(cm), None, C.byref(cp), None, None, 0, None) == Bd.E_INVAL
    assert ctx.value is None
    assert lib.polestar_init(None, C.byref(cm), None, C.byref(cp), None, None, 0, None) == Bd.E_INVAL
    assert lib.polestar_step(None, None) == Bd.E_INVAL
    assert lib.polestar_commit(None, None) == Bd.E_INVAL
    assert lib.polestar_tokens(None, None) == Bd.E_INVAL
    lib.polestar_destroy(None)


def test_init_charges_the_alignment_loss_to_the_callers_buffer(lib):
    # the plan starts at the next 1024-byte boundary: a buffer that is too small once those bytes are lost must be
    # refused (E_NOSPACE) before anything is written; polestar_workspace_bytes() itself suffices for any
    # 256-byte aligned base.  Fake pointers: the checks run before the device or any pointer is touched.
    m, p = I.config("c1")
    cm, cp = Bd.c_model(m), Bd.c_params(p)
    need = lib.polestar_workspace_bytes(C.byref(cm), C.byref(cp))
    L = m.n_layers
    fake = (C.c_void_p * L)(*([0x1000] * L))
    cw = Bd.CWeights(0x1000, 0x1000, 0x1000, fake, fake, fake, fake, fake, fake)
    prompt = (C.c_int32 * (p.batch * p.prompt_len))(*([1] * (p.batch * p.prompt_len)))
    ctx = C.c_void_p()
    base = 0x7000000100                 # 256 mod 1024: 768 bytes are lost to the alignment
    assert base % 1024 == 256
    assert lib.polestar_init(C.byref(ctx), C.byref(cm), C.byref(cw), C.byref(cp), prompt, C.c_void_p(base),
                             need - 1024 + 767, None) == Bd.E_NOSPACE
    assert lib.polestar_init(C.byref(ctx), C.byref(cm), C.byref(cw), C.byref(cp), prompt, C.c_void_p(base + 0x300),
                             need - 1025, None) == Bd.E_NOSPACE
    assert lib.polestar_init(C.byref(ctx), C.byref(cm), C.byref(cw), C.byref(cp), prompt, C.c_void_p(base + 1),
                             need, None) == Bd.E_INVAL         # not 256-byte aligned
    assert ctx.value is None


def test_confidence_entry_points_check_alignment_and_empty_input(lib):
    ok = C.c_void_p(0x7000001000)
    # vocabulary a multiple of four: rows are read with 16-byte loads, the base must be 16-byte aligned
    for fn, extra in ((lib.polestar_k_confidence, (ok, 1 << 20, None)), (lib.polestar_k_confidence_noalloc, (None,))):
        assert fn(C.c_void_p(0x7000001004), 2, 1024, 1023, ok, ok, *extra) == Bd.E_INVAL
        assert fn(None, 2, 1024, 1023, ok, ok, *extra) == Bd.E_INVAL
        assert fn(None, 0, 1024, 1023, None, None, *extra) == Bd.OK          # no rows: a no-op, null pointers allowed
        assert fn(ok, -1, 1024, 1023, ok, ok, *extra) == Bd.E_INVAL
    assert lib.polestar_k_confidence_noalloc(ok, Bd.NOALLOC_MAX_ROWS + 1, 1024, 1023, ok, ok, None) == Bd.E_NOSPACE
    assert lib.polestar_reload_env() == Bd.OK


def test_kernel_entry_points_validate(lib):
    assert lib.polestar_k_select(None, 1, 96, 0, 1, 0.0, 0.0, None, None, None) == Bd.E_INVAL
    assert lib.polestar_k_attention(None, None, None, None, None, None, None, 1, 1, 1, 1, 64, 0, None) == Bd.E_INVAL
    assert lib.polestar_k_hidden_delta(None, None, None, 1, 8, 0, None) == Bd.E_INVAL
    assert lib.polestar_k_refresh_scratch_bytes(0, 1, 1, 1, 1, 1) == 0
    assert lib.polestar_k_refresh_scratch_bytes(1, 128, 4096, 32, 32, 128) > 128 * 4096 * 2


def test_strerror(lib):
    assert lib.polestar_strerror(0) == b"ok"
    for code in range(-7, 0):
        if code != Bd.E_CUDA:
            assert len(lib.polestar_strerror(code)) > 3


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    m, p = I.config("c1")
    with pytest.raises(Bd.PolestarError):
        Bd.Polestar(m, {}, p, [[0] * p.prompt_len])


def test_pack_weights_layout():
    import torch
    m = I.ModelCfg(1, 16, 2, 1, 8, 24, 32)
    w = I.make_weights(m)
    pk = Bd.pack_weights(m, w, device="cpu")
    l = w["layers"][0]
    qkv = pk["wqkv"][0]
    assert qkv.shape == (2 * 8 + 2 * 8, 16)
    # head 1 of q: packed row 2i = logical row i, 2i+1 = logical row i + 4
    assert torch.equal(qkv[8 + 0], l["wq"][8 + 0]) and torch.equal(qkv[8 + 1], l["wq"][8 + 4])
    assert torch.equal(qkv[8 + 6], l["wq"][8 + 3]) and torch.equal(qkv[8 + 7], l["wq"][8 + 7])
    assert torch.equal(qkv[16 + 1], l["wk"][4]) and torch.equal(qkv[24:], l["wv"])
    gu = pk["w_gate_up"][0]
    assert torch.equal(gu[0], l["wg"][0]) and torch.equal(gu[1], l["wu"][0]) and torch.equal(gu[47], l["wu"][23])
    # interleaving is a permutation of the head dimension: q.k is unchanged
    x = torch.randn(16)
    qa, ka = l["wq"][:8] @ x, l["wk"] @ x
    qb, kb = qkv[:8] @ x, qkv[16:24] @ x
    assert torch.allclose(qa @ ka, qb @ kb, atol=1e-6)
    # tile-major storage of bf16 GEMM weights: block (o / 128, i / 64) is contiguous
    wt = torch.arange(512 * 128, dtype=torch.float32).view(512, 128).to(torch.bfloat16)
    tm = Bd.tile_major(wt)
    assert torch.equal(tm.flatten()[:64], wt[0, :64]) and torch.equal(tm.flatten()[64:128], wt[1, :64])
    assert torch.equal(tm.flatten()[256 * 64:256 * 64 + 64], wt[0, 64:128])
    assert torch.equal(tm.flatten()[2 * 256 * 64:2 * 256 * 64 + 64], wt[256, :64])
    assert torch.equal(Bd.untile(tm), wt)
    assert torch.equal(Bd.tile_major(wt.float()), wt.float())          # fp32 stays row-major


def test_generator_is_device_independent_and_sliceable():
    import torch
    key = I.tensor_key(0, 3, I.T_WO)
    a = I.normal_tensor(key, (64, 33), 0.02)
    b = I.normal_range(key, 64 * 33 - 100, 100, 0.02)
    assert torch.equal(a.flatten()[-100:], b)
    assert abs(a.std().item() - 0.02) < 2e-3 and abs(a.mean().item()) < 2e-3
    ids = I.make_prompt(*I.config("c2"))
    assert ids.shape == (1, 256) and int(ids.max()) < 126463 and int(ids.min()) >= 0
