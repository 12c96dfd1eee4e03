"""ctypes binding of libpolestar.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and streams.  Every step of the decoding path
runs inside the library's CUDA kernels; there is no Python or CPU fallback: if
the shared library is missing, or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional

import numpy as np
import torch

from . import inputs as I

_HERE = os.path.dirname(os.path.abspath(__file__))
# POLESTAR_LIB selects another build of the same library (e.g. the time-stamping build of `build.py --trace`)
LIB_PATH = os.environ.get("POLESTAR_LIB") or os.path.join(_HERE, "libpolestar.so")

OK, E_INVAL, E_STATE, E_NOSPACE, E_CUDA, E_NONFINITE, E_TIMEOUT, E_DONE = 0, -1, -2, -3, -4, -5, -6, -7

READ_LOGITS, READ_CONF, READ_YHAT, READ_DELTA, READ_DRIFT, READ_SEL_COUNT, READ_SEL_IDX = 1, 2, 3, 4, 5, 6, 7
READ_HIDDEN, READ_KCACHE, READ_VCACHE, READ_HCACHE, READ_COMMIT, READ_PPREV, READ_SUFFIX = 8, 9, 10, 11, 12, 13, 14
READ_DRIFT_DELTA, READ_TAU_D, READ_THETA, READ_THETA_COUNT, READ_OWN_COMMIT, READ_LABELS = 15, 16, 17, 18, 19, 20
READ_TRACE_KERNELS, READ_TRACE_GEMM = 98, 99
FORCE_SELECT, FORCE_COMMIT, FORCE_CLEAR, FORCE_TOKENS, FORCE_LABELS, FORCE_HCODES = 1, 2, 3, 4, 5, 6
FLAG_SIMT_GEMM, FLAG_PROMPT_DEVICE, FLAG_PROFILE, FLAG_NVFP4_HCACHE = 1 << 5, 1 << 6, 1 << 7, 1 << 8
PROF_FAMILIES = ["gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head", "attention", "stage", "select",
                 "confidence", "commit", "misc"]

EXPORTS = [
    "polestar_workspace_bytes", "polestar_init", "polestar_step", "polestar_commit", "polestar_tokens",
    "polestar_read", "polestar_force", "polestar_profile", "polestar_destroy", "polestar_strerror",
    "polestar_reload_env", "polestar_k_refresh_status", "polestar_k_nvfp4_residual", "polestar_k_wait_probe",
    "polestar_k_attention", "polestar_k_hidden_delta", "polestar_k_select",
    "polestar_k_refresh_scratch_bytes", "polestar_k_refresh", "polestar_k_confidence",
    "polestar_k_confidence_noalloc", "polestar_sm_count",
]


class PolestarError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"polestar error {code}: {msg}")
        self.code = code


class CModel(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn",
                                         "vocab", "dtype")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("mask_id", C.c_int32), ("eos_id", C.c_int32)]


class CWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
                ("w_gate_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p)),
                ("norm1", C.POINTER(C.c_void_p)), ("norm2", C.POINTER(C.c_void_p))]


class CParams(C.Structure):
    _fields_ = [("batch", C.c_int32), ("prompt_len", C.c_int32), ("gen_len", C.c_int32), ("block", C.c_int32),
                ("max_steps", C.c_int32), ("win_prefix_blocks", C.c_int32), ("win_suffix_blocks", C.c_int32),
                ("full_entry_period", C.c_int32), ("select_mode", C.c_int32), ("select_frac", C.c_float),
                ("select_k", C.c_int32), ("select_thresh", C.c_float), ("drift_floor", C.c_float),
                ("tau_upd", C.c_int32), ("hist", C.c_int32), ("tau_s", C.c_float), ("alpha", C.c_float),
                ("tau_suffix", C.c_float), ("logit_scale", C.c_float), ("flags", C.c_uint32),
                ("n_clusters", C.c_int32), ("cluster_k", C.c_int32), ("kmeans_iters", C.c_int32)]


class CStepInfo(C.Structure):
    _fields_ = [("kind", C.c_int32), ("block_index", C.c_int32), ("n_refreshing", C.c_int32), ("rows", C.c_int32),
                ("forwards", C.c_int64)]


class CCommitInfo(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_committed", "n_by_conf", "n_by_drift", "n_by_quota", "n_suffix", "n_eos",
                                         "rows_refreshed", "block_index", "block_done", "all_done")] + \
               [("forwards", C.c_int64), ("generated", C.c_int64), ("generated_non_eos", C.c_int64),
                ("launches", C.c_int64)]


_lib = None


def load():
    """Load libpolestar.so (built in-tree by `build.py`).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise PolestarError(E_INVAL, f"{LIB_PATH} not built: run `python -m paper_2607_14107_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, f32, sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
    lib.polestar_workspace_bytes.restype = sz
    lib.polestar_workspace_bytes.argtypes = [C.POINTER(CModel), C.POINTER(CParams)]
    lib.polestar_init.restype = C.c_int
    lib.polestar_init.argtypes = [C.POINTER(vp), C.POINTER(CModel), C.POINTER(CWeights), C.POINTER(CParams),
                                  C.POINTER(i32), vp, sz, vp]
    lib.polestar_step.restype = C.c_int
    lib.polestar_step.argtypes = [vp, C.POINTER(CStepInfo)]
    lib.polestar_commit.restype = C.c_int
    lib.polestar_commit.argtypes = [vp, C.POINTER(CCommitInfo)]
    lib.polestar_tokens.restype = C.c_int
    lib.polestar_tokens.argtypes = [vp, C.POINTER(i32)]
    lib.polestar_read.restype = C.c_int
    lib.polestar_read.argtypes = [vp, i32, i32, vp, sz]
    lib.polestar_force.restype = C.c_int
    lib.polestar_force.argtypes = [vp, i32, i32, C.POINTER(i32), i32]
    lib.polestar_profile.restype = C.c_int
    lib.polestar_profile.argtypes = [vp, C.POINTER(C.c_double), i32]
    lib.polestar_destroy.restype = None
    lib.polestar_destroy.argtypes = [vp]
    lib.polestar_strerror.restype = C.c_char_p
    lib.polestar_strerror.argtypes = [C.c_int]
    lib.polestar_k_attention.restype = C.c_int
    lib.polestar_k_attention.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp]
    lib.polestar_k_hidden_delta.restype = C.c_int
    lib.polestar_k_hidden_delta.argtypes = [vp, vp, vp, i32, i32, i32, vp]
    lib.polestar_k_select.restype = C.c_int
    lib.polestar_k_select.argtypes = [vp, i32, i32, i32, i32, f32, f32, vp, vp, vp]
    lib.polestar_k_refresh_scratch_bytes.restype = sz
    lib.polestar_k_refresh_scratch_bytes.argtypes = [i32] * 6
    lib.polestar_k_refresh.restype = C.c_int
    lib.polestar_k_refresh.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, f32, f32,
                                       i32, vp, sz, vp]
    lib.polestar_k_confidence.restype = C.c_int
    lib.polestar_k_confidence.argtypes = [vp, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.polestar_k_confidence_noalloc.restype = C.c_int
    lib.polestar_k_confidence_noalloc.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    lib.polestar_sm_count.restype = C.c_int
    lib.polestar_sm_count.argtypes = []
    lib.polestar_k_nvfp4_residual.restype = C.c_int
    lib.polestar_k_nvfp4_residual.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    lib.polestar_k_wait_probe.restype = C.c_int
    lib.polestar_k_wait_probe.argtypes = [vp, C.c_uint32, C.c_int64, vp, vp]
    lib.polestar_reload_env.restype = C.c_int
    lib.polestar_reload_env.argtypes = []
    lib.polestar_k_refresh_status.restype = C.c_int
    lib.polestar_k_refresh_status.argtypes = [vp, sz, i32, i32, i32, i32, vp]
    _lib = lib
    return lib


def _check(code: int):
    if code != OK:
        raise PolestarError(code, load().polestar_strerror(code).decode())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def c_model(m: I.ModelCfg) -> CModel:
    return CModel(m.n_layers, m.d_model, m.n_heads, m.n_kv_heads, m.head_dim, m.d_ffn, m.vocab, m.dtype,
                  m.rms_eps, m.rope_theta, m.mask_id, m.eos_id)


def c_params(p: I.Params) -> CParams:
    return CParams(p.batch, p.prompt_len, p.gen_len, p.block, p.max_steps, p.win_prefix_blocks, p.win_suffix_blocks,
                   p.full_entry_period, p.select_mode, p.select_frac, p.select_k, p.select_thresh, p.drift_floor,
                   p.tau_upd, p.hist, p.tau_s, p.alpha, p.tau_suffix, p.logit_scale, p.flags,
                   p.n_clusters, p.cluster_k, p.kmeans_iters)


def polestar_workspace_bytes(m: I.ModelCfg, p: I.Params) -> int:
    cm, cp = c_model(m), c_params(p)
    return int(load().polestar_workspace_bytes(C.byref(cm), C.byref(cp)))


# ------------------------------------------------------------------------------------------
# weight layout of the library (see include/polestar.h)
# ------------------------------------------------------------------------------------------

def rope_interleave_index(head_dim: int) -> torch.Tensor:
    """packed index p -> logical index inside a head: 2i -> i, 2i+1 -> i + head_dim/2."""
    half = head_dim // 2
    idx = torch.empty(head_dim, dtype=torch.long)
    idx[0::2] = torch.arange(half)
    idx[1::2] = torch.arange(half) + half
    return idx


TILE_ROWS = 256   # out-features per weight block of the tile-major layout


def tile_major(w: torch.Tensor) -> torch.Tensor:
    """[out, in] -> contiguous [256][64] blocks (bf16, out % 256 == 0, in % 64 == 0); else unchanged."""
    o, i = w.shape
    if w.dtype != torch.bfloat16 or o % TILE_ROWS or i % 64:
        return w.contiguous()
    return w.view(o // TILE_ROWS, TILE_ROWS, i // 64, 64).permute(0, 2, 1, 3).contiguous().view(o, i)


def untile(w: torch.Tensor) -> torch.Tensor:
    o, i = w.shape
    if w.dtype != torch.bfloat16 or o % TILE_ROWS or i % 64:
        return w
    return w.view(o // TILE_ROWS, i // 64, TILE_ROWS, 64).permute(0, 2, 1, 3).contiguous().view(o, i)


def pack_weights(m: I.ModelCfg, w: Dict, device="cuda", consume: bool = False) -> Dict:
    """Logical weights (inputs.make_weights) -> the library's device layout."""
    dev = torch.device(device)
    dt = I.torch_dtype(m)
    perm = rope_interleave_index(m.head_dim)

    def heads_perm(x, n_heads):
        x = x.view(n_heads, m.head_dim, x.shape[-1])
        return x[:, perm.to(x.device), :].reshape(n_heads * m.head_dim, -1)

    out = {"wqkv": [], "wo": [], "w_gate_up": [], "w_down": [], "norm1": [], "norm2": []}
    if "embed" in w:
        out.update({"embed": w["embed"].to(dev, dt).contiguous(), "lm_head": tile_major(w["lm_head"].to(dev, dt)),
                    "final_norm": w["final_norm"].to(dev, torch.float32).contiguous()})
    layers = w["layers"]
    for i in range(len(layers)):
        l = layers[i]
        q = heads_perm(l["wq"].to(dev, dt), m.n_heads)
        k = heads_perm(l["wk"].to(dev, dt), m.n_kv_heads)
        out["wqkv"].append(tile_major(torch.cat([q, k, l["wv"].to(dev, dt)], 0)))
        out["wo"].append(tile_major(l["wo"].to(dev, dt)))
        out["w_gate_up"].append(tile_major(torch.stack([l["wg"].to(dev, dt), l["wu"].to(dev, dt)], 1)
                                           .reshape(2 * m.d_ffn, m.d_model)))
        out["w_down"].append(tile_major(l["wd"].to(dev, dt)))
        out["norm1"].append(l["norm1"].to(dev, torch.float32).contiguous())
        out["norm2"].append(l["norm2"].to(dev, torch.float32).contiguous())
        if consume:
            layers[i] = None
    return out


def make_packed_weights(m: I.ModelCfg, seed: int = 0, device="cuda", std: float = 0.02) -> Dict:
    """Generate the seeded model directly on the device, one layer at a time."""
    out = None
    for l in range(m.n_layers):
        w = I.make_weights(m, seed, device, std, layers=[l], with_globals=(l == 0))
        pk = pack_weights(m, w, device)
        if out is None:
            out = pk
        else:
            for k in ("wqkv", "wo", "w_gate_up", "w_down", "norm1", "norm2"):
                out[k].extend(pk[k])
        del w, pk
    return out


# ------------------------------------------------------------------------------------------
# the decoding path
# ------------------------------------------------------------------------------------------

class Polestar:
    """polestar_init / polestar_step / polestar_commit on torch-owned device memory."""

    def __init__(self, m: I.ModelCfg, packed: Dict, p: I.Params, prompt):
        if not torch.cuda.is_available():
            raise PolestarError(E_CUDA, "no CUDA device: the Polestar path has no CPU fallback")
        lib = load()
        self.m, self.p, self.packed = m, p, packed
        self.N = p.prompt_len + p.gen_len
        self.W_max = max(1, min((p.win_prefix_blocks + p.win_suffix_blocks) * p.block, self.N - p.block))
        cm, cp = c_model(m), c_params(p)
        need = int(lib.polestar_workspace_bytes(C.byref(cm), C.byref(cp)))
        if need == 0:
            raise PolestarError(E_INVAL, "invalid model / parameters")
        self.workspace = torch.empty(need, dtype=torch.uint8, device="cuda")       # torch allocations are 512-byte aligned
        L = m.n_layers
        arr = lambda ts: (C.c_void_p * L)(*[t.data_ptr() for t in ts])
        self._arrays = [arr(packed[k]) for k in ("wqkv", "wo", "w_gate_up", "w_down", "norm1", "norm2")]
        cw = CWeights(packed["embed"].data_ptr(), packed["lm_head"].data_ptr(), packed["final_norm"].data_ptr(),
                      *self._arrays)
        if p.flags & FLAG_PROMPT_DEVICE:
            self._prompt = prompt.to(device="cuda", dtype=torch.int32).contiguous()
            prompt_ptr = C.cast(C.c_void_p(self._prompt.data_ptr()), C.POINTER(C.c_int32))
        else:
            self._prompt = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32).reshape(p.batch, p.prompt_len))
            prompt_ptr = self._prompt.ctypes.data_as(C.POINTER(C.c_int32))
        self.ctx = C.c_void_p()
        _check(lib.polestar_init(C.byref(self.ctx), C.byref(cm), C.byref(cw), C.byref(cp),
                                 prompt_ptr, C.c_void_p(self.workspace.data_ptr()), need, C.c_void_p(_stream())))
        self.done = False

    def step(self) -> CStepInfo:
        info = CStepInfo()
        _check(load().polestar_step(self.ctx, C.byref(info)))
        return info

    def commit(self) -> CCommitInfo:
        info = CCommitInfo()
        _check(load().polestar_commit(self.ctx, C.byref(info)))
        self.done = bool(info.all_done)
        return info

    def tokens(self) -> np.ndarray:
        out = np.empty((self.p.batch, self.N), np.int32)
        _check(load().polestar_tokens(self.ctx, out.ctypes.data_as(C.POINTER(C.c_int32))))
        return out

    def decode(self):
        """Run to completion; returns the last commit info."""
        info = self.commit()
        while not info.all_done:
            self.step()
            info = self.commit()
        return info

    def read(self, what: int, layer: int = 0) -> np.ndarray:
        m, p = self.m, self.p
        bs, B, Wm, N = p.batch, p.block, self.W_max, self.N
        dkv = m.n_kv_heads * m.head_dim
        el = np.float32 if m.dtype == I.DTYPE_F32 else np.uint16
        shapes = {READ_LOGITS: ((bs, B, m.vocab), np.float32), READ_CONF: ((bs, B), np.float32),
                  READ_YHAT: ((bs, B), np.int32), READ_DELTA: ((bs, B), np.float32),
                  READ_DRIFT: ((bs, Wm), np.float32), READ_SEL_COUNT: ((bs,), np.int32),
                  READ_SEL_IDX: ((bs, Wm), np.int32), READ_HIDDEN: ((bs, B, m.d_model), np.float32),
                  READ_KCACHE: ((bs, N, dkv), el), READ_VCACHE: ((bs, N, dkv), el),
                  READ_HCACHE: ((bs, Wm, m.d_model), np.float32), READ_COMMIT: ((bs, B), np.int32),
                  READ_PPREV: ((bs, p.n_clusters if p.select_mode == I.SELECT_CLUSTER_TOPK else Wm, m.n_heads, N), np.float32),
                  READ_SUFFIX: ((bs, Wm), np.int32), READ_LABELS: ((bs, Wm), np.int32),
                  READ_DRIFT_DELTA: ((bs, B), np.float32), READ_TAU_D: ((bs, B), np.float32),
                  READ_THETA: ((bs, max(1, p.hist), B), np.float32), READ_THETA_COUNT: ((bs,), np.int32),
                  READ_OWN_COMMIT: ((bs, B), np.int32),
                  READ_TRACE_KERNELS: ((8192,), np.int64), READ_TRACE_GEMM: ((2048,), np.int64)}
        shape, dt = shapes[what]
        out = np.empty(shape, dt)
        _check(load().polestar_read(self.ctx, what, layer, out.ctypes.data_as(C.c_void_p), out.nbytes))
        if dt == np.uint16:
            out = (out.astype(np.uint32) << 16).view(np.float32)
        if what == READ_KCACHE:   # undo the rotary pair interleave of the key layout
            inv = np.argsort(rope_interleave_index(m.head_dim).numpy())
            out = out.reshape(bs, N, m.n_kv_heads, m.head_dim)[..., inv].reshape(bs, N, dkv)
        return out

    def profile(self, reset: bool = False) -> Dict:
        out = (C.c_double * (len(PROF_FAMILIES) * 4))()
        _check(load().polestar_profile(self.ctx, out, 1 if reset else 0))
        return {f: dict(calls=out[4 * i], ms=out[4 * i + 1], bytes=out[4 * i + 2], flops=out[4 * i + 3])
                for i, f in enumerate(PROF_FAMILIES)}

    def force_select(self, layer: int, idx) -> None:
        idx = np.ascontiguousarray(np.asarray(idx, np.int32).reshape(self.p.batch, -1))
        _check(load().polestar_force(self.ctx, FORCE_SELECT, layer, idx.ctypes.data_as(C.POINTER(C.c_int32)),
                                     idx.shape[1]))

    def force_commit(self, positions, tokens=None) -> None:
        pos = np.ascontiguousarray(np.asarray(positions, np.int32).reshape(self.p.batch, -1))
        _check(load().polestar_force(self.ctx, FORCE_COMMIT, 0, pos.ctypes.data_as(C.POINTER(C.c_int32)),
                                     pos.shape[1]))
        if tokens is not None:
            tok = np.ascontiguousarray(np.asarray(tokens, np.int32).reshape(self.p.batch, -1))
            _check(load().polestar_force(self.ctx, FORCE_TOKENS, 0, tok.ctypes.data_as(C.POINTER(C.c_int32)),
                                         tok.shape[1]))

    def force_labels(self, layer: int, labels) -> None:
        lab = np.ascontiguousarray(np.asarray(labels, np.int32).reshape(self.p.batch, -1))
        _check(load().polestar_force(self.ctx, FORCE_LABELS, layer, lab.ctypes.data_as(C.POINTER(C.c_int32)), lab.shape[1]))

    def force_hcodes(self, layer: int, mask, codes, scales) -> None:
        """mask uint8 [batch][n], codes uint8 [batch][n][d/2], scales uint8 [batch][n][d/16] (E4M3 bit patterns)."""
        mask = np.ascontiguousarray(mask, np.uint8)
        blob = np.concatenate([mask.ravel(), np.ascontiguousarray(codes, np.uint8).ravel(),
                               np.ascontiguousarray(scales, np.uint8).ravel()])
        pad = np.zeros((-len(blob)) % 4, np.uint8)
        blob = np.ascontiguousarray(np.concatenate([blob, pad]))
        _check(load().polestar_force(self.ctx, FORCE_HCODES, layer, blob.ctypes.data_as(C.POINTER(C.c_int32)), mask.shape[1]))

    def force_clear(self) -> None:
        _check(load().polestar_force(self.ctx, FORCE_CLEAR, 0, None, 0))

    def destroy(self):
        if getattr(self, "ctx", None) is not None and self.ctx.value:
            load().polestar_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


# ------------------------------------------------------------------------------------------
# single kernels
# ------------------------------------------------------------------------------------------

def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return I.DTYPE_BF16
    if t.dtype == torch.float32:
        return I.DTYPE_F32
    raise PolestarError(E_INVAL, f"unsupported dtype {t.dtype}")


def polestar_k_attention(q, k, v, row_prev, lse_prev, kl, out, n_heads, n_kv_heads, head_dim):
    """Stored rows are pairs (row_prev, lse_prev) with log-probability = row_prev - lse_prev[..., None]."""
    R, N = q.shape[0], k.shape[0]
    _check(load().polestar_k_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(row_prev), _ptr(lse_prev), _ptr(kl), _ptr(out), R, N,
                                       n_heads, n_kv_heads, head_dim, _dtype_code(q), C.c_void_p(_stream())))


def polestar_k_hidden_delta(a, b, out):
    rows, d = a.shape
    _check(load().polestar_k_hidden_delta(_ptr(a), _ptr(b), _ptr(out), rows, d, _dtype_code(a), C.c_void_p(_stream())))


def polestar_k_select(drift, mode, k, thresh, floor_, idx, count):
    batch, W = drift.shape
    _check(load().polestar_k_select(_ptr(drift), batch, W, mode, k, thresh, floor_, _ptr(idx), _ptr(count),
                                    C.c_void_p(_stream())))


def polestar_k_refresh_scratch_bytes(batch, max_rows, d, n_heads, n_kv_heads, head_dim) -> int:
    return int(load().polestar_k_refresh_scratch_bytes(batch, max_rows, d, n_heads, n_kv_heads, head_dim))


def polestar_k_refresh(h, idx, counts, wqkv, norm, kc, vc, q_out, max_rows, n_heads, n_kv_heads, head_dim,
                       rms_eps, rope_theta, scratch):
    batch, P, d = h.shape
    _check(load().polestar_k_refresh(_ptr(h), _ptr(idx), _ptr(counts), _ptr(wqkv), _ptr(norm), _ptr(kc), _ptr(vc),
                                     _ptr(q_out), batch, P, max_rows, d, n_heads, n_kv_heads, head_dim, rms_eps,
                                     rope_theta, _dtype_code(h), _ptr(scratch), scratch.numel() * scratch.element_size(),
                                     C.c_void_p(_stream())))


def polestar_k_nvfp4_residual(x, ref, codes, scales, deq):
    rows, d = x.shape
    _check(load().polestar_k_nvfp4_residual(_ptr(x), _ptr(ref), rows, d, _ptr(codes), _ptr(scales), _ptr(deq),
                                            C.c_void_p(_stream())))


def polestar_k_wait_probe(counter, expect: int, limit_cycles: int, status) -> int:
    """Returns the library's code (OK or E_TIMEOUT) instead of raising: the time-out is the expected outcome."""
    return load().polestar_k_wait_probe(_ptr(counter), expect, limit_cycles, _ptr(status), C.c_void_p(_stream()))


def polestar_reload_env() -> None:
    """Make the stand-alone kernel calls re-read the POLESTAR_* environment switches."""
    _check(load().polestar_reload_env())


def polestar_k_refresh_status(scratch, batch, max_rows, d, head_dim) -> int:
    return int(load().polestar_k_refresh_status(_ptr(scratch), scratch.numel() * scratch.element_size(), batch,
                                                max_rows, d, head_dim, C.c_void_p(_stream())))


def polestar_k_confidence(logits, mask_id, yhat, conf, scratch):
    rows, V = logits.shape
    _check(load().polestar_k_confidence(_ptr(logits), rows, V, mask_id, _ptr(yhat), _ptr(conf), _ptr(scratch),
                                        scratch.numel() * scratch.element_size(), C.c_void_p(_stream())))


NOALLOC_MAX_ROWS = 1024


def polestar_k_confidence_noalloc(logits, mask_id, yhat, conf):
    """Confidence of logits rows using the library's built-in scratch (no allocation, rows <= 1024).
    For callers that cannot hand over scratch memory; concurrent calls on one device must be serialised."""
    rows, V = logits.shape
    _check(load().polestar_k_confidence_noalloc(_ptr(logits), rows, V, mask_id, _ptr(yhat), _ptr(conf),
                                                C.c_void_p(_stream())))
