"""Seeded synthetic inputs: model shapes, decoding parameters, weights, prompts.

This module holds no arithmetic of the decoding method itself.  It only
describes workloads (shapes, hyper-parameters) and draws reproducible random
tensors.  Both the CPU oracle's tests and the CUDA path's tests / benchmark
take their inputs from here, so the two sides always see the same numbers.

Random values come from a counter-based generator: element ``i`` of tensor
``(seed, layer, tensor_id)`` is a pure function of those four integers.  Only
integer operations and one float multiply are used, so a CPU tensor and a CUDA
tensor generated from the same key are bit-identical, any sub-range can be
regenerated on its own, and 8-billion-parameter models can be filled directly
in device memory.

The "normal" values are an Irwin-Hall sum: eight independent 16-bit uniforms,
centred and scaled to the requested standard deviation (range +-4.9 sigma,
excess kurtosis -0.15).  They stand in for the N(0, 0.02^2) random
initialisation the workloads name.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import torch

# --------------------------------------------------------------------------
# Workload descriptions
# --------------------------------------------------------------------------

DTYPE_F32 = 0
DTYPE_BF16 = 1

SELECT_TOPK_FRAC = 0
SELECT_TOPK_COUNT = 1
SELECT_THRESHOLD = 2
SELECT_ALL = 3
SELECT_NONE = 4
SELECT_CLUSTER_TOPK = 5

FLAG_DRIFT_COMMIT = 1 << 0
FLAG_SUFFIX_COMMIT = 1 << 1
FLAG_GE_COMPARE = 1 << 2
FLAG_NOCACHE = 1 << 3
FLAG_KEEP_HIDDEN = 1 << 4
FLAG_NVFP4_HCACHE = 1 << 8
FLAG_DEFAULT = FLAG_DRIFT_COMMIT | FLAG_SUFFIX_COMMIT | FLAG_GE_COMPARE

TAU_UPD_NEVER = 2**31 - 1


@dataclass
class ModelCfg:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: int = DTYPE_F32
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    mask_id: int = -1
    eos_id: int = -1

    def __post_init__(self):
        if self.mask_id < 0:
            self.mask_id = self.vocab - 1
        if self.eos_id < 0:
            self.eos_id = self.vocab - 2

    @property
    def d_q(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim


@dataclass
class Params:
    batch: int = 1
    prompt_len: int = 64
    gen_len: int = 64
    block: int = 32
    max_steps: int = 32
    win_prefix_blocks: int = 2
    win_suffix_blocks: int = 1
    full_entry_period: int = 2
    select_mode: int = SELECT_TOPK_FRAC
    select_frac: float = 0.25
    select_k: int = 0
    select_thresh: float = 0.0
    drift_floor: float = 0.0
    tau_upd: int = 3
    hist: int = 5
    tau_s: float = 0.9
    alpha: float = 10.0
    tau_suffix: float = 0.9
    logit_scale: float = 1.0
    flags: int = FLAG_DEFAULT
    # centroid proxies (select_mode = SELECT_CLUSTER_TOPK): K clusters of the window's hidden states per layer,
    # the cluster_k clusters with the largest drift are refreshed; Lloyd iterations of the spherical K-means
    n_clusters: int = 8
    cluster_k: int = 4
    kmeans_iters: int = 4

    @property
    def seq_len(self) -> int:
        return self.prompt_len + self.gen_len

    @property
    def n_blocks(self) -> int:
        return self.gen_len // self.block


def config(name: str):
    """Named workloads.  Returns (ModelCfg, Params).

    c1  tiny fp32 model the oracle decodes in seconds
    c1b tiny bf16 model with 128-wide heads (tensor-core path at oracle size)
    c2  LLaDA-8B shape, batch 1, prompt 256 + gen 256, block 32
    c3  Dream-7B shape (GQA 28/4), batch 4, prompt 512 + gen 512
    c4  long generation on the LLaDA-8B shape, batch 8, 1024 + 1024, block 64
    c6  short generations on the LLaDA-8B shape (Sec. 5.2, hard-to-parallelise tasks: generation length 32,
        block 8), batch 1, prompt 128
    """
    if name == "c1":
        m = ModelCfg(2, 256, 4, 4, 64, 1024, 1024, DTYPE_F32, 1e-5, 10000.0)
        p = Params(batch=1, prompt_len=64, gen_len=64, block=32, max_steps=32)
    elif name == "c1b":
        m = ModelCfg(2, 256, 2, 2, 128, 512, 2048, DTYPE_BF16, 1e-5, 10000.0)
        p = Params(batch=1, prompt_len=64, gen_len=64, block=32, max_steps=32)
    elif name == "c2":
        m = ModelCfg(32, 4096, 32, 32, 128, 12288, 126464, DTYPE_BF16, 1e-5, 500000.0)
        p = Params(batch=1, prompt_len=256, gen_len=256, block=32, max_steps=256)
    elif name == "c3":
        m = ModelCfg(28, 3584, 28, 4, 128, 18944, 152064, DTYPE_BF16, 1e-5, 1000000.0)
        p = Params(batch=4, prompt_len=512, gen_len=512, block=32, max_steps=512)
    elif name == "c4":
        m = ModelCfg(32, 4096, 32, 32, 128, 12288, 126464, DTYPE_BF16, 1e-5, 500000.0)
        p = Params(batch=8, prompt_len=1024, gen_len=1024, block=64, max_steps=1024)
    elif name == "c6":
        m = ModelCfg(32, 4096, 32, 32, 128, 12288, 126464, DTYPE_BF16, 1e-5, 500000.0)
        p = Params(batch=1, prompt_len=128, gen_len=32, block=8, max_steps=32)
    else:
        raise KeyError(name)
    return m, p


SHAPES = {"c1": "tiny fp32 model", "c1b": "tiny bf16 model", "c2": "LLaDA-8B shape", "c3": "Dream-7B shape (GQA 28/4)",
          "c4": "LLaDA-8B shape, long generation", "c6": "LLaDA-8B shape, short generation"}


def reduced_depth(m: ModelCfg, n_layers: int) -> ModelCfg:
    """Same widths and vocabulary, fewer layers (for CPU-sized comparisons)."""
    return dataclasses.replace(m, n_layers=n_layers)


# --------------------------------------------------------------------------
# Counter-based generator
# --------------------------------------------------------------------------

_M32 = 0xFFFFFFFF
# std of the sum of eight uniforms on {0..65535}: sqrt(8 * (65536^2 - 1) / 12)
_IH8_STD = math.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0)
_IH8_MEAN = 8 * 65535 // 2  # 262140


def _splitmix64(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    return z ^ (z >> 31)


def tensor_key(seed: int, layer: int, tensor_id: int) -> int:
    """64-bit key of one tensor; every tensor gets its own random stream."""
    k = _splitmix64(seed & 0xFFFFFFFFFFFFFFFF)
    k = _splitmix64(k ^ ((layer + 1) * 0x100000001B3))
    k = _splitmix64(k ^ ((tensor_id + 1) * 0xC2B2AE3D27D4EB4F))
    return k


def _hash32(x: torch.Tensor) -> torch.Tensor:
    """Integer avalanche hash on int64 tensors holding values in [0, 2^32)."""
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _M32
    x = x ^ (x >> 15)
    x = (x * 0x846CA68B) & _M32
    x = x ^ (x >> 16)
    return x


def _words(key: int, start: int, count: int, n_words: int, device) -> List[torch.Tensor]:
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    out = []
    for w in range(n_words):
        salt = _splitmix64(key ^ (w + 1)) & _M32
        salt2 = _splitmix64(key ^ (0x5851F42D4C957F2D * (w + 1))) & _M32
        lo = (idx & _M32) ^ salt
        hi = ((idx >> 32) * 0x9E3779B1) & _M32
        out.append(_hash32((_hash32(lo ^ hi) + salt2) & _M32))
    return out


def normal_range(key: int, start: int, count: int, std: float, device="cpu") -> torch.Tensor:
    """fp32 values start..start+count of the stream ``key`` (approx. N(0, std^2))."""
    ws = _words(key, start, count, 4, device)
    s = torch.zeros(count, dtype=torch.int64, device=device)
    for w in ws:
        s += (w & 0xFFFF) + (w >> 16)
    s -= _IH8_MEAN
    scale = torch.tensor(std / _IH8_STD, dtype=torch.float32, device=device)
    return s.to(torch.float32) * scale


def normal_tensor(key: int, shape, std: float, dtype=torch.float32, device="cpu",
                  chunk: int = 1 << 24) -> torch.Tensor:
    """Tensor of the given shape filled from stream ``key`` (row-major order)."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    for st in range(0, n, chunk):
        c = min(chunk, n - st)
        out[st:st + c] = normal_range(key, st, c, std, device).to(dtype)
    return out.view(*shape)


def uniform_ids(key: int, count: int, modulus: int, device="cpu") -> torch.Tensor:
    """int32 ids uniform on [0, modulus)."""
    (w,) = _words(key, 0, count, 1, device)
    return (w % modulus).to(torch.int32)


# --------------------------------------------------------------------------
# Model weights and prompts
# --------------------------------------------------------------------------

# tensor ids inside a layer (layer = -1 for the global tensors)
T_WQ, T_WK, T_WV, T_WO, T_WG, T_WU, T_WD, T_NORM1, T_NORM2 = range(9)
T_EMBED, T_LM_HEAD, T_FINAL_NORM = 16, 17, 18
T_PROMPT = 32
T_HCACHE, T_DRIFT = 48, 49


def torch_dtype(m: ModelCfg):
    return torch.bfloat16 if m.dtype == DTYPE_BF16 else torch.float32


def make_weights(m: ModelCfg, seed: int = 0, device="cpu", std: float = 0.02,
                 layers: Optional[List[int]] = None, with_globals: bool = True,
                 gain_std: float = 0.1) -> Dict:
    """Logical weights, every matrix stored [out_features, in_features].

    Values are rounded to the model's storage dtype (bf16 models hold
    bf16-representable numbers).  RMSNorm gains are 1 + gain_std * normal, one
    stream per norm (two per layer and the final one), so that a swapped or
    dropped gain changes the result; ``gain_std = 0`` gives unit gains.
    ``layers`` limits generation to a subset of layers (same values as in the
    full model).
    """
    dt = torch_dtype(m)
    d, dq, dkv, F, V = m.d_model, m.d_q, m.d_kv, m.d_ffn, m.vocab

    def mk(layer, tid, shape):
        return normal_tensor(tensor_key(seed, layer, tid), shape, std, dt, device)

    def gain(layer, tid):
        g = normal_tensor(tensor_key(seed, layer, tid), (d,), gain_std, torch.float32, device)
        return (1.0 + g).to(dt)

    w = {"layers": []}
    if with_globals:
        w.update({"embed": mk(-1, T_EMBED, (V, d)), "lm_head": mk(-1, T_LM_HEAD, (V, d)),
                  "final_norm": gain(-1, T_FINAL_NORM)})
    for l in (range(m.n_layers) if layers is None else layers):
        w["layers"].append({
            "wq": mk(l, T_WQ, (dq, d)), "wk": mk(l, T_WK, (dkv, d)), "wv": mk(l, T_WV, (dkv, d)),
            "wo": mk(l, T_WO, (d, dq)), "wg": mk(l, T_WG, (F, d)), "wu": mk(l, T_WU, (F, d)),
            "wd": mk(l, T_WD, (d, F)),
            "norm1": gain(l, T_NORM1), "norm2": gain(l, T_NORM2),
        })
    return w


def make_prompt(m: ModelCfg, p: Params, seed: int = 1) -> torch.Tensor:
    """[batch, prompt_len] int32 ids, uniform over the vocabulary minus [MASK]."""
    n = p.batch * p.prompt_len
    ids = uniform_ids(tensor_key(seed, -1, T_PROMPT), n, m.vocab - 1)
    ids = torch.where(ids >= m.mask_id, ids + 1, ids) if m.mask_id < m.vocab - 1 else ids
    return ids.view(p.batch, p.prompt_len).contiguous()


def weights_to_numpy(w: Dict) -> Dict:
    """fp32 numpy copy of a weight dict (for the CPU oracle)."""
    def cv(t):
        return t.detach().to("cpu", torch.float32).numpy()
    return {"embed": cv(w["embed"]), "lm_head": cv(w["lm_head"]), "final_norm": cv(w["final_norm"]),
            "layers": [{k: cv(v) for k, v in l.items()} for l in w["layers"]]}


# --------------------------------------------------------------------------
# Refresh-kernel microbenchmark inputs (cache of 4096 positions x 4096 hidden)
# --------------------------------------------------------------------------

def make_refresh_inputs(batch: int, positions: int = 4096, d_model: int = 4096,
                        seed_h: int = 3, seed_d: int = 2, clustered: bool = False,
                        device="cpu"):
    """Hidden-state cache [batch, positions, d] (bf16, N(0,1)-like) and drift
    scores [batch, positions] fp32 = exp(normal(0,1)) (seeded lognormal).

    ``clustered`` multiplies the scores by exp(-|pos - positions/2| / 256) so the
    largest scores sit near one "active block", the structure drift shows in
    practice (concentration in a local window); the plain variant scatters the
    selected rows uniformly, the worst case for the gather.
    """
    h = normal_tensor(tensor_key(seed_h, -1, T_HCACHE), (batch, positions, d_model), 1.0,
                      torch.bfloat16, device)
    z = normal_tensor(tensor_key(seed_d, -1, T_DRIFT), (batch, positions), 1.0, torch.float32, "cpu")
    drift = torch.exp(z.double())
    if clustered:
        pos = torch.arange(positions, dtype=torch.float64)
        drift = drift * torch.exp(-(pos - positions / 2).abs() / 256.0)[None, :]
    return h, drift.float().to(device)


def refresh_count(frac: float, positions: int = 4096) -> int:
    return int(math.floor(frac * positions + 0.5))
