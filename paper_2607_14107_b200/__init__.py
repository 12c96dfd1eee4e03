"""Polestar denoising hot path for masked-diffusion LLMs on B200 (sm_100a).

`inputs` describes workloads and draws seeded synthetic tensors; `binding`
is the ctypes layer over the C-ABI library built from `csrc/`.
"""
from . import inputs  # noqa: F401
