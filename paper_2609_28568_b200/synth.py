"""Seeded synthetic inputs, identical bit for bit on CPU and GPU.

This module holds none of the method's arithmetic. It only produces the random
bf16 tensors (activations ~N(0,1), weights ~N(0,0.02), gradients ~N(0,1e-3) ...)
that both the CUDA path and the CPU oracle are fed, standing in for the paper's
token-derived activations and trained weights (Method/Model gives the init
distribution and the vocabulary padding).

Generation is counter based so that any element can be produced anywhere:
``value[i] = Q[hash32(seed, i) >> 16] * std`` rounded to bf16, where ``Q`` is a
table of the 65536 mid-point quantiles of N(0,1). Integer hashing, one table
lookup and one fp32 multiply behave identically on every device, so a tensor
generated on the GPU for a full-size run and its rows regenerated on the CPU for
the oracle agree exactly.
"""
from __future__ import annotations

import torch

_MASK32 = 0xFFFFFFFF
_TABLES: dict = {}
_CHUNK = 1 << 24

VOCAB_REAL = 50257
VOCAB_PADDED = 50304
BASE_SEED = 1337  # the paper's seed


def _quantile_table(device) -> torch.Tensor:
    key = str(device)
    if key not in _TABLES:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        q = torch.special.ndtri(p).to(torch.float32)  # always computed on the CPU
        _TABLES[key] = q.to(device)
    return _TABLES[key]


def _hash32(idx: torch.Tensor, seed: int) -> torch.Tensor:
    """32-bit avalanche hash of (seed, idx), carried in int64 lanes."""
    s0 = (seed * 0x9E3779B1 + 0x7F4A7C15) & _MASK32
    s1 = ((seed >> 32) * 0x85EBCA77 + 0x165667B1) & _MASK32
    lo = idx & _MASK32
    hi = (idx >> 32) & _MASK32
    h = (lo ^ s0) & _MASK32
    h = (h * 0x85EBCA6B) & _MASK32
    h = h ^ (h >> 13)
    h = (h + hi * 0x27D4EB2F + s1) & _MASK32
    h = (h * 0xC2B2AE35) & _MASK32
    h = h ^ (h >> 16)
    h = (h * 0x7FEB352D) & _MASK32
    h = h ^ (h >> 15)
    h = (h * 0x846CA68B) & _MASK32
    h = h ^ (h >> 16)
    return h


def normal_flat(seed: int, start: int, count: int, std: float, device="cpu") -> torch.Tensor:
    """Elements [start, start+count) of the stream ``seed`` as bf16 ~N(0, std^2)."""
    table = _quantile_table(device)
    out = torch.empty(count, dtype=torch.bfloat16, device=device)
    scale = torch.tensor(std, dtype=torch.float32, device=device)
    for off in range(0, count, _CHUNK):
        n = min(_CHUNK, count - off)
        idx = torch.arange(start + off, start + off + n, dtype=torch.int64, device=device)
        h = _hash32(idx, seed)
        out[off:off + n] = (table[h >> 16] * scale).to(torch.bfloat16)
    return out


def normal(seed: int, shape, std: float, device="cpu") -> torch.Tensor:
    """A bf16 tensor of ``shape`` ~N(0, std^2), row-major over the stream ``seed``."""
    n = 1
    for s in shape:
        n *= int(s)
    return normal_flat(seed, 0, n, std, device).reshape(*shape)


def normal_rows(seed: int, rows, ncols: int, std: float, device="cpu") -> torch.Tensor:
    """Rows ``rows`` of the [*, ncols] tensor that ``normal(seed, (*, ncols), std)`` makes."""
    table = _quantile_table(device)
    rows = torch.as_tensor(rows, dtype=torch.int64, device=device)
    idx = rows[:, None] * ncols + torch.arange(ncols, dtype=torch.int64, device=device)[None, :]
    h = _hash32(idx, seed)
    scale = torch.tensor(std, dtype=torch.float32, device=device)
    return (table[h >> 16] * scale).to(torch.bfloat16)


def tensor_seed(config: int, layer: int, role: int, micro_step: int = 0) -> int:
    """Seed of one tensor: base 1337 + 1000*config + 100*layer + 10*role + micro-step.

    role: 0 inp, 1 weight, 2 bias, 3 dout (further roles are free for a caller).
    """
    return BASE_SEED + 1000 * config + 100 * layer + 10 * role + micro_step


def zero_pad_vocab_rows(weight: torch.Tensor) -> torch.Tensor:
    """Zero rows [50257, 50304) of a [50304, C] head weight (padding rows)."""
    if weight.shape[0] == VOCAB_PADDED:
        weight[VOCAB_REAL:].zero_()
    return weight


def zero_pad_vocab_cols(dlogits: torch.Tensor) -> torch.Tensor:
    """Zero columns [50257, 50304) of a [BT, 50304] logits gradient: padding gets no gradient."""
    if dlogits.shape[1] == VOCAB_PADDED:
        dlogits[:, VOCAB_REAL:].zero_()
    return dlogits
