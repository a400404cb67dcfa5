"""Shapes of the linear layers on the hot path, and their flop / byte accounting.

GPT-2 124M (paper, Method/Model and Figure 1): 12 blocks, 768 channels, 12 heads,
MLP 768 -> 3072 -> 768, head tied to the 50304-row padded embedding, every linear
but the head has a bias. Residual-writing projections are initialised with
std 0.02 / sqrt(2 L). The adapter stage (Method/The clinical stage) uses
Qwen3-0.6B's seven projections per layer over 28 layers.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

ACT_NONE, ACT_GELU, ACT_SWIGLU = 0, 1, 2

GPT2_LAYERS = 12
GPT2_CHANNELS = 768
GPT2_CTX = 1024
VOCAB_REAL = 50257
VOCAB_PADDED = 50304
QWEN3_LAYERS = 28


@dataclass(frozen=True)
class LinearSpec:
    name: str
    C: int            # input channels
    OC: int           # weight rows (for SwiGLU: gate rows then up rows)
    bias: bool
    act: int = ACT_NONE
    w_std: float = 0.02
    fused_gelu_bwd: bool = False  # dgrad epilogue applies gelu'(pre) of the producer of inp

    @property
    def out_cols(self) -> int:
        return self.OC // 2 if self.act == ACT_SWIGLU else self.OC

    def flops(self, BT: int, wgrad: bool = True) -> int:
        """2*BT*C*OC for each of forward, dgrad and (optionally) wgrad."""
        return 2 * BT * self.C * self.OC * (3 if wgrad else 2)


def gpt2_block() -> list[LinearSpec]:
    resid = 0.02 / math.sqrt(2 * GPT2_LAYERS)
    return [
        LinearSpec("qkv", 768, 2304, True),
        LinearSpec("attn_proj", 768, 768, True, w_std=resid),
        LinearSpec("fc", 768, 3072, True, act=ACT_GELU),
        LinearSpec("proj", 3072, 768, True, w_std=resid, fused_gelu_bwd=True),
    ]


def gpt2_lm_head() -> LinearSpec:
    return LinearSpec("lm_head", 768, VOCAB_PADDED, False)


def qwen3_block() -> list[LinearSpec]:
    return [
        LinearSpec("q", 1024, 2048, False),
        LinearSpec("k", 1024, 1024, False),
        LinearSpec("v", 1024, 1024, False),
        LinearSpec("o", 2048, 1024, False),
        LinearSpec("gate_up", 1024, 6144, False, act=ACT_SWIGLU),
        LinearSpec("down", 3072, 1024, False),
    ]


def qwen3_lora_projections() -> list[LinearSpec]:
    """The seven adapted projections of a Qwen3-0.6B layer (no bias, no fused activation)."""
    return [
        LinearSpec("q", 1024, 2048, False),
        LinearSpec("k", 1024, 1024, False),
        LinearSpec("v", 1024, 1024, False),
        LinearSpec("o", 2048, 1024, False),
        LinearSpec("gate", 1024, 3072, False),
        LinearSpec("up", 1024, 3072, False),
        LinearSpec("down", 3072, 1024, False),
    ]


def gpt2_param_count() -> tuple[int, int]:
    """(parameters, tensors) of GPT-2 124M with the real vocabulary, tied head."""
    C, L = GPT2_CHANNELS, GPT2_LAYERS
    n = VOCAB_REAL * C + GPT2_CTX * C
    t = 2
    for _ in range(L):
        n += 2 * (2 * C)  # two layer norms, weight and bias
        t += 4
        for s in gpt2_block():
            n += s.OC * s.C + (s.OC if s.bias else 0)
            t += 2 if s.bias else 1
    n += 2 * C  # final layer norm
    t += 2
    return n, t


def qwen3_lora_param_count(r: int = 16) -> int:
    """Trainable parameters of rank-r adapters on the seven projections per layer."""
    per_layer = 0
    for cin, cout in ((1024, 2048), (1024, 1024), (1024, 1024), (2048, 1024),
                      (1024, 3072), (1024, 3072), (3072, 1024)):
        per_layer += r * (cin + cout)
    return QWEN3_LAYERS * per_layer


def gpt2_stack_flops_per_token() -> int:
    """Forward + dgrad + wgrad flops per token of 12 blocks plus the padded head."""
    w = sum(s.C * s.OC for s in gpt2_block()) * GPT2_LAYERS + gpt2_lm_head().C * gpt2_lm_head().OC
    return 6 * w


def qwen3_stack_flops_per_token(wgrad: bool = True) -> int:
    w = sum(s.C * s.OC for s in qwen3_block()) * QWEN3_LAYERS
    return (6 if wgrad else 4) * w
