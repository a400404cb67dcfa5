"""Seeded random walks over the argument space of the forward and backward entry points.

The other parity tests choose their shapes and flag combinations by hand; here they are drawn: row
counts on both sides of every kernel-selection threshold (one CTA or a pair, narrow or full-width
tiles, one launch per layer backward or two), ragged widths, each activation, with and without a
bias, every subset of the three backward products, overwrite followed by accumulate, either dtype
of the weight gradient, the producer's GELU derivative fused into dinp. Every element of every
result is compared with the oracle, and every buffer sits between canaries.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28568_b200 import binding as nb
from paper_2609_28568_b200 import synth
from parity import Guarded, check_bf16, check_f32, f32

pytestmark = pytest.mark.gpu
DEV = "cuda"

_BT_CHOICES = (1, 7, 64, 127, 128, 129, 200, 256, 257, 333, 520, 777, 1100, 2100, 4099)
_ACTS = (nb.ACT_NONE, nb.ACT_GELU, nb.ACT_SWIGLU)


def _draw_case(rng):
    BT = int(rng.choice(_BT_CHOICES))
    C = 8 * int(rng.integers(1, 70))
    OC = 16 * int(rng.integers(1, 40))   # a multiple of 16, so that SwiGLU's halves are multiples of 8
    act = int(rng.choice(_ACTS))
    return BT, C, OC, act


@pytest.mark.parametrize("case", range(100))
def test_random_forward_backward_case_equals_the_oracle(case):
    rng = np.random.default_rng(90_000 + case)
    BT, C, OC, act = _draw_case(rng)
    bias = bool(rng.integers(0, 2))
    fused = act == nb.ACT_NONE and bool(rng.integers(0, 2))   # inp was produced by a GELU layer
    want_dinp, want_dw, want_db = (bool(rng.integers(0, 4)) for _ in range(3))   # each present 3 times in 4
    want_db = want_db and bias
    bf16_dw = want_dw and bool(rng.integers(0, 4) == 0)
    seed = 91_000 + 10 * case
    inp = synth.normal(seed, (BT, C), 1.0, DEV)
    w = synth.normal(seed + 1, (OC, C), 0.05, DEV)
    b = synth.normal(seed + 2, (OC,), 0.05, DEV) if bias else None
    ocols = OC // 2 if act == nb.ACT_SWIGLU else OC
    dout = synth.normal(seed + 3, (BT, ocols), 1e-3, DEV)
    ipre = synth.normal(seed + 4, (BT, C), 1.0, DEV) if fused else None
    tag = f"case {case}: BT={BT} C={C} OC={OC} act={act} bias={bias} fused={fused}"

    # ---- forward
    out = Guarded((BT, ocols), torch.bfloat16)
    pre = Guarded((BT, OC), torch.bfloat16) if act != nb.ACT_NONE else None
    nb.nb_linear_forward_ex(out.t, pre.t if pre else None, inp, w, b, BT, C, OC, act)
    o_ref, p_ref = oracle.linear_forward(f32(inp), f32(w), f32(b) if bias else None, act)
    check_bf16(out.t, o_ref, "out, " + tag)
    out.check("out")
    if pre:
        check_bf16(pre.t, p_ref, "pre_act, " + tag)
        pre.check("pre_act")

    # ---- backward: overwrite, then (fp32 gradients only) accumulate the same gradient again
    if not (want_dinp or want_dw or want_db):
        want_dinp = True
    dinp = Guarded((BT, C), torch.bfloat16) if want_dinp else None
    dw = Guarded((OC, C), torch.bfloat16 if bf16_dw else torch.float32, fill=3.0) if want_dw else None
    db = Guarded((OC,), torch.float32, fill=-3.0) if want_db else None
    passes = 1 if bf16_dw else 2
    for acc in range(passes):
        nb.nb_linear_backward_ex(dinp.t if dinp else None, dw.t if dw else None, db.t if db else None, dout,
                                 inp if want_dw else None, w if want_dinp else None, pre.t if pre else None,
                                 ipre if want_dinp else None,   # rejected without dinp: it has nothing to scale
                                 BT, C, OC, act, acc,
                                 nb.DTYPE_BF16 if bf16_dw else nb.DTYPE_F32)
    r = oracle.linear_backward(f32(dout), f32(inp), f32(w), pre=f32(pre.t) if pre else None,
                               inp_pre=f32(ipre) if fused else None, act=act)
    if dinp:
        check_bf16(dinp.t, r["dinp"], "dinp, " + tag)
        dinp.check("dinp")
    if dw:
        if bf16_dw:
            check_bf16(dw.t, r["dweight"], "dweight (bf16), " + tag)
        else:
            check_f32(dw.t, passes * r["dweight"], "dweight, " + tag)
        dw.check("dweight")
    if db:
        check_f32(db.t, passes * r["dbias"], "dbias, " + tag)
        db.check("dbias")
    nb.nb_check_status()


_LORA_BT = (1, 100, 128, 129, 300, 1000, 2500, 19333, 40001)   # the last two: more row panels than SMs


@pytest.mark.parametrize("case", range(36))
def test_random_adapter_layer_case_equals_the_oracle(case):
    """The adapter layer on drawn shapes and ranks: t, out, u, dinp, dA and dB of two accumulating
    micro-steps, every element. The large row counts give each CTA of the fused u / dB kernel several
    row panels in turn, which the hand-picked shapes of the adapter tests do not."""
    rng = np.random.default_rng(95_000 + case)
    BT = int(_LORA_BT[case % len(_LORA_BT)])
    big = BT > 10_000
    C = 8 * int(rng.integers(1, 12 if big else 60))
    OC = 8 * int(rng.integers(1, 40 if big else 90))
    r = int(rng.choice((8, 16, 24, 32, 48, 64)))
    bias = bool(rng.integers(0, 2))
    scale = 32.0 / float(np.sqrt(r))
    seed = 96_000 + 10 * case
    inp = synth.normal(seed, (BT, C), 1.0, DEV)
    w = synth.normal(seed + 1, (OC, C), 0.02, DEV)
    b = synth.normal(seed + 2, (OC,), 0.02, DEV) if bias else None
    a = synth.normal(seed + 3, (r, C), 0.02, DEV)
    bb = synth.normal(seed + 4, (OC, r), 0.02, DEV)
    tag = f"case {case}: BT={BT} C={C} OC={OC} r={r} bias={bias}"

    def slack(mid_ref, other):   # the one bf16 rounding of the rank-r intermediate, through the second factor
        return 2.0 ** -9 * (np.abs(mid_ref) @ np.abs(np.asarray(other, np.float64)))

    out = Guarded((BT, OC), torch.bfloat16)
    t = Guarded((BT, r), torch.bfloat16)
    nb.nb_lora_linear_forward(out.t, t.t, inp, w, b, a, bb, scale, BT, C, OC, r)
    o_ref = oracle.lora_forward(f32(inp), f32(w), f32(b) if bias else None, f32(a), f32(bb), scale)
    t_ref, _ = oracle.linear_forward(f32(inp), f32(a))
    check_bf16(t.t, scale * t_ref, "t, " + tag)
    check_bf16(out.t, o_ref, "out, " + tag, extra=slack(scale * t_ref, f32(bb).T))
    out.check("out")
    t.check("t")

    dinp = Guarded((BT, C), torch.bfloat16)
    u = Guarded((BT, r), torch.bfloat16)
    dA = Guarded((r, C), torch.float32, fill=5.0)
    dB = Guarded((OC, r), torch.float32, fill=-5.0)
    dA_ref = dB_ref = None
    for step in range(2):
        dout = synth.normal(seed + 5 + step, (BT, OC), 1e-3, DEV)
        nb.nb_lora_linear_backward(dinp.t, dA.t, dB.t, u.t, dout, inp, w, a, bb, t.t, scale, BT, C, OC, r, step)
        di_ref, dA_ref, dB_ref = oracle.lora_backward(f32(dout), f32(inp), f32(w), f32(a), f32(bb), scale,
                                                      dA=dA_ref, dB=dB_ref, accumulate=step > 0)
        u_ref = oracle.linear_backward(f32(dout), None, f32(bb), want=("dinp",))["dinp"]
        check_bf16(u.t, scale * u_ref, f"u step {step}, " + tag)
        check_bf16(dinp.t, di_ref, f"dinp step {step}, " + tag, extra=slack(scale * u_ref, f32(a)))
        check_f32(dA.t, dA_ref, f"dlora_a step {step}, " + tag)
        check_f32(dB.t, dB_ref, f"dlora_b step {step}, " + tag)
    for g, n in ((dinp, "dinp"), (u, "u"), (dA, "dlora_a"), (dB, "dlora_b")):
        g.check(n)
    nb.nb_check_status()
