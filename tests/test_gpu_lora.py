"""GPU-vs-oracle parity of the low-rank adapter layer (frozen base weight, rank-r A and B):
every element on small and odd shapes, sampled rows at the adapter workload's full size."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2609_28568_b200 import binding as nb
from paper_2609_28568_b200 import synth
from parity import Guarded, check_bf16, check_f32, f32, sample_indices

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(autouse=True)
def _status_clean():
    yield
    nb.nb_check_status()


def gen(seed, shape, std):
    return synth.normal(seed, shape, std, DEV)


def _rounding_slack(mid_ref, other):
    """The call rounds its rank-r intermediate (t or u) to bf16 once, a relative error of at most
    2^-9 per element; through the second factor that moves an output by at most this much."""
    return 2.0 ** -9 * (np.abs(mid_ref) @ np.abs(np.asarray(other, np.float64)))


def _tensors(BT, C, OC, r, bias, seed):
    inp = gen(seed, (BT, C), 1.0)
    w = gen(seed + 1, (OC, C), 0.02)
    b = gen(seed + 2, (OC,), 0.02) if bias else None
    a = gen(seed + 3, (r, C), 0.02)
    bb = gen(seed + 4, (OC, r), 0.02)  # a trained adapter: B is no longer zero
    dout = gen(seed + 5, (BT, OC), 1e-3)
    return inp, w, b, a, bb, dout


@pytest.mark.parametrize("bias", [False, True])
@pytest.mark.parametrize("BT,C,OC,r", [
    (1, 8, 8, 8),            # smallest legal problem
    (200, 72, 136, 16),      # ragged in every dimension, one tile
    (300, 328, 520, 16),     # several n-tiles, ragged tails, a CTA pair
    (640, 256, 768, 64),     # the extension fills a whole k-block
    (520, 1024, 1024, 24),   # many k-blocks before the extension
])
def test_adapter_layer_every_element(BT, C, OC, r, bias):
    scale = 32.0 / math.sqrt(r)  # rank-stabilised scaling
    inp, w, b, a, bb, dout = _tensors(BT, C, OC, r, bias, seed=900)
    out = Guarded((BT, OC), torch.bfloat16)
    t = Guarded((BT, r), torch.bfloat16)
    nb.nb_lora_linear_forward(out.t, t.t, inp, w, b, a, bb, scale, BT, C, OC, r)
    o_ref = oracle.lora_forward(f32(inp), f32(w), f32(b) if bias else None, f32(a), f32(bb), scale)
    t_ref, _ = oracle.linear_forward(f32(inp), f32(a))
    check_bf16(t.t, scale * t_ref, "t")
    check_bf16(out.t, o_ref, "out", extra=_rounding_slack(scale * t_ref, f32(bb).T))
    # and with the stored t as the oracle's input the layer is one product over [inp | t]
    o_ref2, _ = oracle.linear_forward(np.concatenate([f32(inp), f32(t.t)], axis=1),
                                      np.concatenate([f32(w), f32(bb)], axis=1), f32(b) if bias else None)
    check_bf16(out.t, o_ref2, "out from stored t")
    out.check("out")
    t.check("t")
    # the adapter term must be visible in this test, or the comparison proves nothing about it
    base, _ = oracle.linear_forward(f32(inp), f32(w), f32(b) if bias else None)
    assert np.abs(o_ref - base).max() > 0.05 * np.abs(base).max()

    dinp = Guarded((BT, C), torch.bfloat16)
    u = Guarded((BT, r), torch.bfloat16)
    dA = Guarded((r, C), torch.float32, fill=777.0)   # accumulate=0 must overwrite
    dB = Guarded((OC, r), torch.float32, fill=-55.0)
    nb.nb_lora_linear_backward(dinp.t, dA.t, dB.t, u.t, dout, inp, w, a, bb, t.t, scale, BT, C, OC, r, 0)
    di_ref, dA_ref, dB_ref = oracle.lora_backward(f32(dout), f32(inp), f32(w), f32(a), f32(bb), scale)
    u_ref = oracle.linear_backward(f32(dout), None, f32(bb), want=("dinp",))["dinp"]
    check_bf16(u.t, scale * u_ref, "u")
    check_bf16(dinp.t, di_ref, "dinp", extra=_rounding_slack(scale * u_ref, f32(a)))
    di_ref2 = oracle.linear_backward(np.concatenate([f32(dout), f32(u.t)], axis=1), None,
                                     np.concatenate([f32(w), f32(a)], axis=0), want=("dinp",))["dinp"]
    check_bf16(dinp.t, di_ref2, "dinp from stored u")
    check_f32(dA.t, dA_ref, "dlora_a")
    check_f32(dB.t, dB_ref, "dlora_b")
    for g, n in ((dinp, "dinp"), (u, "u"), (dA, "dlora_a"), (dB, "dlora_b")):
        g.check(n)

    # a second micro-step accumulates; dinp is skipped
    dout2 = gen(990, (BT, OC), 1e-3)
    nb.nb_lora_linear_backward(None, dA.t, dB.t, u.t, dout2, inp, w, a, bb, t.t, scale, BT, C, OC, r, 1)
    _, dA_ref2, dB_ref2 = oracle.lora_backward(f32(dout2), f32(inp), f32(w), f32(a), f32(bb), scale,
                                               dA=dA_ref.copy(), dB=dB_ref.copy(), accumulate=True,
                                               want_dinp=False)
    check_f32(dA.t, dA_ref2, "dlora_a step 2")
    check_f32(dB.t, dB_ref2, "dlora_b step 2")


def test_zero_b_reduces_to_the_base_layer_bit_for_bit():
    """A freshly initialised adapter (B = 0) must give exactly the base layer's output and dinp."""
    BT, C, OC, r = 400, 264, 392, 16
    inp, w, b, a, _, dout = _tensors(BT, C, OC, r, True, seed=940)
    zb = torch.zeros((OC, r), dtype=torch.bfloat16, device=DEV)
    out = torch.empty((BT, OC), dtype=torch.bfloat16, device=DEV)
    t = torch.empty((BT, r), dtype=torch.bfloat16, device=DEV)
    nb.nb_lora_linear_forward(out, t, inp, w, b, a, zb, 8.0, BT, C, OC, r)
    base, _ = nb.linear_forward(inp, w, b, nb.ACT_NONE)
    assert torch.equal(out, base)
    dinp = torch.empty((BT, C), dtype=torch.bfloat16, device=DEV)
    u = torch.empty((BT, r), dtype=torch.bfloat16, device=DEV)
    dA = torch.empty((r, C), dtype=torch.float32, device=DEV)
    nb.nb_lora_linear_backward(dinp, dA, None, u, dout, inp, w, a, zb, None, 8.0, BT, C, OC, r, 0)
    dbase, _, _ = nb.linear_backward(dout, inp, w, need_dweight=False, need_dbias=False)
    assert torch.equal(dinp, dbase)
    assert float(u.float().abs().max()) == 0.0 and float(dA.abs().max()) == 0.0


def test_adapter_rejects_bad_rank_and_missing_tensors():
    BT, C, OC = 64, 64, 64
    x = torch.zeros((BT, C), dtype=torch.bfloat16, device=DEV)
    w = torch.zeros((OC, C), dtype=torch.bfloat16, device=DEV)
    for r in (4, 12, 72):
        a = torch.zeros((r, C), dtype=torch.bfloat16, device=DEV)
        b = torch.zeros((OC, r), dtype=torch.bfloat16, device=DEV)
        t = torch.zeros((BT, r), dtype=torch.bfloat16, device=DEV)
        with pytest.raises(nb.NbError) as e:
            nb.nb_lora_linear_forward(x, t, x, w, None, a, b, 1.0, BT, C, OC, r)
        assert e.value.code == nb.NB_ERR_UNSUPPORTED
    a = torch.zeros((16, C), dtype=torch.bfloat16, device=DEV)
    b = torch.zeros((OC, 16), dtype=torch.bfloat16, device=DEV)
    t = torch.zeros((BT, 16), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(nb.NbError) as e:
        nb.nb_lora_linear_forward(x, None, x, w, None, a, b, 1.0, BT, C, OC, 16)
    assert e.value.code == nb.NB_ERR_INVALID_ARG
    dB = torch.zeros((OC, 16), dtype=torch.float32, device=DEV)
    with pytest.raises(nb.NbError) as e:  # dlora_b needs the forward call's t
        nb.nb_lora_linear_backward(None, None, dB, t, x, x, w, a, b, None, 1.0, BT, C, OC, 16, 0)
    assert e.value.code == nb.NB_ERR_INVALID_ARG


@pytest.mark.parametrize("C,OC", [(1024, 2048), (3072, 1024)])
def test_adapter_workload_full_batch_sampled(C, OC):
    """Qwen3-0.6B q and down projections with rank-16 adapters at B=8, T=2048."""
    BT, r = 16384, 16
    scale = 32.0 / math.sqrt(r)
    inp, w, _, a, bb, dout = _tensors(BT, C, OC, r, False, seed=960)
    out = torch.empty((BT, OC), dtype=torch.bfloat16, device=DEV)
    t = torch.empty((BT, r), dtype=torch.bfloat16, device=DEV)
    nb.nb_lora_linear_forward(out, t, inp, w, None, a, bb, scale, BT, C, OC, r)
    dinp = torch.empty((BT, C), dtype=torch.bfloat16, device=DEV)
    u = torch.empty((BT, r), dtype=torch.bfloat16, device=DEV)
    dA = torch.empty((r, C), dtype=torch.float32, device=DEV)
    dB = torch.empty((OC, r), dtype=torch.float32, device=DEV)
    nb.nb_lora_linear_backward(dinp, dA, dB, u, dout, inp, w, a, bb, t, scale, BT, C, OC, r, 0)

    rows = sample_indices(BT, 64, 961)
    rt = torch.as_tensor(rows, device=DEV)
    o_ref = oracle.lora_forward(f32(inp[rt]), f32(w), None, f32(a), f32(bb), scale)
    t_ref, _ = oracle.linear_forward(f32(inp[rt]), f32(a))
    check_bf16(out[rt], o_ref, "out rows", extra=_rounding_slack(scale * t_ref, f32(bb).T))
    di_ref, _, _ = oracle.lora_backward(f32(dout[rt]), f32(inp[rt]), f32(w), f32(a), f32(bb), scale)
    u_ref = oracle.linear_backward(f32(dout[rt]), None, f32(bb), want=("dinp",))["dinp"]
    check_bf16(dinp[rt], di_ref, "dinp rows", extra=_rounding_slack(scale * u_ref, f32(a)))
    # the adapter gradients sum over every row: the oracle runs them in full (they are cheap)
    _, dA_ref, dB_ref = oracle.lora_backward(f32(dout), f32(inp), f32(w), f32(a), f32(bb), scale,
                                             want_dinp=False)
    check_f32(dA, dA_ref, "dlora_a")
    check_f32(dB, dB_ref, "dlora_b")


@pytest.mark.parametrize("bias", [False, True])
@pytest.mark.parametrize("BT,C,ocs,r", [
    (200, 72, (136, 64, 200), 16),     # three adapters on one input, ragged, one tile
    (520, 328, (520, 264), 24),        # two adapters, rank 24 (R = 48), several tiles, a CTA pair
    (300, 1024, (1024, 2048, 8), 8),   # R = 24, many k-blocks before the extension, a tiny projection
])
def test_stacked_adapters_equal_the_oracle_per_adapter(BT, C, ocs, r, bias):
    """Adapters that share an input, stacked: the group's down-projection and A gradient are single
    products over all adapters, each projection reads and writes its own column slice of t_stack /
    u_stack. Every result is compared with the oracle of that adapter alone (t and u slices, out,
    dinp, dB, the rows of dA), with canaries around every buffer, over two accumulating micro-steps."""
    n = len(ocs)
    R = n * r
    scale = 32.0 / math.sqrt(r)
    inp = gen(1200, (BT, C), 1.0)
    a_stack = gen(1201, (R, C), 0.02)
    t_stack = Guarded((BT, R), torch.bfloat16)
    u_stack = Guarded((BT, R), torch.bfloat16)
    da_stack = Guarded((R, C), torch.float32, fill=777.0)
    ws = [gen(1210 + j, (oc, C), 0.02) for j, oc in enumerate(ocs)]
    bs = [gen(1220 + j, (oc,), 0.02) if bias else None for j, oc in enumerate(ocs)]
    lbs = [gen(1230 + j, (oc, r), 0.02) for j, oc in enumerate(ocs)]
    nb.nb_lora_down_stacked(t_stack.t, inp, a_stack, scale, BT, C, R)
    t_ref, _ = oracle.linear_forward(f32(inp), f32(a_stack))
    check_bf16(t_stack.t, scale * t_ref, "t_stack")
    t_stack.check("t_stack")
    outs, dinps, dBs, dAref, dBref = [], [], [], [None] * n, [None] * n
    for j, oc in enumerate(ocs):
        a_j = a_stack[j * r:(j + 1) * r]
        out = Guarded((BT, oc), torch.bfloat16)
        nb.nb_lora_linear_forward_stacked(out.t, inp, ws[j], bs[j], t_stack.t, lbs[j], BT, C, oc, r, R, j * r)
        o_ref = oracle.lora_forward(f32(inp), f32(ws[j]), f32(bs[j]) if bias else None, f32(a_j), f32(lbs[j]), scale)
        check_bf16(out.t, o_ref, f"out {j}", extra=_rounding_slack(scale * t_ref[:, j * r:(j + 1) * r], f32(lbs[j]).T))
        out.check(f"out {j}")
        dinps.append(Guarded((BT, C), torch.bfloat16))
        dBs.append(Guarded((oc, r), torch.float32, fill=-55.0))
    for ms in range(2):
        douts = [gen(1240 + 10 * ms + j, (BT, oc), 1e-3) for j, oc in enumerate(ocs)]
        u_stack.t.fill_(99.0)  # every column must be rewritten by its own adapter's call
        for j in reversed(range(n)):
            oc = ocs[j]
            a_j = a_stack[j * r:(j + 1) * r]
            nb.nb_lora_linear_backward_stacked(dinps[j].t, dBs[j].t, u_stack.t, douts[j], ws[j], a_j, lbs[j],
                                               t_stack.t, scale, BT, C, oc, r, R, j * r, ms)
            di_ref, dAref[j], dBref[j] = oracle.lora_backward(
                f32(douts[j]), f32(inp), f32(ws[j]), f32(a_j), f32(lbs[j]), scale,
                dA=dAref[j], dB=dBref[j], accumulate=ms > 0)
            u_ref = oracle.linear_backward(f32(douts[j]), None, f32(lbs[j]), want=("dinp",))["dinp"]
            check_bf16(u_stack.t[:, j * r:(j + 1) * r], scale * u_ref, f"u slice {j}")
            check_bf16(dinps[j].t, di_ref, f"dinp {j}", extra=_rounding_slack(scale * u_ref, f32(a_j)))
            check_f32(dBs[j].t, dBref[j], f"dlora_b {j} step {ms}")
            dinps[j].check(f"dinp {j}")
            dBs[j].check(f"dlora_b {j}")
        u_stack.check("u_stack")
        nb.nb_lora_da_stacked(da_stack.t, u_stack.t, inp, BT, C, R, ms)
        for j in range(n):
            check_f32(da_stack.t[j * r:(j + 1) * r], dAref[j], f"dlora_a {j} step {ms}")
        da_stack.check("da_stack")
    t_stack.check("t_stack after backward")


def test_stacked_rejects_bad_slices():
    x = torch.zeros((64, 64), dtype=torch.bfloat16, device=DEV)
    t = torch.zeros((64, 48), dtype=torch.bfloat16, device=DEV)
    b = torch.zeros((64, 16), dtype=torch.bfloat16, device=DEV)
    for r, R, off, code in ((16, 48, 40, nb.NB_ERR_INVALID_ARG), (16, 48, 4, nb.NB_ERR_INVALID_ARG),
                            (16, 72, 0, nb.NB_ERR_UNSUPPORTED), (12, 48, 0, nb.NB_ERR_UNSUPPORTED)):
        with pytest.raises(nb.NbError) as e:
            nb.nb_lora_linear_forward_stacked(x, x, x, None, t, b, 64, 64, 64, r, R, off)
        assert e.value.code == code


@pytest.mark.parametrize("stacked", [True, False])
def test_adapter_stack_driver_two_micro_steps(stacked):
    """The adapter-stage driver: one Qwen3 layer's seven adapted projections, two micro-steps; outputs
    and dinp of the last micro-step and the accumulated adapter gradients against the oracle, with the
    adapters of a group stacked (the default) and with one set of calls per projection."""
    from paper_2609_28568_b200.stack import LoraStack
    BT = 384
    st = LoraStack(BT, micro_steps=2, device=DEV, layers=1, stacked=stacked)
    st.step()
    torch.cuda.synchronize()
    assert [L.spec.name for L in st.layers] == ["q", "k", "v", "o", "gate", "up", "down"]
    for L in st.layers:
        w, a, b = f32(L.weight), f32(L.lora_a), f32(L.lora_b)
        o_ref = oracle.lora_forward(f32(L.inp[1]), w, None, a, b, st.scale)
        t_ref, _ = oracle.linear_forward(f32(L.inp[1]), a)
        check_bf16(L.out, o_ref, L.spec.name + " out", extra=_rounding_slack(st.scale * t_ref, b.T))
        dA = dB = None
        for ms in range(2):
            di_ref, dA, dB = oracle.lora_backward(f32(L.dout[ms]), f32(L.inp[ms]), w, a, b, st.scale,
                                                  dA=dA, dB=dB, accumulate=ms > 0)
        u_ref = oracle.linear_backward(f32(L.dout[1]), None, b, want=("dinp",))["dinp"]
        check_bf16(L.dinp, di_ref, L.spec.name + " dinp", extra=_rounding_slack(st.scale * u_ref, a))
        check_f32(L.dlora_a, dA, L.spec.name + " dlora_a")
        check_f32(L.dlora_b, dB, L.spec.name + " dlora_b")
    assert st.flops_per_micro_step() == sum(
        4 * BT * c * oc + 6 * BT * 16 * (c + oc)
        for c, oc in ((1024, 2048), (1024, 1024), (1024, 1024), (2048, 1024), (1024, 3072), (1024, 3072),
                      (3072, 1024)))


def test_adapter_stack_driver_fused_groups():
    """The projections of a group as one linear layer (weights stacked by rows, B block-diagonal): every
    member's output columns, adapter gradients and the group's summed input gradient against the oracle
    of each adapter alone, over two accumulating micro-steps; and the same values as the unfused driver
    produces from the same seeds."""
    from paper_2609_28568_b200.stack import LoraStack
    BT, r = 384, 16
    st = LoraStack(BT, micro_steps=2, device=DEV, layers=1, fused=True)
    ref = LoraStack(BT, micro_steps=2, device=DEV, layers=1)
    st.step()
    ref.step()
    torch.cuda.synchronize()
    assert [L.spec.name for L in st.layers] == ["q_k_v", "o", "gate_up", "down"]
    assert st.flops_per_micro_step() == ref.flops_per_micro_step()
    by_name = {L.spec.name: L for L in ref.layers}
    for (L,) in st.groups:
        di_sum, slack_sum = 0.0, 0.0
        for j, (s, row, _) in enumerate(L.members):
            cols = slice(row, row + s.OC)
            w, a = f32(L.weight[cols]), f32(L.a_stack[j * r:(j + 1) * r])
            b = f32(L.lora_b[cols, j * r:(j + 1) * r])
            U = by_name[s.name]   # the unfused driver's projection: same seeds, same tensors
            assert torch.equal(L.weight[cols], U.weight) and torch.equal(L.lora_b[cols, j * r:(j + 1) * r], U.lora_b)
            assert torch.equal(L.dout[1][:, cols], U.dout[1]) and torch.equal(L.inp[1], U.inp[1])
            # zero blocks beside the member's own: its output takes nothing from the other adapters
            assert float(L.lora_b[cols].float().abs().sum()) == float(L.lora_b[cols, j * r:(j + 1) * r].float().abs().sum())
            o_ref = oracle.lora_forward(f32(L.inp[1]), w, None, a, b, st.scale)
            t_ref, _ = oracle.linear_forward(f32(L.inp[1]), a)
            check_bf16(L.out[:, cols], o_ref, s.name + " out", extra=_rounding_slack(st.scale * t_ref, b.T))
            assert torch.equal(L.out[:, cols], U.out), s.name + ": fused and unfused outputs differ"
            dA = dB = None
            for ms in range(2):
                di_ref, dA, dB = oracle.lora_backward(f32(L.dout[ms][:, cols]), f32(L.inp[ms]), w, a, b, st.scale,
                                                      dA=dA, dB=dB, accumulate=ms > 0)
            u_ref = oracle.linear_backward(f32(L.dout[1][:, cols]), None, b, want=("dinp",))["dinp"]
            di_sum = di_sum + di_ref
            slack_sum = slack_sum + _rounding_slack(st.scale * u_ref, a)
            check_f32(L.da_stack[j * r:(j + 1) * r], dA, s.name + " dlora_a")
            check_f32(L.dlora_b[cols, j * r:(j + 1) * r], dB, s.name + " dlora_b")
        check_bf16(L.dinp, di_sum, L.spec.name + " dinp (sum over the group)", extra=slack_sum)
