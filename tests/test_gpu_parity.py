"""GPU-vs-oracle parity through the C ABI: every element on small and odd shapes and on the
two small workloads; sampled rows, columns and elements at the full-size workloads."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2609_28568_b200 import binding as nb
from paper_2609_28568_b200 import shapes, synth
from parity import (Guarded, check_bf16, check_f32, f32, rel_frob, sample_indices, stratified_indices)

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(autouse=True)
def _status_clean():
    yield
    nb.nb_check_status()  # no kernel may have given up on a wait


def gen(seed, shape, std):
    return synth.normal(seed, shape, std, DEV)


# --------------------------------------------------------------------------- every element

def run_layer_full(BT, C, OC, act, bias=True, w_std=0.02, dout_std=1e-3, seed=100):
    """Forward + backward of one layer on the GPU and in the oracle, compared element by element.
    Backward applies the layer's own activation derivative through the GPU-stored pre-activation,
    which is also what the oracle is handed, so each call is checked on its own."""
    inp = gen(seed, (BT, C), 1.0)
    w = gen(seed + 1, (OC, C), w_std)
    b = gen(seed + 2, (OC,), 0.02) if bias else None
    ocols = OC // 2 if act == nb.ACT_SWIGLU else OC
    dout = gen(seed + 3, (BT, ocols), dout_std)

    out = Guarded((BT, ocols), torch.bfloat16)
    pre = Guarded((BT, OC), torch.bfloat16) if act != nb.ACT_NONE else None
    nb.nb_linear_forward_ex(out.t, pre.t if pre else None, inp, w, b, BT, C, OC, act)
    o_ref, p_ref = oracle.linear_forward(f32(inp), f32(w), f32(b) if bias else None, act)
    check_bf16(out.t, o_ref, "out")
    out.check("out")
    if pre:
        check_bf16(pre.t, p_ref, "pre_act")
        pre.check("pre_act")

    dinp = Guarded((BT, C), torch.bfloat16)
    dw = Guarded((OC, C), torch.float32, fill=777.0)  # accumulate=0 must overwrite
    db = Guarded((OC,), torch.float32, fill=-55.0) if bias else None
    nb.nb_linear_backward_ex(dinp.t, dw.t, db.t if db else None, dout, inp, w,
                             pre.t if pre else None, None, BT, C, OC, act, 0)
    r = oracle.linear_backward(f32(dout), f32(inp), f32(w), pre=f32(pre.t) if pre else None, act=act)
    check_bf16(dinp.t, r["dinp"], "dinp")
    check_f32(dw.t, r["dweight"], "dweight")
    dinp.check("dinp")
    dw.check("dweight")
    if db:
        check_f32(db.t, r["dbias"], "dbias")
        db.check("dbias")


@pytest.mark.parametrize("act", [nb.ACT_NONE, nb.ACT_GELU, nb.ACT_SWIGLU])
@pytest.mark.parametrize("BT,C,OC", [
    (1, 8, 16),          # a single row, one k block
    (128, 64, 256),      # exactly one tile
    (136, 72, 208),      # ragged in every dimension
    (392, 328, 528),     # several tiles with ragged tails
    (700, 200, 1040),    # more than one tile along OC with a tail
])
def test_small_shapes_every_element(BT, C, OC, act):
    run_layer_full(BT, C, OC, act, w_std=0.05, dout_std=1e-3, seed=7 * BT + OC + act)


@pytest.mark.parametrize("BT,C,OC", [
    (129, 8, 8),          # one row past a single tile: the smallest pair problem, one k-block each way
    (256, 2056, 24),      # one dinp row tile, nine column tiles, a single ragged dweight tile
    (4100, 72, 136),      # 65 k-blocks of K = BT for dweight, five rows past a tile
    (1000, 520, 2304),    # more dweight tiles than dinp tiles
])
def test_one_launch_backward_edge_shapes(BT, C, OC):
    """Shapes that stress the work list of the one-launch layer backward (BT > 128: dinp tiles and
    dweight k-chunks in one kernel): with and without the bias gradient, overwrite then accumulate,
    and with the producer's GELU derivative in the dinp epilogue; every element against the oracle."""
    inp, w = gen(300 + BT, (BT, C), 1.0), gen(301 + BT, (OC, C), 0.05)
    dout, ipre = gen(302 + BT, (BT, OC), 1e-3), gen(303 + BT, (BT, C), 1.0)
    for bias in (True, False):
        for fused in (False, True):
            dinp = Guarded((BT, C), torch.bfloat16)
            dw = Guarded((OC, C), torch.float32, fill=9.0)
            db = Guarded((OC,), torch.float32, fill=9.0) if bias else None
            for acc in (0, 1):
                nb.nb_linear_backward_ex(dinp.t, dw.t, db.t if db else None, dout, inp, w, None,
                                         ipre if fused else None, BT, C, OC, nb.ACT_NONE, acc)
            r = oracle.linear_backward(f32(dout), f32(inp), f32(w), inp_pre=f32(ipre) if fused else None)
            tag = f"bias={bias} fused={fused}"
            check_bf16(dinp.t, r["dinp"], "dinp " + tag)
            check_f32(dw.t, 2.0 * r["dweight"], "dweight " + tag)
            if db:
                check_f32(db.t, 2.0 * r["dbias"], "dbias " + tag)
                db.check("dbias")
            dinp.check("dinp")
            dw.check("dweight")


@pytest.mark.parametrize("BT,C,OC,fused", [(8192, 768, 2304, False), (4096, 3072, 768, True)])
def test_one_launch_backward_is_stable_over_repeated_launches(BT, C, OC, fused):
    """Sixty launches of the one-launch layer backward, with copies on another stream perturbing the
    schedule: dinp has no reduction across units and must come out bit for bit the same; dweight and
    dbias are summed by reduce-adds in varying order and must agree to rounding. A stage handed back
    too early or a barrier phase off by one shows up here as a rare mismatch."""
    inp, w = gen(331, (BT, C), 1.0), gen(332, (OC, C), 0.02)
    dout, ipre = gen(333, (BT, OC), 1e-3), gen(334, (BT, C), 1.0)
    side = torch.cuda.Stream()
    ref = None
    for it in range(60):
        dinp = torch.empty((BT, C), dtype=torch.bfloat16, device=DEV)
        dw = torch.full((OC, C), 7.0, dtype=torch.float32, device=DEV)
        db = torch.full((OC,), 7.0, dtype=torch.float32, device=DEV)
        if it % 3 == 1:
            with torch.cuda.stream(side):
                torch.empty(1 << 24, device=DEV).fill_(1.0)
        nb.nb_linear_backward_ex(dinp, dw, db, dout, inp, w, None, ipre if fused else None, BT, C, OC,
                                 nb.ACT_NONE, 0)
        if ref is None:
            ref = (dinp, dw, db)
        else:
            assert torch.equal(dinp, ref[0]), f"dinp differs at launch {it}"
            assert rel_frob(f32(dw[:256]), f32(ref[1][:256])) < 1e-5
            assert rel_frob(f32(db), f32(ref[2])) < 1e-5
    torch.cuda.synchronize()


def test_integer_inputs_are_exact():
    """Small integers: products and sums are exact in bf16 x bf16 -> fp32, so GPU == oracle exactly.
    Catches any indexing or layout error that a tolerance could hide."""
    BT, C, OC = 200, 136, 328
    g = torch.Generator().manual_seed(3)
    ri = lambda *s: torch.randint(-4, 5, s, generator=g).to(torch.bfloat16).to(DEV)
    inp, w, b, dz = ri(BT, C), ri(OC, C), ri(OC), ri(BT, OC)
    out, _ = nb.linear_forward(inp, w, b, nb.ACT_NONE)
    o_ref, _ = oracle.linear_forward(f32(inp), f32(w), f32(b))
    small = np.abs(o_ref) <= 256  # integers up to 2^8 are representable in bf16
    assert small.mean() > 0.9
    assert np.array_equal(f32(out).astype(np.float64)[small], o_ref[small])
    dinp, dw, db = nb.linear_backward(dz, inp, w)
    r = oracle.linear_backward(f32(dz), f32(inp), f32(w))
    assert np.array_equal(f32(dw).astype(np.float64), r["dweight"])
    assert np.array_equal(f32(db).astype(np.float64), r["dbias"])
    exact = np.abs(r["dinp"]) <= 256
    assert exact.mean() > 0.9
    assert np.array_equal(f32(dinp).astype(np.float64)[exact], r["dinp"][exact])


def test_config1_fc_layer_forward_backward():
    """Workload 1: one GPT-2 MLP fc layer, B=2 T=64, tanh-GELU, own pre-activation in backward."""
    run_layer_full(128, 768, 3072, nb.ACT_GELU, seed=synth.tensor_seed(1, 0, 0))


def test_short_form_calls_two_plane_out():
    """The 8- and 11-argument entry points: `out` carries the activated and pre-activation planes."""
    BT, C, OC = 128, 768, 3072
    inp, w, b = gen(1, (BT, C), 1.0), gen(2, (OC, C), 0.02), gen(3, (OC,), 0.02)
    dout = gen(4, (BT, OC), 1e-3)
    n = nb.nb_linear_out_elems(BT, OC, nb.ACT_GELU)
    planes = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    nb.nb_linear_forward(planes, inp, w, b, BT, C, OC, nb.ACT_GELU)
    out, pre = planes[:BT * OC].view(BT, OC), planes[BT * OC:].view(BT, OC)
    out2, pre2 = nb.linear_forward(inp, w, b, nb.ACT_GELU)
    assert torch.equal(out, out2) and torch.equal(pre, pre2)
    dinp = torch.empty((BT, C), dtype=torch.bfloat16, device=DEV)
    dw = torch.empty((OC, C), dtype=torch.float32, device=DEV)
    db = torch.empty((OC,), dtype=torch.float32, device=DEV)
    nb.nb_linear_backward(dinp, dw, db, dout, inp, w, pre, BT, C, OC, 0)
    r = oracle.linear_backward(f32(dout), f32(inp), f32(w), pre=f32(pre), act=oracle.ACT_GELU)
    check_bf16(dinp, r["dinp"], "dinp")
    check_f32(dw, r["dweight"], "dweight")
    check_f32(db, r["dbias"], "dbias")
    # SwiGLU planes
    OC2 = 512
    w2 = gen(5, (OC2, C), 0.02)
    n2 = nb.nb_linear_out_elems(BT, OC2, nb.ACT_SWIGLU)
    planes2 = torch.empty(n2, dtype=torch.bfloat16, device=DEV)
    nb.nb_linear_forward(planes2, inp, w2, None, BT, C, OC2, nb.ACT_SWIGLU)
    o_ref, p_ref = oracle.linear_forward(f32(inp), f32(w2), None, oracle.ACT_SWIGLU)
    check_bf16(planes2[:BT * OC2 // 2].view(BT, OC2 // 2), o_ref, "swiglu out")
    check_bf16(planes2[BT * OC2 // 2:].view(BT, OC2), p_ref, "swiglu pre")


def test_config2_block_linears():
    """Workload 2: the four linears of one GPT-2 block at B=4, T=1024, every element."""
    BT = 4096
    for li, s in enumerate(shapes.gpt2_block()):
        inp = gen(synth.tensor_seed(2, li, 0), (BT, s.C), 1.0)
        w = gen(synth.tensor_seed(2, li, 1), (s.OC, s.C), s.w_std)
        b = gen(synth.tensor_seed(2, li, 2), (s.OC,), 0.02)
        dout = gen(synth.tensor_seed(2, li, 3), (BT, s.OC), 1e-3)
        out, pre = nb.linear_forward(inp, w, b, s.act)
        o_ref, p_ref = oracle.linear_forward(f32(inp), f32(w), f32(b), s.act)
        check_bf16(out, o_ref, s.name + " out")
        if pre is not None:
            check_bf16(pre, p_ref, s.name + " pre")
        dinp, dw, db = nb.linear_backward(dout, inp, w, pre_act=pre, act=s.act)
        r = oracle.linear_backward(f32(dout), f32(inp), f32(w),
                                   pre=f32(pre) if pre is not None else None, act=s.act)
        check_bf16(dinp, r["dinp"], s.name + " dinp")
        check_f32(dw, r["dweight"], s.name + " dweight")
        check_f32(db, r["dbias"], s.name + " dbias")


def test_config2_fused_gelu_backward_equals_composed():
    """fc -> proj chain: proj's dgrad epilogue applies gelu'(fc.pre), giving fc's dz directly.
    It must agree with the oracle and, to rounding, with the composed form (dgrad, then the
    elementwise product inside fc's own backward)."""
    BT = 4096
    fc, proj = shapes.gpt2_block()[2], shapes.gpt2_block()[3]
    x = gen(11, (BT, fc.C), 1.0)
    w_fc, b_fc = gen(12, (fc.OC, fc.C), fc.w_std), gen(13, (fc.OC,), 0.02)
    w_pr = gen(14, (proj.OC, proj.C), proj.w_std)
    dout = gen(15, (BT, proj.OC), 1e-3)
    h, pre = nb.linear_forward(x, w_fc, b_fc, nb.ACT_GELU)
    # fused: dz_fc = (dout . W_proj) * gelu'(pre)
    dz_fused, dw_pr, _ = nb.linear_backward(dout, h, w_pr, inp_pre_act=pre, need_dbias=False)
    r = oracle.linear_backward(f32(dout), f32(h), f32(w_pr), inp_pre=f32(pre))
    check_bf16(dz_fused, r["dinp"], "fused dz")
    check_f32(dw_pr, r["dweight"], "proj dweight")
    # composed: plain dgrad, then fc's backward applies gelu'(pre) itself
    dh, _, _ = nb.linear_backward(dout, h, w_pr, need_dweight=False, need_dbias=False)
    dx_c, dw_c, db_c = nb.linear_backward(dh, x, w_fc, pre_act=pre, act=nb.ACT_GELU)
    dx_f, dw_f, db_f = nb.linear_backward(dz_fused, x, w_fc)
    assert rel_frob(f32(dx_f), f32(dx_c)) < 5e-3
    assert rel_frob(f32(dw_f), f32(dw_c)) < 5e-3
    assert rel_frob(f32(db_f), f32(db_c)) < 5e-3
    rr = oracle.linear_backward(f32(dz_fused), f32(x), f32(w_fc))
    check_bf16(dx_f, rr["dinp"], "fc dinp")
    check_f32(dw_f, rr["dweight"], "fc dweight")
    check_f32(db_f, rr["dbias"], "fc dbias")


# --------------------------------------------------------------------------- accumulation

def test_accumulation_over_micro_steps():
    """Four micro-steps into one fp32 buffer (first overwrites, the rest add) equal the oracle's
    four accumulate calls; the buffers start out dirty."""
    BT, C, OC = 1024, 768, 2304
    w = gen(21, (OC, C), 0.02)
    dw = Guarded((OC, C), torch.float32, fill=3.0)
    db = Guarded((OC,), torch.float32, fill=3.0)
    dw_ref = np.full((OC, C), -9.0)
    db_ref = np.full((OC,), -9.0)
    for ms in range(4):
        inp = gen(synth.tensor_seed(4, 0, 0, ms), (BT, C), 1.0)
        dout = gen(synth.tensor_seed(4, 0, 3, ms), (BT, OC), 1e-3)
        nb.nb_linear_backward_ex(None, dw.t, db.t, dout, inp, w, None, None, BT, C, OC, nb.ACT_NONE,
                                 1 if ms > 0 else 0)
        oracle.linear_backward(f32(dout), f32(inp), f32(w), dweight=dw_ref, dbias=db_ref,
                               accumulate=ms > 0, want=("dweight", "dbias"))
    check_f32(dw.t, dw_ref, "accumulated dweight")
    check_f32(db.t, db_ref, "accumulated dbias")
    dw.check()
    db.check()


def test_reduce_dbias_standalone():
    for BT, OC in ((1, 8), (77, 200), (4096, 2304), (5000, 776)):
        dout = gen(31 + BT, (BT, OC), 1e-3)
        db = Guarded((OC,), torch.float32, fill=1.5)
        nb.nb_reduce_dbias(db.t, dout, BT, OC, 0)
        ref = oracle.reduce_dbias(f32(dout))
        check_f32(db.t, ref, "dbias")
        nb.nb_reduce_dbias(db.t, dout, BT, OC, 1)
        check_f32(db.t, 2 * ref, "dbias twice")
        db.check()


# --------------------------------------------------------------------------- edge cases

def test_skipped_products_and_empty_batch():
    BT, C, OC = 256, 128, 192
    inp, w, dout = gen(41, (BT, C), 1.0), gen(42, (OC, C), 0.02), gen(43, (BT, OC), 1e-3)
    r = oracle.linear_backward(f32(dout), f32(inp), f32(w))
    # frozen weights: only dinp
    dinp = Guarded((BT, C), torch.bfloat16)
    nb.nb_linear_backward_ex(dinp.t, None, None, dout, None, w, None, None, BT, C, OC, 0, 0)
    check_bf16(dinp.t, r["dinp"], "dinp only")
    dinp.check()
    # only dweight
    dw = Guarded((OC, C), torch.float32)
    nb.nb_linear_backward_ex(None, dw.t, None, dout, inp, None, None, None, BT, C, OC, 0, 0)
    check_f32(dw.t, r["dweight"], "dweight only")
    # BT == 0: nothing launched; accumulate=0 zeroes the gradients, accumulate=1 leaves them
    dw.t.fill_(5.0)
    db = torch.full((OC,), 5.0, device=DEV)
    e = torch.empty((0, OC), dtype=torch.bfloat16, device=DEV)
    ei = torch.empty((0, C), dtype=torch.bfloat16, device=DEV)
    nb.nb_linear_backward_ex(None, dw.t, db, e.data_ptr() or 16, ei.data_ptr() or 16, w, None, None, 0, C, OC, 0, 1)
    assert torch.all(dw.t == 5.0) and torch.all(db == 5.0)
    nb.nb_linear_backward_ex(None, dw.t, db, e.data_ptr() or 16, ei.data_ptr() or 16, w, None, None, 0, C, OC, 0, 0)
    assert torch.all(dw.t == 0.0) and torch.all(db == 0.0)
    dw.check()


def test_bf16_dweight_variant():
    BT, C, OC = 512, 256, 384
    inp, w, dout = gen(51, (BT, C), 1.0), gen(52, (OC, C), 0.02), gen(53, (BT, OC), 1e-3)
    dw = Guarded((OC, C), torch.bfloat16)
    nb.nb_linear_backward_ex(None, dw.t, None, dout, inp, None, None, None, BT, C, OC, 0, 0,
                             nb.DTYPE_BF16)
    r = oracle.linear_backward(f32(dout), f32(inp), f32(w), want=("dweight",))
    check_bf16(dw.t, r["dweight"], "bf16 dweight")
    dw.check()


def test_bounded_wait_reports_timeout_and_context_survives():
    nb.nb_debug_wait_timeout(2000)
    with pytest.raises(nb.NbError) as e:
        nb.nb_check_status()
    assert e.value.code == nb.NB_ERR_TIMEOUT
    nb.nb_check_status()  # status word cleared; the context still works:
    run_layer_full(128, 64, 256, nb.ACT_NONE, seed=61)


def test_gemm_kernel_time_out_exit_and_recovery():
    """The GEMM kernel's own abort path: a producer that stops half way makes the issuer's bounded
    wait expire; the kernel must return by itself (no trap, no fault), report which wait gave up,
    leave the canaries around its output alone, and the next call on the same context must be right."""
    inp, w = gen(91, (128, 256), 1.0), gen(92, (256, 256), 0.02)
    out = Guarded((128, 256), torch.bfloat16)
    nb.nb_debug_gemm_timeout(out.t, inp, w, 3000)
    with pytest.raises(nb.NbError) as e:
        nb.nb_check_status()
    assert e.value.code == nb.NB_ERR_TIMEOUT
    assert "wait id 302" in str(e.value)  # the issuer's wait for the third stage
    out.check("aborted GEMM")
    nb.nb_check_status()  # cleared
    nb.nb_linear_forward_ex(out.t, None, inp, w, None, 128, 256, 256, nb.ACT_NONE)
    o_ref, _ = oracle.linear_forward(f32(inp), f32(w))
    check_bf16(out.t, o_ref, "the same product after the aborted one")
    out.check("after recovery")
    run_layer_full(392, 328, 528, nb.ACT_GELU, seed=93)


def test_other_stream():
    s = torch.cuda.Stream()
    BT, C, OC = 512, 256, 512
    inp, w = gen(71, (BT, C), 1.0), gen(72, (OC, C), 0.02)
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        out, _ = nb.linear_forward(inp, w, None, nb.ACT_NONE)
    s.synchronize()
    o_ref, _ = oracle.linear_forward(f32(inp), f32(w))
    check_bf16(out, o_ref, "out on side stream")


# --------------------------------------------------------------------------- full-size, sampled

def _fwd_sampled(name, inp, w, b, act, out, pre, seed, nrows=48, ncols=24):
    """Compare sampled full rows and full columns of out / pre with the oracle."""
    BT, OC = inp.shape[0], w.shape[0]
    H = OC // 2
    rows = sample_indices(BT, nrows, seed)
    o_ref, p_ref = oracle.linear_forward(f32(inp[rows]), f32(w), f32(b) if b is not None else None, act)
    check_bf16(out[rows], o_ref, name + " out rows")
    if pre is not None:
        check_bf16(pre[rows], p_ref, name + " pre rows")
    ocols = H if act == nb.ACT_SWIGLU else OC
    cols = sample_indices(ocols, ncols, seed + 1)
    wsel = np.concatenate([cols, cols + H]) if act == nb.ACT_SWIGLU else cols
    wsel_t = torch.as_tensor(wsel, device=DEV)
    o_ref, p_ref = oracle.linear_forward(f32(inp), f32(w[wsel_t]),
                                         f32(b[wsel_t]) if b is not None else None, act)
    check_bf16(out[:, torch.as_tensor(cols, device=DEV)], o_ref, name + " out cols")
    if pre is not None:
        check_bf16(pre[:, wsel_t], p_ref, name + " pre cols")
    # 16,384 scattered elements: a random 128 x 128 sub-grid (each element its own dot product)
    gr = torch.as_tensor(sample_indices(BT, 128, seed + 2), device=DEV)
    gc = sample_indices(ocols, 128, seed + 3)
    gsel = torch.as_tensor(np.concatenate([gc, gc + H]) if act == nb.ACT_SWIGLU else gc, device=DEV)
    o_ref, p_ref = oracle.linear_forward(f32(inp[gr]), f32(w[gsel]),
                                         f32(b[gsel]) if b is not None else None, act)
    check_bf16(out[gr][:, torch.as_tensor(gc, device=DEV)], o_ref, name + " out grid")
    if pre is not None:
        check_bf16(pre[gr][:, gsel], p_ref, name + " pre grid")
    # a stratified grid: one row in every 32-row box and one column in every 64-column box of the
    # result, compared at their crossings, so that every tile and every 32 x 64 box an epilogue
    # warp stores holds an element the oracle has checked
    sr = torch.as_tensor(stratified_indices(BT, 32, seed + 4), device=DEV)
    sc = stratified_indices(ocols, 64, seed + 5)
    ssel = torch.as_tensor(np.concatenate([sc, sc + H]) if act == nb.ACT_SWIGLU else sc, device=DEV)
    o_ref, p_ref = oracle.linear_forward(f32(inp[sr]), f32(w[ssel]),
                                         f32(b[ssel]) if b is not None else None, act)
    check_bf16(out[sr][:, torch.as_tensor(sc, device=DEV)], o_ref, name + " out stratified")
    if pre is not None:
        check_bf16(pre[sr][:, ssel], p_ref, name + " pre stratified")


def _bwd_sampled(name, dz, inp, w, dinp, dw, db, seed, inp_pre=None, dw_prev=None, nrows=48, ncols=8,
                 check_dinp_cols=True):
    """dz is the gradient that entered the products (after any activation derivative)."""
    BT, (OC, C) = dz.shape[0], w.shape
    if dinp is not None:
        rows = sample_indices(BT, nrows, seed)
        r = oracle.linear_backward(f32(dz[rows]), None, f32(w),
                                   inp_pre=f32(inp_pre[rows]) if inp_pre is not None else None,
                                   want=("dinp",))
        check_bf16(dinp[rows], r["dinp"], name + " dinp rows")
        if check_dinp_cols and BT * OC <= 2e8:
            cols = torch.as_tensor(sample_indices(C, ncols, seed + 1), device=DEV)
            r = oracle.linear_backward(f32(dz), None, f32(w[:, cols]),
                                       inp_pre=f32(inp_pre[:, cols]) if inp_pre is not None else None,
                                       want=("dinp",))
            check_bf16(dinp[:, cols], r["dinp"], name + " dinp cols")
    if dw is not None:
        orow = torch.as_tensor(sample_indices(OC, nrows, seed + 2), device=DEV)
        r = oracle.linear_backward(f32(dz[:, orow]), f32(inp), f32(w[orow]), want=("dweight",))
        ref = r["dweight"] + (dw_prev[orow.cpu().numpy()] if dw_prev is not None else 0.0)
        check_f32(dw[orow], ref, name + " dweight rows")
        ccol = torch.as_tensor(sample_indices(C, ncols, seed + 3), device=DEV)
        if BT * OC <= 2e8:
            r = oracle.linear_backward(f32(dz), f32(inp[:, ccol]), f32(w[:, ccol]), want=("dweight",))
            ref = r["dweight"] + (dw_prev[:, ccol.cpu().numpy()] if dw_prev is not None else 0.0)
            check_f32(dw[:, ccol], ref, name + " dweight cols")
    if db is not None:
        check_f32(db, oracle.reduce_dbias(f32(dz)), name + " dbias")
    # stratified grids (see _fwd_sampled): dinp in 32 x 64 bf16 boxes, dweight in 32 x 32 fp32 boxes
    if dinp is not None:
        sr = torch.as_tensor(stratified_indices(BT, 32, seed + 4), device=DEV)
        sc = torch.as_tensor(stratified_indices(C, 64, seed + 5), device=DEV)
        r = oracle.linear_backward(f32(dz[sr]), None, f32(w[:, sc]),
                                   inp_pre=f32(inp_pre[sr][:, sc]) if inp_pre is not None else None,
                                   want=("dinp",))
        check_bf16(dinp[sr][:, sc], r["dinp"], name + " dinp stratified")
    if dw is not None:
        so = torch.as_tensor(stratified_indices(OC, 32, seed + 6), device=DEV)
        sc = torch.as_tensor(stratified_indices(C, 32, seed + 7), device=DEV)
        r = oracle.linear_backward(f32(dz[:, so]), f32(inp[:, sc]), f32(w[so][:, sc]), want=("dweight",))
        ref = r["dweight"] + (dw_prev[so.cpu().numpy()][:, sc.cpu().numpy()] if dw_prev is not None else 0.0)
        check_f32(dw[so][:, sc], ref, name + " dweight stratified")


def test_config3_lm_head_full_size_sampled():
    """Workload 3: tied head at B=16, T=1024: [16384, 768] x [50304, 768]^T, no bias, padded rows."""
    BT, C, OC = 16384, 768, shapes.VOCAB_PADDED
    inp = gen(synth.tensor_seed(3, 0, 0), (BT, C), 1.0)
    w = synth.zero_pad_vocab_rows(gen(synth.tensor_seed(3, 0, 1), (OC, C), 0.02))
    dout = synth.zero_pad_vocab_cols(gen(synth.tensor_seed(3, 0, 3), (BT, OC), 1e-4))
    logits, _ = nb.linear_forward(inp, w, None, nb.ACT_NONE)
    assert torch.all(logits[:, shapes.VOCAB_REAL:] == 0)  # padding rows of the weight: exact zeros
    _fwd_sampled("head", inp, w, None, nb.ACT_NONE, logits, None, seed=301)
    del logits
    dinp, dw, _ = nb.linear_backward(dout, inp, w, need_dbias=False)
    assert torch.all(dw[shapes.VOCAB_REAL:] == 0)  # padding columns of dlogits: no gradient
    _bwd_sampled("head", dout, inp, w, dinp, dw, None, seed=311, check_dinp_cols=False)
    # second micro-step accumulates into the same buffer (read-modify-write of 155 MB)
    prev = f32(dw).astype(np.float64)
    nb.linear_backward(dout, inp, w, dweight=dw, accumulate=True, need_dinp=False, need_dbias=False)
    orow = sample_indices(OC, 48, 313)
    assert rel_frob(f32(dw[torch.as_tensor(orow, device=DEV)]), 2 * prev[orow]) < 1e-5


def test_config4_block_and_head_at_full_batch_sampled():
    """Workload 4 (one block at B=16, T=1024 and two accumulation steps), sampled: includes the
    fused GELU backward in proj's dgrad."""
    BT = 16384
    blk = shapes.gpt2_block()
    for li, s in enumerate(blk):
        w = gen(synth.tensor_seed(4, li, 1), (s.OC, s.C), s.w_std)
        b = gen(synth.tensor_seed(4, li, 2), (s.OC,), 0.02)
        dw = torch.empty((s.OC, s.C), dtype=torch.float32, device=DEV)
        db = torch.empty((s.OC,), dtype=torch.float32, device=DEV)
        dw_prev = None
        for ms in range(2):
            inp = gen(synth.tensor_seed(4, li, 0, ms), (BT, s.C), 1.0)
            dout = gen(synth.tensor_seed(4, li, 3, ms), (BT, s.OC), 1e-3)
            out, pre = nb.linear_forward(inp, w, b, s.act)
            if ms == 0:
                _fwd_sampled(s.name, inp, w, b, s.act, out, pre, seed=400 + li)
            inp_pre = gen(synth.tensor_seed(4, li, 4, ms), (BT, s.C), 1.0) if s.fused_gelu_bwd else None
            dinp, _, _ = nb.linear_backward(dout, inp, w, inp_pre_act=inp_pre, dweight=dw, dbias=db,
                                            accumulate=ms > 0)
            if ms == 0:
                _bwd_sampled(s.name, dout, inp, w, dinp, dw, db, seed=410 + li, inp_pre=inp_pre)
                dw_prev = f32(dw).astype(np.float64)
                db_prev = f32(db).astype(np.float64)
            else:
                _bwd_sampled(s.name + " step2", dout, inp, w, None, dw, None, seed=420 + li,
                             dw_prev=dw_prev)
                check_f32(db, db_prev + oracle.reduce_dbias(f32(dout)), s.name + " dbias step2")


def test_config5_adapter_shapes_sampled():
    """Workload 5: Qwen3-0.6B-shaped linears at B=8, T=2048, no bias, SwiGLU fused in gate|up."""
    BT = 16384
    for li, s in enumerate(shapes.qwen3_block()):
        inp = gen(synth.tensor_seed(5, li, 0), (BT, s.C), 1.0)
        w = gen(synth.tensor_seed(5, li, 1), (s.OC, s.C), 0.02)
        dout = gen(synth.tensor_seed(5, li, 3), (BT, s.out_cols), 1e-3)
        out, pre = nb.linear_forward(inp, w, None, s.act)
        _fwd_sampled(s.name, inp, w, None, s.act, out, pre, seed=500 + li, nrows=32, ncols=16)
        # 5a: with wgrad; 5b (frozen base): dinp only
        dinp, dw, _ = nb.linear_backward(dout, inp, w, pre_act=pre, act=s.act, need_dbias=False)
        dinp_b, _, _ = nb.linear_backward(dout, inp, w, pre_act=pre, act=s.act, need_dweight=False,
                                          need_dbias=False)
        assert torch.equal(dinp, dinp_b)
        if s.act == nb.ACT_SWIGLU:
            rows = sample_indices(BT, 32, 520 + li)
            r = oracle.linear_backward(f32(dout[rows]), None, f32(w), pre=f32(pre[rows]),
                                       act=oracle.ACT_SWIGLU, want=("dinp", "dz"))
            check_bf16(dinp[rows], r["dinp"], s.name + " dinp rows")
            orow = sample_indices(s.OC, 32, 521 + li)
            ot = torch.as_tensor(orow, device=DEV)
            # dweight rows need dz columns: take them from the oracle's dz for all rows
            rz = oracle.linear_backward(f32(dout), None, f32(w), pre=f32(pre), act=oracle.ACT_SWIGLU,
                                        want=("dz",))
            dzs = rz["dz"][:, orow].astype(np.float32)
            rw = oracle.linear_backward(dzs, f32(inp), f32(w[ot]), want=("dweight",))
            check_f32(dw[ot], rw["dweight"], s.name + " dweight rows")
        else:
            _bwd_sampled(s.name, dout, inp, w, dinp, dw, None, seed=510 + li, nrows=32, ncols=8)


def test_run_to_run_determinism_report():
    """Forward and dgrad involve no atomics: repeated runs must agree bit for bit. wgrad / dbias sum
    split-K slices and row blocks with reduce-adds in any order, so only closeness is required; the
    observed state is printed (pytest -s) as the determinism report."""
    BT, C, OC = 4096, 768, 2304
    inp, w, b = gen(81, (BT, C), 1.0), gen(82, (OC, C), 0.02), gen(83, (OC,), 0.02)
    dout = gen(84, (BT, OC), 1e-3)
    outs, dinps, dws, dbs = [], [], [], []
    for _ in range(3):
        out, pre = nb.linear_forward(inp, w, b, nb.ACT_GELU)
        dinp, dw, db = nb.linear_backward(dout, inp, w)
        torch.cuda.synchronize()
        outs.append((out.clone(), pre.clone()))
        dinps.append(dinp.clone())
        dws.append(dw.clone())
        dbs.append(db.clone())
    for i in (1, 2):
        assert torch.equal(outs[i][0], outs[0][0]) and torch.equal(outs[i][1], outs[0][1])
        assert torch.equal(dinps[i], dinps[0])
        assert rel_frob(f32(dws[i]), f32(dws[0])) < 1e-5
        assert rel_frob(f32(dbs[i]), f32(dbs[0])) < 1e-5
    print("determinism: forward bitwise, dgrad bitwise, dweight bitwise =",
          all(torch.equal(dws[i], dws[0]) for i in (1, 2)), ", dbias bitwise =",
          all(torch.equal(dbs[i], dbs[0]) for i in (1, 2)))


def test_master_weight_cast_bit_exact():
    """fp32 -> bf16 cast: integer work, so bit-exact against the oracle, ragged tails included."""
    g = torch.Generator().manual_seed(9)
    for n in (1, 7, 8, 9, 4099, 768 * 2304, 50304 * 768 + 5):
        x = (torch.randn(n, generator=g) * 0.02)
        if n > 64:  # special values: ties, carries, infinities, subnormals, zeros
            sp = torch.tensor([0x3F808000, 0x3F818000, 0x3F808001, 0x7F7FFFFF, 0x7F800000, 0x00008000,
                               0x00018000, 0x00000000], dtype=torch.int64).to(torch.int32).view(torch.float32)
            x[:8] = sp
            x[8:16] = -sp
        xd = x.to(DEV)
        dst = Guarded((n,), torch.bfloat16) if n % 8 == 0 else None
        out = dst.t if dst else torch.empty(n, dtype=torch.bfloat16, device=DEV)
        nb.nb_cast_f32_to_bf16(out, xd, n)
        got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got, oracle.cast_f32_bf16(x.numpy())), n
        if dst:
            dst.check("cast")


# --------------------------------------------------------------------------- head + cross-entropy

def _ce_case(BT, C, Vp, V, seed, full=True):
    inp = gen(seed, (BT, C), 1.0)
    w = gen(seed + 1, (Vp, C), 0.02 if full else 0.05)
    if V < Vp:
        w[V:].zero_()
    g = torch.Generator().manual_seed(seed)
    targets = torch.randint(0, V, (BT,), generator=g, dtype=torch.int32).to(DEV)
    logits = Guarded((BT, Vp), torch.bfloat16)
    loss = Guarded((BT,), torch.float32)
    lse = Guarded((BT,), torch.float32)
    nb.nb_lm_head_ce_forward(logits.t, loss.t, lse.t, inp, w, targets, BT, C, Vp, V)
    ref_logits, _ = nb.linear_forward(inp, w, None, nb.ACT_NONE)
    assert torch.equal(logits.t, ref_logits)  # the statistics ride along: same logits, bit for bit
    for gbuf in (logits, loss, lse):
        gbuf.check("ce forward")
    return inp, w, targets, logits.t, loss.t, lse.t


@pytest.mark.parametrize("BT,C,Vp,V", [(1, 8, 16, 11), (136, 72, 520, 517), (300, 328, 1040, 1000),
                                        (512, 768, 5120, 5000)])
def test_head_cross_entropy_small_every_element(BT, C, Vp, V):
    inp, w, targets, logits, loss, lse = _ce_case(BT, C, Vp, V, 600 + BT, full=False)
    l_ref, lse_ref, d_ref = oracle.cross_entropy(f32(logits), targets.cpu().numpy(), V, 1.0 / BT)
    assert np.max(np.abs(f32(lse) - lse_ref)) < 2e-4 * np.max(np.abs(lse_ref)) + 1e-4
    assert np.max(np.abs(f32(loss) - l_ref)) < 2e-4 * np.max(np.abs(lse_ref)) + 1e-4
    for in_place in (False, True):
        src = logits.clone()
        dl = src if in_place else torch.empty_like(src)
        nb.nb_ce_backward(dl, src, lse, targets, 1.0 / BT, BT, Vp, V)
        assert torch.all(dl[:, V:] == 0)  # padding: exactly no gradient
        check_bf16(dl, d_ref, "dlogits")
    # an out-of-range target is loud, not silent
    bad = targets.clone()
    bad[0] = V
    loss2 = torch.zeros_like(loss)
    nb.nb_lm_head_ce_forward(logits, loss2, lse, inp, w, bad, BT, C, Vp, V)
    assert torch.isnan(loss2[0]) and not torch.isnan(loss2[1:]).any()


def test_head_cross_entropy_full_size_sampled():
    """B=16, T=1024 micro-batch on the padded vocabulary: losses of every row against the oracle on
    sampled rows, the gradient on sampled rows, and the chain into the head's backward."""
    BT, C, Vp, V = 16384, 768, shapes.VOCAB_PADDED, shapes.VOCAB_REAL
    inp, w, targets, logits, loss, lse = _ce_case(BT, C, Vp, V, 700)
    rows = sample_indices(BT, 48, 701)
    rt = torch.as_tensor(rows, device=DEV)
    gscale = 1.0 / BT
    l_ref, lse_ref, d_ref = oracle.cross_entropy(f32(logits[rt]), targets[rt].cpu().numpy(), V, gscale)
    assert np.max(np.abs(f32(lse[rt]) - lse_ref)) < 1e-3
    assert np.max(np.abs(f32(loss[rt]) - l_ref)) < 1e-3
    # logits ~ N(0, C * 0.02^2): the expected loss at initialisation is log V + variance / 2
    assert abs(float(loss.mean()) - (math.log(V) + 0.5 * C * 0.02 ** 2)) < 0.02
    dl = torch.empty_like(logits)
    nb.nb_ce_backward(dl, logits, lse, targets, gscale, BT, Vp, V)
    assert torch.all(dl[:, V:] == 0)
    check_bf16(dl[rt], d_ref, "dlogits rows")
    rowsum = dl.float().sum(1)
    assert float(rowsum.abs().max()) < 2e-2 * gscale  # softmax - onehot sums to ~0 (bf16 rounding)
    dinp, dw, _ = nb.linear_backward(dl, inp, w, need_dbias=False)
    assert torch.all(dw[V:] == 0)
    _bwd_sampled("head after ce", dl, inp, w, dinp, dw, None, seed=702, check_dinp_cols=False)


def test_flat_gradient_buckets_give_the_same_gradients_on_one_rank():
    """The data-parallel step on one rank (no collective runs): gradients written through the flat
    bucket buffer equal those of the plain step, and every view meets the kernels' alignment rule."""
    from paper_2609_28568_b200 import dp
    from paper_2609_28568_b200.stack import LinearStack
    a = LinearStack("gpt2_block", BT=384, micro_steps=2, device=DEV, config_id=2)
    a.step()
    b = LinearStack("gpt2_block", BT=384, micro_steps=2, device=DEV, config_id=2, shared_weights=True)
    gb = b.attach_gradient_buckets(bucket_bytes=4 << 20)
    red = dp.GradAllReducer(gb, None)
    b.step_dp(red)
    torch.cuda.synchronize()
    assert red.launched == len(gb.buckets) >= 2
    for La, Lb in zip(a.layers, b.layers):
        assert Lb.dweight.data_ptr() % 16 == 0
        assert rel_frob(f32(Lb.dweight), f32(La.dweight)) < 1e-5
        assert rel_frob(f32(Lb.dbias), f32(La.dbias)) < 1e-5


def test_data_parallel_step_with_the_second_stream_orders_its_accumulations():
    """`step_dp` on a stack that issues weight gradients on a second stream: the micro-steps before
    the last leave accumulations on that stream, the last one (and the reducer's events) runs on the
    current stream. The gradients must equal those of the plain step."""
    from paper_2609_28568_b200 import dp
    from paper_2609_28568_b200.stack import LinearStack
    a = LinearStack("gpt2_block", BT=2048, micro_steps=4, device=DEV, config_id=2)
    a.step()
    b = LinearStack("gpt2_block", BT=2048, micro_steps=4, device=DEV, config_id=2, wgrad_stream=True)
    gb = b.attach_gradient_buckets(bucket_bytes=4 << 20)
    red = dp.GradAllReducer(gb, None)
    for _ in range(3):
        b.step_dp(red)
    torch.cuda.synchronize()
    for La, Lb in zip(a.layers, b.layers):
        assert rel_frob(f32(Lb.dweight), f32(La.dweight)) < 1e-5, La.spec.name
        assert rel_frob(f32(Lb.dbias), f32(La.dbias)) < 1e-5, La.spec.name
        assert torch.equal(Lb.dinp, La.dinp), La.spec.name


@pytest.mark.parametrize("act", [nb.ACT_NONE, nb.ACT_GELU])
def test_bias_reaches_every_tile_full_tensor(act):
    """Every element of a many-tile result carries ITS column's bias: the result with a large bias
    equals the bias-free result plus the bias, to the rounding of the two bf16 conversions. (The
    epilogue warps keep the bias in buffers they reuse from tile to tile without a barrier.)"""
    BT, C, OC = 16384, 768, 3072 if act == nb.ACT_GELU else 2304
    inp = gen(7001, (BT, C), 1.0)
    w = gen(7002, (OC, C), 0.02)
    b = gen(7003, (OC,), 1.0)
    out_b = torch.empty((BT, OC), dtype=torch.bfloat16, device=DEV)
    pre_b = torch.empty((BT, OC), dtype=torch.bfloat16, device=DEV) if act != nb.ACT_NONE else None
    out_0 = torch.empty_like(out_b)
    pre_0 = torch.empty_like(out_b) if act != nb.ACT_NONE else None
    for _ in range(3):  # repeated launches: persistent CTAs walk different tile sequences
        nb.nb_linear_forward_ex(out_b, pre_b, inp, w, b, BT, C, OC, act)
    nb.nb_linear_forward_ex(out_0, pre_0, inp, w, None, BT, C, OC, act)
    got = (pre_b if act != nb.ACT_NONE else out_b).float()
    base = (pre_0 if act != nb.ACT_NONE else out_0).float()
    expect = base + b.float()[None, :]
    err = (got - expect).abs()
    bound = 2.0 ** -7 * expect.abs() + 2.0 ** -8 * base.abs() + 1e-3
    bad = err > bound
    assert not bool(bad.any()), f"{int(bad.sum())} elements carry a wrong bias, worst {float(err.max()):.3f}"


def test_results_beyond_two_to_the_31_elements():
    """The largest case: 49152 rows on the padded vocabulary, 2.47e9 logits (> 2^31 elements, 4.9 GB).
    Rows from the far end of every tensor are checked against the oracle: head forward with the
    statistics, the in-place gradient of the loss, and the head's backward products."""
    BT, C, Vp, V = 49152, 768, shapes.VOCAB_PADDED, shapes.VOCAB_REAL
    assert BT * Vp > 2 ** 31
    inp = gen(7100, (BT, C), 1.0)
    w = gen(7101, (Vp, C), 0.02)
    w[V:].zero_()
    g = torch.Generator().manual_seed(7102)
    targets = torch.randint(0, V, (BT,), generator=g, dtype=torch.int32).to(DEV)
    logits = torch.empty((BT, Vp), dtype=torch.bfloat16, device=DEV)
    loss = torch.empty((BT,), dtype=torch.float32, device=DEV)
    lse = torch.empty((BT,), dtype=torch.float32, device=DEV)
    nb.nb_lm_head_ce_forward(logits, loss, lse, inp, w, targets, BT, C, Vp, V)
    rows = np.concatenate([sample_indices(BT, 16, 7103), np.arange(BT - 8, BT)])
    rows = np.unique(rows)
    rt = torch.as_tensor(rows, device=DEV)
    o_ref, _ = oracle.linear_forward(f32(inp[rt]), f32(w))
    check_bf16(logits[rt], o_ref, "logits rows")
    gscale = 1.0 / BT
    l_ref, lse_ref, d_ref = oracle.cross_entropy(f32(logits[rt]), targets[rt].cpu().numpy(), V, gscale)
    assert np.max(np.abs(f32(loss[rt]) - l_ref)) < 1e-3
    assert bool(torch.isfinite(loss).all())
    nb.nb_ce_backward(logits, logits, lse, targets, gscale, BT, Vp, V)  # in place: logits become dlogits
    dl = logits
    check_bf16(dl[rt], d_ref, "dlogits rows")
    assert torch.all(dl[BT - 64:, V:] == 0)
    dinp, dw, _ = nb.linear_backward(dl, inp, w, need_dbias=False)
    r = oracle.linear_backward(f32(dl[rt]), None, f32(w), want=("dinp",))
    check_bf16(dinp[rt], r["dinp"], "dinp rows")
    # weight-gradient rows (sums over all 49152 rows): a few vocabulary rows, every column
    orow = sample_indices(V, 6, 7104)
    ot = torch.as_tensor(orow, device=DEV)
    rw = oracle.linear_backward(f32(dl[:, ot]), f32(inp), f32(w[ot]), want=("dweight",))
    check_f32(dw[ot], rw["dweight"], "dweight rows")
    assert torch.all(dw[V:] == 0)


@pytest.mark.parametrize("model,config_id", [("gpt2_block", 2), ("gpt2", 4), ("qwen3", 5)])
def test_graph_replay_of_a_step_equals_the_eager_step(model, config_id):
    """bench.py times a captured CUDA graph of the step: the replay must produce what the eager
    launches produce (outputs and dinp bit for bit, the atomically accumulated gradients to rounding)
    with programmatic dependent launch on, both for the own-activation backward (config 2) and the
    chained fc -> proj form with the fused GELU backward (config 4)."""
    from paper_2609_28568_b200.stack import LinearStack
    BT = 2048 if model == "gpt2_block" else 1024
    a = LinearStack(model, BT=BT, micro_steps=3, device=DEV, config_id=config_id)
    a.step()
    b = LinearStack(model, BT=BT, micro_steps=3, device=DEV, config_id=config_id)
    b.step()  # warm-up: workspace and tensor maps exist before the capture
    for L in b.layers:
        L.dweight.fill_(7.0)
        if L.dbias is not None:
            L.dbias.fill_(7.0)
        L.dinp.zero_()
        L.out.zero_()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cap):
            b.step()
    torch.cuda.current_stream().wait_stream(cap)
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    for La, Lb in zip(a.layers, b.layers):
        assert torch.equal(Lb.out, La.out), La.spec.name
        assert torch.equal(Lb.dinp, La.dinp), La.spec.name
        assert rel_frob(f32(Lb.dweight[:64]), f32(La.dweight[:64])) < 1e-5, La.spec.name
        assert rel_frob(f32(Lb.dweight[-64:]), f32(La.dweight[-64:])) < 1e-5, La.spec.name
        if La.dbias is not None:
            assert rel_frob(f32(Lb.dbias), f32(La.dbias)) < 1e-5, La.spec.name


@pytest.mark.parametrize("model,config_id", [("gpt2_block", 2), ("gpt2", 4), ("qwen3", 5)])
def test_weight_gradients_on_a_second_stream_match_the_single_stream_step(model, config_id):
    """The stack driver's two-stream backward (dgrad chain on one stream, dweight / dbias on another)
    orders every buffer the two streams share: same gradients, outputs and dinp as the single-stream
    step, eagerly and when the step is replayed from a captured CUDA graph (where a launch that
    follows a cross-stream wait gives up programmatic dependent launch)."""
    from paper_2609_28568_b200.stack import LinearStack
    BT = 2048 if model == "gpt2_block" else 1024
    a = LinearStack(model, BT=BT, micro_steps=3, device=DEV, config_id=config_id)
    a.step()
    b = LinearStack(model, BT=BT, micro_steps=3, device=DEV, config_id=config_id, wgrad_stream=True)
    b.step()
    torch.cuda.synchronize()

    def same(tag):
        for La, Lb in zip(a.layers, b.layers):
            assert rel_frob(f32(Lb.dweight[:64]), f32(La.dweight[:64])) < 1e-5, (tag, La.spec.name)
            assert rel_frob(f32(Lb.dweight[-64:]), f32(La.dweight[-64:])) < 1e-5, (tag, La.spec.name)
            if La.dbias is not None:
                assert rel_frob(f32(Lb.dbias), f32(La.dbias)) < 1e-5, (tag, La.spec.name)
            assert torch.equal(Lb.dinp, La.dinp), (tag, La.spec.name)
            assert torch.equal(Lb.out, La.out), (tag, La.spec.name)
    same("eager")
    for L in b.layers:
        L.dweight.fill_(7.0)
        if L.dbias is not None:
            L.dbias.fill_(7.0)
        L.dinp.zero_()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cap):
            b.step()
    torch.cuda.current_stream().wait_stream(cap)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    same("graph")


def _round_bf16(a: np.ndarray) -> np.ndarray:
    """The oracle's fp64 values as the bf16 numbers a stored activation would hold."""
    return torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16).float().numpy()


@pytest.mark.parametrize("wgrad_stream", [False, True])
def test_timed_path_block_graph_replay_matches_the_oracle(wgrad_stream):
    """The path bench.py times (the stack driver's step inside a replayed CUDA graph, one launch per
    layer backward on one stream or dgrad / wgrad chains on two) against the oracle as a whole:
    one GPT-2 block, four accumulating micro-steps, fc.out feeding proj and proj's fused dgrad
    feeding fc's backward. The last micro-step's activations and input gradients are compared with
    the oracle fed the very buffers the GPU calls read; the accumulated weight and bias gradients
    with the oracle's own chain over all four micro-steps, rounding to bf16 where the path stores
    an activation (fc.out, fc.pre, proj.dinp)."""
    from paper_2609_28568_b200.stack import LinearStack
    BT, MS = 384, 4
    st = LinearStack("gpt2_block", BT=BT, micro_steps=MS, device=DEV, config_id=2, wgrad_stream=wgrad_stream)
    st.step()  # warm-up outside the capture: tensor maps and schedules exist
    for L in st.layers:
        L.dweight.fill_(3.0)
        L.dbias.fill_(3.0)
        L.out.zero_()
        L.dinp.zero_()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cap):
            st.step()
    torch.cuda.current_stream().wait_stream(cap)
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    nb.nb_check_status()
    qkv, aproj, fc, proj = st.layers
    last = MS - 1
    # ---- the last micro-step, call by call, on the buffers the calls read
    for L in st.layers:
        s = L.spec
        x = fc.out if L is proj else L.inp[last]
        o_ref, p_ref = oracle.linear_forward(f32(x), f32(L.weight), f32(L.bias), s.act)
        check_bf16(L.out, o_ref, s.name + " out")
        if L.pre is not None:
            check_bf16(L.pre, p_ref, s.name + " pre")
        dz = proj.dinp if L is fc else L.dout[last]
        r = oracle.linear_backward(f32(dz), None, f32(L.weight),
                                   inp_pre=f32(fc.pre) if L is proj else None, want=("dinp",))
        check_bf16(L.dinp, r["dinp"], s.name + " dinp")
    # ---- gradients accumulated over the four micro-steps
    for L in st.layers:
        dw_ref = np.zeros((L.spec.OC, L.spec.C))
        db_ref = np.zeros((L.spec.OC,))
        for ms in range(MS):
            if L is proj:    # its input is fc's stored output of that micro-step
                o, _ = oracle.linear_forward(f32(fc.inp[ms]), f32(fc.weight), f32(fc.bias), oracle.ACT_GELU)
                x, dz = _round_bf16(o), f32(proj.dout[ms])
            elif L is fc:    # its dz is proj's fused dgrad of that micro-step
                _, pz = oracle.linear_forward(f32(fc.inp[ms]), f32(fc.weight), f32(fc.bias), oracle.ACT_GELU)
                r = oracle.linear_backward(f32(proj.dout[ms]), None, f32(proj.weight),
                                           inp_pre=_round_bf16(pz), want=("dinp",))
                x, dz = f32(fc.inp[ms]), _round_bf16(r["dinp"])
            else:
                x, dz = f32(L.inp[ms]), f32(L.dout[ms])
            oracle.linear_backward(dz, x, f32(L.weight), dweight=dw_ref, dbias=db_ref, accumulate=ms > 0,
                                   want=("dweight", "dbias"))
        check_f32(L.dweight, dw_ref, L.spec.name + " dweight over micro-steps")
        check_f32(L.dbias, db_ref, L.spec.name + " dbias over micro-steps")


def test_timed_path_full_stack_graph_replay_sampled_against_the_oracle():
    """The whole GPT-2 stack driver (12 blocks and the tied head, two accumulating micro-steps) in a
    replayed graph: the last block and the head are compared with the oracle on stratified samples
    of every output, from the buffers the GPU calls read."""
    from paper_2609_28568_b200.stack import LinearStack
    BT, MS = 512, 2
    st = LinearStack("gpt2", BT=BT, micro_steps=MS, device=DEV, config_id=4)
    st.step()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cap):
            st.step()
    torch.cuda.current_stream().wait_stream(cap)
    g.replay()
    torch.cuda.synchronize()
    nb.nb_check_status()
    last = MS - 1
    blk = st.layers[-5:-1]
    head = st.layers[-1]
    fc, proj = blk[2], blk[3]
    for i, L in enumerate(blk + [head]):
        s = L.spec
        x = fc.out if L is proj else L.inp[last]
        _fwd_sampled("stack " + s.name, x, L.weight, L.bias, s.act, L.out, L.pre, seed=900 + 10 * i,
                     nrows=8, ncols=8)
        dz = proj.dinp if L is fc else L.dout[last]
        # the weight gradient holds both micro-steps: subtract nothing, compare the sum
        _bwd_sampled("stack " + s.name, dz, x, L.weight, L.dinp, None, None, seed=905 + 10 * i,
                     inp_pre=fc.pre if L is proj else None, nrows=8, ncols=4)
        if L is not proj and L is not fc:   # inputs of both micro-steps are still in memory
            so = torch.as_tensor(stratified_indices(s.OC, 32, 907 + 10 * i), device=DEV)
            sc = torch.as_tensor(stratified_indices(s.C, 32, 908 + 10 * i), device=DEV)
            ref = 0.0
            for ms in range(MS):
                r = oracle.linear_backward(f32(L.dout[ms][:, so]), f32(L.inp[ms][:, sc]), f32(L.weight[so][:, sc]),
                                           want=("dweight",))
                ref = ref + r["dweight"]
            check_f32(L.dweight[so][:, sc], ref, "stack " + s.name + " dweight over micro-steps")
            if L.dbias is not None:
                ref_b = sum(oracle.reduce_dbias(f32(L.dout[ms])) for ms in range(MS))
                check_f32(L.dbias, ref_b, "stack " + s.name + " dbias over micro-steps")


def test_end_to_end_path_of_the_bench_returns_the_step_gradients():
    """The bench's end-to-end leg streams every micro-step's inputs from pinned host memory on a copy
    stream, computes on the main stream and reads the gradients back on a third one, steps overlapping.
    What arrives on the host after three such steps must be the gradients of one plain step (the inputs
    are the same every step; fp32 sums may differ in their last bits)."""
    import argparse
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    from paper_2609_28568_b200.stack import LinearStack
    stack = LinearStack("gpt2_block", 1024, 3, device=torch.device("cuda", 0), config_id=2)
    stack.step()
    torch.cuda.synchronize()
    want = [g.clone() for g in stack.gradient_tensors()]
    for g in stack.gradient_tensors():
        g.fill_(float("nan"))
    args = argparse.Namespace(e2e_steps=3)
    res, host = bench.measure_e2e(torch, nb, stack, args, None, torch.device("cuda", 0), 1.0, 1, return_host=True)
    assert res["h2d_bytes_per_step"] > 0 and res["d2h_bytes_per_step"] == sum(w.numel() * 4 for w in want)
    for h, w in zip(host, want):
        assert torch.isfinite(h).all()
        assert rel_frob(h.numpy(), f32(w)) < 1e-5


def test_layer_backward_beyond_the_one_launch_schedule_falls_back_to_separate_launches():
    """A layer with more dinp tiles than the one-launch schedule's round mask holds (79 x 64 tiles for 74
    CTA pairs) is declined by the planner; the call must then issue dinp and dweight as launches of their
    own and still give the oracle's results (sampled rows, columns and a stratified grid; dbias whole)."""
    BT, C, OC = 20000, 16384, 8
    with pytest.raises(nb.NbError):
        nb.nb_debug_layer_bwd_plan(BT, C, OC, 74, False)
    inp, w = gen(7001, (BT, C), 1.0), gen(7002, (OC, C), 0.05)
    dout = gen(7003, (BT, OC), 1e-3)
    dinp = Guarded((BT, C), torch.bfloat16)
    dw = Guarded((OC, C), torch.float32, fill=4.0)
    db = Guarded((OC,), torch.float32, fill=4.0)
    before = nb.nb_kernel_launches()
    nb.nb_linear_backward_ex(dinp.t, dw.t, db.t, dout, inp, w, None, None, BT, C, OC, nb.ACT_NONE, 0)
    assert nb.nb_kernel_launches() - before == 2   # dinp, and dweight with the bias gradient inside
    _bwd_sampled("fallback", dout, inp, w, dinp.t, dw.t, db.t, seed=77)
    for g, n in ((dinp, "dinp"), (dw, "dweight"), (db, "dbias")):
        g.check(n)


def test_release_and_workspace_growth_refused_during_capture():
    """nb_release drops the library's device state (workspace, status word, tensor-map cache); the next
    call builds it again. With the workspace back at zero, an own-activation backward issued while its
    stream is being captured would have to allocate: it is refused with a message naming
    nb_workspace_reserve, the capture survives and replays what it recorded, and after a reserve the same
    call captures and gives the oracle's bias gradient."""
    nb.nb_check_status()
    nb.nb_release()
    BT, OC = 1024, 520
    dout, pre = gen(7101, (BT, OC), 1e-3), gen(7102, (BT, OC), 1.0)
    x, w = gen(7103, (BT, 64), 1.0), gen(7104, (OC, 64), 0.05)
    out = torch.zeros((BT, OC), dtype=torch.bfloat16, device=DEV)
    db = torch.zeros((OC,), dtype=torch.float32, device=DEV)
    nb.nb_linear_forward_ex(out, None, x, w, None, BT, 64, OC, nb.ACT_NONE)   # state and tensor maps exist again
    torch.cuda.synchronize()
    want_out = out.clone()
    out.zero_()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            nb.nb_linear_forward_ex(out, None, x, w, None, BT, 64, OC, nb.ACT_NONE)
            with pytest.raises(nb.NbError) as ei:
                nb.nb_linear_backward_ex(None, None, db, dout, None, None, pre, None, BT, 8, OC, nb.ACT_GELU, 0)
            assert ei.value.code == nb.NB_ERR_UNSUPPORTED and "nb_workspace_reserve" in str(ei.value)
    torch.cuda.current_stream().wait_stream(s)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want_out)
    nb.nb_workspace_reserve(BT * OC * 2)
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=s):
            nb.nb_linear_backward_ex(None, None, db, dout, None, None, pre, None, BT, 8, OC, nb.ACT_GELU, 0)
    torch.cuda.current_stream().wait_stream(s)
    g2.replay()
    torch.cuda.synchronize()
    dz = f32(dout).astype(np.float64) * oracle.gelu_grad(f32(pre).astype(np.float64))
    check_f32(db, oracle.reduce_dbias(dz.astype(np.float32)), "dbias through a captured own-activation backward")
