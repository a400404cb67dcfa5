"""Pins for the CPU oracle: every function is checked against something that is not the oracle.

Pins used: fixed points from the golden file, odd/even identities of the
activations, library GELU / SiLU and library autograd (an independent derivation
of every gradient), integer-exact products, finite differences, adjoint
identities, linearity of accumulation and the column-sum invariant of dbias.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import ACT_GELU, ACT_NONE, ACT_SWIGLU

torch.manual_seed(0)


def _bf16_vals(shape, std, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * std).to(torch.bfloat16).to(torch.float32).numpy()


def relf(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


# ---------------------------------------------------------------- activations

def test_activation_fixed_points(golden_dir):
    fns = {"gelu": oracle.gelu, "gelu_grad": oracle.gelu_grad,
           "silu": oracle.silu, "silu_grad": oracle.silu_grad}
    n = 0
    for line in open(f"{golden_dir}/activation_fixed_points.txt"):
        if line.startswith("#") or not line.strip():
            continue
        name, x, v = line.split()
        got = fns[name](np.array([float(x)]), "f64")[0]
        assert abs(got - float(v)) < 2e-9, (name, x, got, v)
        got32 = fns[name](np.array([float(x)]), "f32")[0]
        assert abs(got32 - float(v)) < 1e-6, (name, x, got32, v)
        n += 1
    assert n == 26


def test_activation_identities():
    x = np.linspace(-9.0, 9.0, 3601)
    # tanh and the logistic's odd part: f(x) - f(-x) = x ; f'(x) + f'(-x) = 1
    assert np.max(np.abs(oracle.gelu(x) - oracle.gelu(-x) - x)) < 1e-14
    assert np.max(np.abs(oracle.gelu_grad(x) + oracle.gelu_grad(-x) - 1.0)) < 1e-14
    assert np.max(np.abs(oracle.silu(x) - oracle.silu(-x) - x)) < 1e-14
    assert np.max(np.abs(oracle.silu_grad(x) + oracle.silu_grad(-x) - 1.0)) < 1e-14
    # limits: gelu(x) -> x, gelu(-x) -> 0 for large x
    big = np.array([8.0, 12.0, 30.0])
    assert np.allclose(oracle.gelu(big), big, rtol=0, atol=1e-12)
    assert np.allclose(oracle.gelu(-big), 0.0, rtol=0, atol=1e-12)
    assert np.allclose(oracle.gelu_grad(big), 1.0, rtol=0, atol=1e-10)


def test_activations_against_library():
    x = torch.linspace(-7.0, 7.0, 2801, dtype=torch.float64, requires_grad=True)
    y = F.gelu(x, approximate="tanh")
    (gy,) = torch.autograd.grad(y.sum(), x)
    xn = x.detach().numpy()
    assert np.max(np.abs(oracle.gelu(xn) - y.detach().numpy())) < 1e-14
    assert np.max(np.abs(oracle.gelu_grad(xn) - gy.numpy())) < 1e-13
    s = F.silu(x)
    (gs,) = torch.autograd.grad(s.sum(), x)
    assert np.max(np.abs(oracle.silu(xn) - s.detach().numpy())) < 1e-14
    assert np.max(np.abs(oracle.silu_grad(xn) - gs.numpy())) < 1e-13
    # the exact-erf GELU is a different function: the oracle must not be it
    assert np.max(np.abs(oracle.gelu(xn) - F.gelu(x.detach()).numpy())) > 1e-4


def test_activation_derivatives_by_finite_differences():
    x = np.linspace(-5.0, 5.0, 1001)
    h = 1e-5
    fd = (oracle.gelu(x + h) - oracle.gelu(x - h)) / (2 * h)
    assert np.max(np.abs(fd - oracle.gelu_grad(x))) < 1e-9
    fd = (oracle.silu(x + h) - oracle.silu(x - h)) / (2 * h)
    assert np.max(np.abs(fd - oracle.silu_grad(x))) < 1e-9


# ---------------------------------------------------------------- forward

def test_forward_integer_exact():
    """Small integers: every product and sum is exact, so equality is exact."""
    rng = np.random.default_rng(1)
    BT, C, OC = 37, 24, 19
    inp = rng.integers(-8, 9, size=(BT, C)).astype(np.float32)
    w = rng.integers(-8, 9, size=(OC, C)).astype(np.float32)
    b = rng.integers(-8, 9, size=(OC,)).astype(np.float32)
    want = inp.astype(np.int64) @ w.astype(np.int64).T + b.astype(np.int64)
    for dt in ("f32", "f64"):
        out, pre = oracle.linear_forward(inp, w, b, ACT_NONE, dt)
        assert np.array_equal(out.astype(np.int64), want) and np.array_equal(out, pre)
        out, _ = oracle.linear_forward(inp, w, None, ACT_NONE, dt)
        assert np.array_equal(out.astype(np.int64), want - b.astype(np.int64))


def test_forward_identity_weight_and_zero_rows():
    inp = _bf16_vals((9, 16), 1.0, 2)
    b = _bf16_vals((16,), 0.02, 3)
    out, _ = oracle.linear_forward(inp, np.eye(16, dtype=np.float32), b, ACT_NONE, "f64")
    assert np.array_equal(out, inp.astype(np.float64) + b)
    w = _bf16_vals((12, 16), 0.02, 4)
    w[7:] = 0.0  # padding rows of a head produce exactly zero logits
    out, _ = oracle.linear_forward(inp, w, None, ACT_NONE, "f32")
    assert np.all(out[:, 7:] == 0.0) and np.any(out[:, :7] != 0.0)


@pytest.mark.parametrize("act", [ACT_NONE, ACT_GELU, ACT_SWIGLU])
def test_forward_against_library(act):
    BT, C, OC = 33, 40, 26
    inp = _bf16_vals((BT, C), 1.0, 5)
    w = _bf16_vals((OC, C), 0.3, 6)
    b = _bf16_vals((OC,), 0.3, 7)
    z = F.linear(torch.tensor(inp, dtype=torch.float64), torch.tensor(w, dtype=torch.float64),
                 torch.tensor(b, dtype=torch.float64))
    if act == ACT_NONE:
        want = z
    elif act == ACT_GELU:
        want = F.gelu(z, approximate="tanh")
    else:
        want = F.silu(z[:, :OC // 2]) * z[:, OC // 2:]
    out, pre = oracle.linear_forward(inp, w, b, act, "f64")
    assert out.shape == tuple(want.shape)
    assert np.max(np.abs(out - want.numpy())) < 1e-12
    assert np.max(np.abs(pre - z.numpy())) < 1e-12
    out32, _ = oracle.linear_forward(inp, w, b, act, "f32")
    assert relf(out32, want.numpy()) < 1e-6


# ---------------------------------------------------------------- backward

def _autograd(inp, w, b, dout, act, inp_pre=None):
    """Library derivation of the layer's gradients in fp64."""
    W = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    B = torch.tensor(b, dtype=torch.float64, requires_grad=True)
    if inp_pre is not None:  # the input is itself gelu(u): return the gradient w.r.t. u
        u = torch.tensor(inp_pre, dtype=torch.float64, requires_grad=True)
        x, xin = None, F.gelu(u, approximate="tanh")
    else:
        x = torch.tensor(inp, dtype=torch.float64, requires_grad=True)
        u, xin = None, x
    z = F.linear(xin, W, B)
    OC = w.shape[0]
    if act == ACT_NONE:
        y = z
    elif act == ACT_GELU:
        y = F.gelu(z, approximate="tanh")
    else:
        y = F.silu(z[:, :OC // 2]) * z[:, OC // 2:]
    loss = (y * torch.tensor(dout, dtype=torch.float64)).sum()
    leaves = [u if u is not None else x, W, B]
    g = torch.autograd.grad(loss, leaves)
    return [t.numpy() for t in g], z.detach().numpy(), xin.detach().numpy()


@pytest.mark.parametrize("act", [ACT_NONE, ACT_GELU, ACT_SWIGLU])
def test_backward_against_library_autograd(act):
    BT, C, OC = 29, 24, 18
    inp = _bf16_vals((BT, C), 1.0, 11)
    w = _bf16_vals((OC, C), 0.3, 12)
    b = _bf16_vals((OC,), 0.3, 13)
    ocols = OC // 2 if act == ACT_SWIGLU else OC
    dout = _bf16_vals((BT, ocols), 1.0, 14)
    (gx, gw, gb), z, _ = _autograd(inp, w, b, dout, act)
    pre = z.astype(np.float32)  # the oracle is handed the pre-activation as an input
    (gx, gw, gb), _, _ = _autograd_with_pre(inp, w, b, dout, act, pre)
    r = oracle.linear_backward(dout, inp, w, pre=pre if act != ACT_NONE else None, act=act,
                               dtype="f64")
    assert r["dinp"].shape == (BT, C) and r["dweight"].shape == (OC, C)
    assert np.max(np.abs(r["dinp"] - gx)) < 1e-11
    assert np.max(np.abs(r["dweight"] - gw)) < 1e-11
    assert np.max(np.abs(r["dbias"] - gb)) < 1e-11
    r32 = oracle.linear_backward(dout, inp, w, pre=pre if act != ACT_NONE else None, act=act,
                                 dtype="f32")
    for k, ref in (("dinp", gx), ("dweight", gw), ("dbias", gb)):
        assert relf(r32[k], ref) < 2e-6, k


def _autograd_with_pre(inp, w, b, dout, act, pre):
    """As _autograd, but the activation derivative is taken at the given (rounded) `pre`."""
    OC = w.shape[0]
    z = torch.tensor(pre, dtype=torch.float64, requires_grad=True)
    if act == ACT_NONE:
        y = z
    elif act == ACT_GELU:
        y = F.gelu(z, approximate="tanh")
    else:
        y = F.silu(z[:, :OC // 2]) * z[:, OC // 2:]
    (dz,) = torch.autograd.grad((y * torch.tensor(dout, dtype=torch.float64)).sum(), z)
    x = torch.tensor(inp, dtype=torch.float64, requires_grad=True)
    W = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    B = torch.tensor(b, dtype=torch.float64, requires_grad=True)
    g = torch.autograd.grad((F.linear(x, W, B) * dz).sum(), [x, W, B])
    return [t.numpy() for t in g], None, None


def test_backward_fused_input_activation_against_library():
    """dinp * gelu'(inp_pre) equals the gradient w.r.t. the producer's pre-activation."""
    BT, C, OC = 21, 32, 12
    u = _bf16_vals((BT, C), 1.0, 21)
    w = _bf16_vals((OC, C), 0.3, 22)
    b = _bf16_vals((OC,), 0.3, 23)
    dout = _bf16_vals((BT, OC), 1.0, 24)
    (gu, gw, gb), _, xin = _autograd(None, w, b, dout, ACT_NONE, inp_pre=u)
    r = oracle.linear_backward(dout, xin.astype(np.float32), w, inp_pre=u, act=ACT_NONE)
    assert np.max(np.abs(r["dinp"] - gu)) < 1e-11
    # composed form: plain dinp, then the elementwise product
    r2 = oracle.linear_backward(dout, xin.astype(np.float32), w, act=ACT_NONE, want=("dinp",))
    assert np.max(np.abs(r2["dinp"] * oracle.gelu_grad(u.astype(np.float64)) - r["dinp"])) < 1e-13


@pytest.mark.parametrize("act", [ACT_NONE, ACT_GELU, ACT_SWIGLU])
def test_backward_by_finite_differences(act):
    """Brute force on a tiny layer: perturb every input, weight and bias entry."""
    BT, C, OC = 3, 4, 6
    rng = np.random.default_rng(5)
    inp = rng.standard_normal((BT, C)).astype(np.float32)
    w = rng.standard_normal((OC, C)).astype(np.float32)
    b = rng.standard_normal((OC,)).astype(np.float32)
    ocols = OC // 2 if act == ACT_SWIGLU else OC
    G = rng.standard_normal((BT, ocols)).astype(np.float32)

    def loss(i, ww, bb):
        out, _ = oracle.linear_forward(i, ww, bb, act, "f64")
        return float((out * G).sum())

    _, pre = oracle.linear_forward(inp, w, b, act, "f64")
    # pre is handed over in fp32 here, so compare at a tolerance above fp32 rounding of pre
    r = oracle.linear_backward(G, inp, w, pre=pre.astype(np.float32), act=act, dtype="f64")
    h = 2.0 ** -8  # exactly representable steps keep the perturbed fp32 inputs exact
    for name, arr, grad in (("dinp", inp, r["dinp"]), ("dweight", w, r["dweight"]),
                            ("dbias", b, r["dbias"])):
        fd = np.zeros(arr.shape)
        for idx in np.ndindex(arr.shape):
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h
            am[idx] -= h
            args_p = {"dinp": (ap, w, b), "dweight": (inp, ap, b), "dbias": (inp, w, ap)}[name]
            args_m = {"dinp": (am, w, b), "dweight": (inp, am, b), "dbias": (inp, w, am)}[name]
            fd[idx] = (loss(*args_p) - loss(*args_m)) / (2 * h)
        tol = 1e-9 if act == ACT_NONE else 5e-4  # central difference error ~ h^2 f'''
        assert np.max(np.abs(fd - grad)) < tol * max(1.0, np.max(np.abs(grad))), name


def test_backward_adjoint_identities():
    """<dz, x' W^T> = <dz W, x'> and <dW, W'> = <dz, x W'^T>: catches a transposed operand."""
    BT, C, OC = 31, 20, 14
    inp = _bf16_vals((BT, C), 1.0, 31)
    w = _bf16_vals((OC, C), 0.3, 32)
    dz = _bf16_vals((BT, OC), 1.0, 33)
    xp = _bf16_vals((BT, C), 1.0, 34)
    wp = _bf16_vals((OC, C), 1.0, 35)
    r = oracle.linear_backward(dz, inp, w)
    f1, _ = oracle.linear_forward(xp, w)
    assert abs((dz * f1).sum() - (r["dinp"] * xp).sum()) < 1e-10 * abs((dz * f1).sum())
    f2, _ = oracle.linear_forward(inp, wp)
    assert abs((dz * f2).sum() - (r["dweight"] * wp).sum()) < 1e-10 * abs((dz * f2).sum())


def test_dinp_is_dout_times_weight_integer_exact():
    rng = np.random.default_rng(9)
    BT, C, OC = 13, 10, 17
    dz = rng.integers(-6, 7, size=(BT, OC)).astype(np.float32)
    w = rng.integers(-6, 7, size=(OC, C)).astype(np.float32)
    inp = rng.integers(-6, 7, size=(BT, C)).astype(np.float32)
    for dt in ("f32", "f64"):
        r = oracle.linear_backward(dz, inp, w, dtype=dt)
        assert np.array_equal(r["dinp"].astype(np.int64), dz.astype(np.int64) @ w.astype(np.int64))
        assert np.array_equal(r["dweight"].astype(np.int64),
                              dz.astype(np.int64).T @ inp.astype(np.int64))
        assert np.array_equal(r["dbias"].astype(np.int64), dz.astype(np.int64).sum(0))


def test_dbias_invariants():
    BT, C, OC = 45, 8, 22
    dz = _bf16_vals((BT, OC), 1e-3, 41)
    w = _bf16_vals((OC, C), 0.02, 42)
    ones = np.ones((BT, C), dtype=np.float32)
    r = oracle.linear_backward(dz, ones, w)
    # dbias is the column sum of dz and equals any column of dweight taken against all-ones inp
    assert np.max(np.abs(r["dbias"] - dz.astype(np.float64).sum(0))) < 1e-15
    assert np.array_equal(r["dweight"][:, 0], r["dbias"])
    assert np.max(np.abs(oracle.reduce_dbias(dz) - r["dbias"])) < 1e-15
    # and equals 1^T dz through the forward product with inp = ones
    out, _ = oracle.linear_forward(np.ones((1, BT), dtype=np.float32), dz.T.copy())
    assert np.max(np.abs(out[0] - r["dbias"])) < 1e-15


@pytest.mark.parametrize("dt,tol", [("f32", 1e-6), ("f64", 1e-13)])
def test_accumulation_is_linear_over_micro_steps(dt, tol):
    """Four accumulate calls on four micro-batches equal one call on their concatenation."""
    C, OC, BT = 16, 12, 25
    w = _bf16_vals((OC, C), 0.02, 50)
    inps = [_bf16_vals((BT, C), 1.0, 51 + i) for i in range(4)]
    dzs = [_bf16_vals((BT, OC), 1e-3, 61 + i) for i in range(4)]
    rt = np.float32 if dt == "f32" else np.float64
    dW = np.full((OC, C), 7.0, dtype=rt)  # accumulate=0 must overwrite whatever is there
    db = np.full((OC,), -3.0, dtype=rt)
    for i in range(4):
        oracle.linear_backward(dzs[i], inps[i], w, dweight=dW, dbias=db, accumulate=(i > 0),
                               dtype=dt, want=("dweight", "dbias"))
    one = oracle.linear_backward(np.concatenate(dzs), np.concatenate(inps), w, dtype=dt)
    assert relf(dW, one["dweight"]) < tol
    assert relf(db, one["dbias"]) < tol


def test_fp32_oracle_close_to_fp64_oracle():
    """The float instance's own rounding is orders below the parity gate (5e-3)."""
    BT, C, OC = 256, 768, 96
    inp = _bf16_vals((BT, C), 1.0, 71)
    w = _bf16_vals((OC, C), 0.02, 72)
    b = _bf16_vals((OC,), 0.02, 73)
    dout = _bf16_vals((BT, OC), 1e-3, 74)
    o32, p32 = oracle.linear_forward(inp, w, b, ACT_GELU, "f32")
    o64, p64 = oracle.linear_forward(inp, w, b, ACT_GELU, "f64")
    assert relf(o32, o64) < 1e-5 and relf(p32, p64) < 1e-5
    pre = p64.astype(np.float32)
    r32 = oracle.linear_backward(dout, inp, w, pre=pre, act=ACT_GELU, dtype="f32")
    r64 = oracle.linear_backward(dout, inp, w, pre=pre, act=ACT_GELU, dtype="f64")
    for k in ("dinp", "dweight", "dbias"):
        assert relf(r32[k], r64[k]) < 1e-5, k


def test_malformed_requests_are_rejected():
    inp = np.zeros((4, 8), dtype=np.float32)
    w = np.zeros((5, 8), dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.linear_forward(inp, w, None, ACT_SWIGLU)  # odd OC
    with pytest.raises(ValueError):
        oracle.linear_backward(np.zeros((4, 5), dtype=np.float32), inp, w, act=ACT_GELU)  # no pre


def test_threads_reported():
    assert oracle.num_threads() >= 1
    assert math.isfinite(oracle.num_threads())


# ---------------------------------------------------------------- fp32 -> bf16 cast

def test_cast_against_library_and_hand_cases():
    """The bit-level cast equals the library's conversion, and the tie / carry / special cases hold."""
    g = torch.Generator().manual_seed(5)
    x = torch.randn(200000, generator=g) * torch.exp(torch.randn(200000, generator=g) * 8)
    bits = x.view(torch.int32).clone()
    bits[:1000] = torch.randint(-2**31, 2**31 - 1, (1000,), generator=g, dtype=torch.int64).to(torch.int32)
    x = bits.view(torch.float32)
    got = oracle.cast_f32_bf16(x.numpy())
    want = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = np.isnan(x.numpy())
    assert np.array_equal(got[~nan], want[~nan])
    assert np.all((got[nan] & 0x7F80) == 0x7F80) and np.all((got[nan] & 0x007F) != 0)  # still NaN

    def f(bits32):
        return np.array([bits32], dtype=np.uint32).view(np.float32)

    cases = [
        (0x3F800000, 0x3F80),  # 1.0
        (0x3F808000, 0x3F80),  # 1 + 2^-8: a tie, kept value even -> stays
        (0x3F818000, 0x3F82),  # 1 + 3*2^-8: a tie, kept value odd -> up
        (0x3F808001, 0x3F81),  # just above the tie -> up
        (0x3F807FFF, 0x3F80),  # just below the tie -> down
        (0x7F7FFFFF, 0x7F80),  # largest fp32 rounds to +inf
        (0x7F800000, 0x7F80), (0xFF800000, 0xFF80),  # infinities
        (0x00000000, 0x0000), (0x80000000, 0x8000),  # signed zeros
        (0x00008000, 0x0000),  # subnormal tie to even (zero)
        (0x00018000, 0x0002),  # subnormal tie, odd -> up
        (0xBF808001, 0xBF81),  # negative, above the tie in magnitude
    ]
    for b32, b16 in cases:
        assert oracle.cast_f32_bf16(f(b32))[0] == b16, hex(b32)


# ---------------------------------------------------------------- cross-entropy over the real vocabulary

def test_cross_entropy_against_library_autograd():
    BT, Vp, V = 23, 48, 41
    g = torch.Generator().manual_seed(12)
    logits = (torch.randn(BT, Vp, generator=g) * 3).to(torch.bfloat16).float()
    targets = torch.randint(0, V, (BT,), generator=g)
    gscale = 1.0 / BT
    x = logits.double().requires_grad_(True)
    per_row = F.cross_entropy(x[:, :V], targets, reduction="none")
    (gx,) = torch.autograd.grad((per_row * gscale).sum(), x)
    loss, lse, dl = oracle.cross_entropy(logits.numpy(), targets.numpy(), V, gscale)
    assert np.max(np.abs(loss - per_row.detach().numpy())) < 1e-12
    assert np.max(np.abs(lse - torch.logsumexp(x[:, :V], 1).detach().numpy())) < 1e-12
    assert np.max(np.abs(dl - gx.numpy())) < 1e-15
    assert np.all(dl[:, V:] == 0.0)                      # padding columns: no gradient
    assert np.max(np.abs(dl.sum(1))) < 1e-15             # softmax - onehot sums to zero per row


def test_cross_entropy_closed_forms():
    BT, Vp, V = 5, 16, 11
    # equal logits: uniform distribution over the V real columns, whatever the padding holds
    logits = np.full((BT, Vp), 0.75, dtype=np.float32)
    logits[:, V:] = 100.0
    t = np.arange(BT) % V
    loss, lse, dl = oracle.cross_entropy(logits, t, V)
    assert np.allclose(loss, math.log(V), atol=1e-14) and np.allclose(lse, 0.75 + math.log(V), atol=1e-14)
    assert np.allclose(dl[0, 1:V], 1.0 / V, atol=1e-15) and abs(dl[0, 0] - (1.0 / V - 1.0)) < 1e-15
    # one dominant logit on the target: loss -> 0, gradient -> 0
    logits = np.zeros((1, Vp), dtype=np.float32)
    logits[0, 3] = 80.0
    loss, _, dl = oracle.cross_entropy(logits, [3], V)
    assert loss[0] < 1e-30 + 1e-12 and np.max(np.abs(dl)) < 1e-12
    # shift invariance of the loss, and rejection of an out-of-range target
    a = np.random.default_rng(0).standard_normal((4, Vp)).astype(np.float32)
    l1, _, _ = oracle.cross_entropy(a, [0, 1, 2, 3], V, want_grad=False)
    l2, _, _ = oracle.cross_entropy(a + np.float32(2.0), [0, 1, 2, 3], V, want_grad=False)
    assert np.max(np.abs(l1 - l2)) < 1e-6
    with pytest.raises(ValueError):
        oracle.cross_entropy(a, [0, 1, 2, V], V)


# ---------------------------------------------------------------- low-rank adapter beside a frozen layer

def test_lora_against_library_autograd():
    BT, C, OC, r = 19, 24, 14, 4
    scale = 32.0 / math.sqrt(16)  # rank-stabilised: alpha / sqrt(r) with the paper's alpha=32, r=16
    x = _bf16_vals((BT, C), 1.0, 91)
    W = _bf16_vals((OC, C), 0.3, 92)
    b = _bf16_vals((OC,), 0.3, 93)
    A = _bf16_vals((r, C), 0.3, 94)
    B = _bf16_vals((OC, r), 0.3, 95)
    dy = _bf16_vals((BT, OC), 1.0, 96)
    tx = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    tA = torch.tensor(A, dtype=torch.float64, requires_grad=True)
    tB = torch.tensor(B, dtype=torch.float64, requires_grad=True)
    tW = torch.tensor(W, dtype=torch.float64)
    y = F.linear(tx, tW, torch.tensor(b, dtype=torch.float64)) + scale * F.linear(F.linear(tx, tA), tB)
    gx, gA, gB = torch.autograd.grad((y * torch.tensor(dy, dtype=torch.float64)).sum(), [tx, tA, tB])
    out = oracle.lora_forward(x, W, b, A, B, scale)
    assert np.max(np.abs(out - y.detach().numpy())) < 1e-11
    dinp, dA, dB = oracle.lora_backward(dy, x, W, A, B, scale)
    assert np.max(np.abs(dinp - gx.numpy())) < 1e-11
    assert np.max(np.abs(dA - gA.numpy())) < 1e-11
    assert np.max(np.abs(dB - gB.numpy())) < 1e-11
    # merged-weight identity: the adapter is a rank-r update of W
    Wm = W.astype(np.float64) + scale * (B.astype(np.float64) @ A.astype(np.float64))
    assert np.max(np.abs(out - (x.astype(np.float64) @ Wm.T + b))) < 1e-11
    assert np.max(np.abs(dinp - dy.astype(np.float64) @ Wm)) < 1e-11
    # B = 0 (the usual initialisation): the layer equals the frozen one and only dB is non-zero
    Z = np.zeros_like(B)
    base, _ = oracle.linear_forward(x, W, b)
    assert np.array_equal(oracle.lora_forward(x, W, b, A, Z, scale), base)
    dinp0, dA0, dB0 = oracle.lora_backward(dy, x, W, A, Z, scale)
    assert np.all(dA0 == 0) and np.any(dB0 != 0)
    assert np.max(np.abs(dinp0 - oracle.linear_backward(dy, x, W, want=("dinp",))["dinp"])) < 1e-12
    # accumulation over two micro-steps is linear
    dA2, dB2 = dA.copy(), dB.copy()
    oracle.lora_backward(dy, x, W, A, B, scale, dA=dA2, dB=dB2, accumulate=True, want_dinp=False)
    assert np.allclose(dA2, 2 * dA, rtol=1e-14) and np.allclose(dB2, 2 * dB, rtol=1e-14)
