"""CPU oracle for the dense linear layers: a ctypes view of ``nb_oracle.c``.

TEST INFRASTRUCTURE ONLY. The oracle is the plain definition of the forward and
backward products (triple loops, tanh-GELU, SiLU, column sums) in fp32 or fp64.
It shares no code with the CUDA library and is never on the product path: only
tests, the smoke check and the benchmark's CPU-baseline leg import this package.

Inputs are numpy float32 arrays that hold bf16 values widened exactly; outputs
are float32 (``dtype="f32"``) or float64 (``dtype="f64"``) and are not rounded.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

ACT_NONE, ACT_GELU, ACT_SWIGLU = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = [os.path.join(_HERE, "nb_oracle.c"), os.path.join(_HERE, "nb_oracle_impl.inc")]
_SO = os.path.join(_HERE, "libnb_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, -O3) if the library is missing or stale."""
    stale = force or not os.path.exists(_SO) or any(
        os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC)
    if stale:
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-Wall", "-Wextra", "-o", _SO, _SRC[0], "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.nbo_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops will use."""
    return int(_load().nbo_num_threads())


def _real(dtype: str):
    if dtype == "f32":
        return np.float32, "_f32"
    if dtype == "f64":
        return np.float64, "_f64"
    raise ValueError("dtype must be 'f32' or 'f64'")


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32c(a):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _scalar_fn(name: str, x, dtype: str):
    rt, suf = _real(dtype)
    x = np.ascontiguousarray(x, dtype=rt)
    y = np.empty_like(x)
    fn = getattr(_load(), name + suf)
    fn.restype = None
    fn(_p(y), _p(x), ctypes.c_int64(x.size))
    return y


def gelu(x, dtype: str = "f64"):
    """tanh-GELU, elementwise."""
    return _scalar_fn("nbo_gelu", x, dtype)


def gelu_grad(x, dtype: str = "f64"):
    """Derivative of tanh-GELU, elementwise."""
    return _scalar_fn("nbo_gelu_grad", x, dtype)


def silu(x, dtype: str = "f64"):
    return _scalar_fn("nbo_silu", x, dtype)


def silu_grad(x, dtype: str = "f64"):
    return _scalar_fn("nbo_silu_grad", x, dtype)


def linear_forward(inp, weight, bias=None, act: int = ACT_NONE, dtype: str = "f64"):
    """Return ``(out, pre)``: ``pre = inp @ weight.T + bias``, ``out = act(pre)``.

    inp [BT, C], weight [OC, C], bias [OC] or None. For SwiGLU the weight rows are
    [gate; up] and ``out`` is [BT, OC/2].
    """
    rt, suf = _real(dtype)
    inp, weight, bias = _f32c(inp), _f32c(weight), _f32c(bias)
    BT, C = inp.shape
    OC, C2 = weight.shape
    assert C == C2 and (bias is None or bias.shape == (OC,))
    out_cols = OC // 2 if act == ACT_SWIGLU else OC
    out = np.empty((BT, out_cols), dtype=rt)
    pre = np.empty((BT, OC), dtype=rt)
    fn = getattr(_load(), "nbo_linear_forward" + suf)
    fn.restype = ctypes.c_int
    rc = fn(_p(out), _p(pre), _p(inp), _p(weight), _p(bias), ctypes.c_int64(BT),
            ctypes.c_int64(C), ctypes.c_int64(OC), ctypes.c_int(act))
    if rc != 0:
        raise ValueError(f"oracle forward rejected the request (rc={rc})")
    return out, pre


def linear_backward(dout, inp, weight, pre=None, inp_pre=None, act: int = ACT_NONE,
                    dweight=None, dbias=None, accumulate: bool = False, dtype: str = "f64",
                    want=("dinp", "dweight", "dbias")):
    """Return a dict with the requested of ``dinp``, ``dweight``, ``dbias`` and ``dz``.

    ``dz = dout * act'(pre)``; ``dinp = dz @ weight`` (times ``gelu'(inp_pre)`` when
    ``inp_pre`` is given); ``dweight (+)= dz.T @ inp``; ``dbias (+)= dz.sum(0)``.
    With ``accumulate`` the passed ``dweight`` / ``dbias`` arrays are added to in place.
    """
    rt, suf = _real(dtype)
    dout, inp, weight = _f32c(dout), _f32c(inp), _f32c(weight)
    pre, inp_pre = _f32c(pre), _f32c(inp_pre)
    BT = dout.shape[0]
    OC, C = weight.shape
    res = {}
    dinp = np.empty((BT, C), dtype=rt) if "dinp" in want else None
    if "dweight" in want:
        if dweight is None:
            assert not accumulate
            dweight = np.empty((OC, C), dtype=rt)
        assert dweight.dtype == rt and dweight.flags.c_contiguous and dweight.shape == (OC, C)
    else:
        dweight = None
    if "dbias" in want:
        if dbias is None:
            assert not accumulate
            dbias = np.empty((OC,), dtype=rt)
        assert dbias.dtype == rt and dbias.flags.c_contiguous and dbias.shape == (OC,)
    else:
        dbias = None
    dz = np.empty((BT, OC), dtype=rt) if "dz" in want else None
    fn = getattr(_load(), "nbo_linear_backward" + suf)
    fn.restype = ctypes.c_int
    rc = fn(_p(dinp), _p(dweight), _p(dbias), _p(dz), _p(dout), _p(inp), _p(weight), _p(pre),
            _p(inp_pre), ctypes.c_int64(BT), ctypes.c_int64(C), ctypes.c_int64(OC),
            ctypes.c_int(act), ctypes.c_int(1 if accumulate else 0))
    if rc != 0:
        raise ValueError(f"oracle backward rejected the request (rc={rc})")
    for k, v in (("dinp", dinp), ("dweight", dweight), ("dbias", dbias), ("dz", dz)):
        if v is not None:
            res[k] = v
    return res


def reduce_dbias(dout, dbias=None, accumulate: bool = False):
    """Column sum ``dbias[o] (+)= sum_m dout[m, o]`` in fp64."""
    dout = _f32c(dout)
    BT, OC = dout.shape
    if dbias is None:
        assert not accumulate
        dbias = np.empty((OC,), dtype=np.float64)
    fn = _load().nbo_reduce_dbias_f64
    fn.restype = ctypes.c_int
    rc = fn(_p(dbias), _p(dout), ctypes.c_int64(BT), ctypes.c_int64(OC),
            ctypes.c_int(1 if accumulate else 0))
    if rc != 0:
        raise ValueError("oracle reduce_dbias rejected the request")
    return dbias


def cast_f32_bf16(src):
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    src = np.ascontiguousarray(src, dtype=np.float32)
    dst = np.empty(src.shape, dtype=np.uint16)
    fn = _load().nbo_cast_f32_bf16
    fn.restype = None
    fn(_p(dst), _p(src), ctypes.c_int64(src.size))
    return dst


def cross_entropy(logits, targets, V: int, gscale: float = 1.0, want_grad: bool = True):
    """Per-row ``(loss, lse, dlogits)`` of the cross-entropy over the first V columns of ``logits``.

    ``dlogits = gscale * (softmax - onehot)`` on the first V columns and 0 on the padding ones.
    """
    logits = _f32c(logits)
    BT, Vp = logits.shape
    targets = np.ascontiguousarray(targets, dtype=np.int32)
    loss = np.empty((BT,), dtype=np.float64)
    lse = np.empty((BT,), dtype=np.float64)
    dl = np.empty((BT, Vp), dtype=np.float64) if want_grad else None
    fn = _load().nbo_cross_entropy_f64
    fn.restype = ctypes.c_int
    rc = fn(_p(loss), _p(lse), _p(dl), _p(logits), _p(targets), ctypes.c_int64(BT), ctypes.c_int64(Vp),
            ctypes.c_int64(V), ctypes.c_double(gscale))
    if rc != 0:
        raise ValueError("oracle cross_entropy rejected the request")
    return loss, lse, dl


def lora_forward(inp, W, bias, A, B, scale: float):
    """``inp @ W.T (+ bias) + scale * (inp @ A.T) @ B.T`` in fp64; A [r, C], B [OC, r]."""
    inp, W, bias, A, B = _f32c(inp), _f32c(W), _f32c(bias), _f32c(A), _f32c(B)
    BT, C = inp.shape
    OC, r = B.shape
    assert W.shape == (OC, C) and A.shape == (r, C)
    out = np.empty((BT, OC), dtype=np.float64)
    fn = _load().nbo_lora_forward_f64
    fn.restype = ctypes.c_int
    rc = fn(_p(out), _p(inp), _p(W), _p(bias), _p(A), _p(B), ctypes.c_double(scale), ctypes.c_int64(BT),
            ctypes.c_int64(C), ctypes.c_int64(OC), ctypes.c_int64(r))
    if rc != 0:
        raise ValueError("oracle lora_forward rejected the request")
    return out


def lora_backward(dout, inp, W, A, B, scale: float, dA=None, dB=None, accumulate: bool = False,
                  want_dinp: bool = True):
    """Gradients of the adapter layer with W frozen: ``(dinp, dA, dB)`` in fp64."""
    dout, inp, W, A, B = _f32c(dout), _f32c(inp), _f32c(W), _f32c(A), _f32c(B)
    BT, C = inp.shape
    OC, r = B.shape
    dinp = np.empty((BT, C), dtype=np.float64) if want_dinp else None
    if dA is None:
        assert not accumulate
        dA = np.empty((r, C), dtype=np.float64)
    if dB is None:
        assert not accumulate
        dB = np.empty((OC, r), dtype=np.float64)
    fn = _load().nbo_lora_backward_f64
    fn.restype = ctypes.c_int
    rc = fn(_p(dinp), _p(dA), _p(dB), _p(dout), _p(inp), _p(W), _p(A), _p(B), ctypes.c_double(scale),
            ctypes.c_int64(BT), ctypes.c_int64(C), ctypes.c_int64(OC), ctypes.c_int64(r),
            ctypes.c_int(1 if accumulate else 0))
    if rc != 0:
        raise ValueError("oracle lora_backward rejected the request")
    return dinp, dA, dB
