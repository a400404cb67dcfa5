"""ctypes binding of the nb_linear C ABI: argument marshalling only.

Functions named like the C entry points take torch CUDA tensors (or raw device
pointers as ints) and pass pointers and sizes straight through; every step of
the computation runs in the CUDA library. There is no CPU path: if the library
has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .build import LIB_PATH

NB_OK, NB_ERR_INVALID_ARG, NB_ERR_UNSUPPORTED, NB_ERR_CUDA, NB_ERR_TIMEOUT = 0, 1, 2, 3, 4
ACT_NONE, ACT_GELU, ACT_SWIGLU = 0, 1, 2
DTYPE_F32, DTYPE_BF16 = 0, 1

EXPORTS = (
    "nb_version", "nb_last_error", "nb_set_stream", "nb_get_stream", "nb_linear_out_elems",
    "nb_linear_forward", "nb_linear_forward_ex", "nb_linear_backward", "nb_linear_backward_ex",
    "nb_reduce_dbias", "nb_workspace_reserve", "nb_release", "nb_check_status",
    "nb_debug_wait_timeout", "nb_kernel_launches", "nb_gelu_dbias_noalloc",
    "nb_debug_split_plan", "nb_cast_f32_to_bf16", "nb_lm_head_ce_forward", "nb_ce_backward",
    "nb_lora_linear_forward", "nb_lora_linear_backward", "nb_debug_layer_bwd_plan", "nb_debug_gemm_timeout",
    "nb_lora_down_stacked", "nb_lora_linear_forward_stacked", "nb_lora_linear_backward_stacked",
    "nb_lora_da_stacked",
)

_lib = None
_vp, _i64, _int = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int


class NbError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"nb_linear error {code}: {msg}")
        self.code = code


def lib() -> ctypes.CDLL:
    """The loaded CUDA library. Raises if it was never built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2609_28568_b200.build` "
                "(the CUDA library is the only implementation)")
        L = ctypes.CDLL(LIB_PATH)
        L.nb_version.restype = _int
        L.nb_last_error.restype = ctypes.c_char_p
        L.nb_set_stream.argtypes = [_vp]
        L.nb_get_stream.restype = _vp
        L.nb_linear_out_elems.argtypes = [_i64, _i64, _int]
        L.nb_linear_out_elems.restype = _i64
        L.nb_linear_forward.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int]
        L.nb_linear_forward_ex.argtypes = [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp]
        L.nb_linear_backward.argtypes = [_vp] * 7 + [_i64, _i64, _i64, _int]
        L.nb_linear_backward_ex.argtypes = [_vp] * 8 + [_i64, _i64, _i64, _int, _int, _int, _vp]
        L.nb_reduce_dbias.argtypes = [_vp, _vp, _i64, _i64, _int]
        L.nb_workspace_reserve.argtypes = [_i64]
        L.nb_debug_wait_timeout.argtypes = [_i64]
        L.nb_kernel_launches.restype = _i64
        L.nb_gelu_dbias_noalloc.argtypes = [_vp, _vp, _vp, _i64, _i64, _int, _vp]
        L.nb_cast_f32_to_bf16.argtypes = [_vp, _vp, _i64, _vp]
        L.nb_lora_linear_forward.argtypes = [_vp] * 7 + [ctypes.c_float] + [_i64] * 4 + [_vp]
        L.nb_lora_linear_backward.argtypes = [_vp] * 10 + [ctypes.c_float] + [_i64] * 4 + [_int, _vp]
        L.nb_lora_down_stacked.argtypes = [_vp, _vp, _vp, ctypes.c_float, _i64, _i64, _i64, _vp]
        L.nb_lora_linear_forward_stacked.argtypes = [_vp] * 6 + [_i64] * 6 + [_vp]
        L.nb_lora_linear_backward_stacked.argtypes = [_vp] * 8 + [ctypes.c_float] + [_i64] * 6 + [_int, _vp]
        L.nb_lora_da_stacked.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _int, _vp]
        L.nb_lm_head_ce_forward.argtypes = [_vp] * 6 + [_i64] * 4 + [_vp]
        L.nb_ce_backward.argtypes = [_vp] * 4 + [ctypes.c_float] + [_i64] * 3 + [_vp]
        L.nb_debug_split_plan.argtypes = [_i64, _i64, _i64, _int, _int, ctypes.POINTER(_int)]
        L.nb_debug_gemm_timeout.argtypes = [_vp, _vp, _vp, _i64]
        L.nb_debug_layer_bwd_plan.argtypes = [_i64, _i64, _i64, _int, _int, ctypes.POINTER(_int), _i64]
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _check(rc: int) -> None:
    if rc != NB_OK:
        raise NbError(rc, lib().nb_last_error().decode())


def _stream():
    return torch.cuda.current_stream().cuda_stream


def nb_version() -> int:
    return lib().nb_version()


def nb_last_error() -> str:
    return lib().nb_last_error().decode()


def nb_linear_out_elems(BT: int, OC: int, act: int) -> int:
    return lib().nb_linear_out_elems(BT, OC, act)


def nb_set_stream(stream) -> None:
    _check(lib().nb_set_stream(stream))


def nb_linear_forward(out, inp, weight, bias, BT, C, OC, act) -> None:
    """Short form: `out` holds the activated plane followed by the pre-activation plane."""
    lib().nb_set_stream(_stream())
    _check(lib().nb_linear_forward(_ptr(out), _ptr(inp), _ptr(weight), _ptr(bias), BT, C, OC, act))


def nb_linear_forward_ex(out, pre_act, inp, weight, bias, BT, C, OC, act, stream=None) -> None:
    _check(lib().nb_linear_forward_ex(_ptr(out), _ptr(pre_act), _ptr(inp), _ptr(weight), _ptr(bias),
                                      BT, C, OC, act, _stream() if stream is None else stream))


def nb_linear_backward(dinp, dweight, dbias, dout, inp, weight, pre_act, BT, C, OC, accumulate) -> None:
    lib().nb_set_stream(_stream())
    _check(lib().nb_linear_backward(_ptr(dinp), _ptr(dweight), _ptr(dbias), _ptr(dout), _ptr(inp),
                                    _ptr(weight), _ptr(pre_act), BT, C, OC, int(accumulate)))


def nb_linear_backward_ex(dinp, dweight, dbias, dout, inp, weight, pre_act, inp_pre_act, BT, C, OC,
                          act, accumulate, dweight_dtype=DTYPE_F32, stream=None) -> None:
    _check(lib().nb_linear_backward_ex(_ptr(dinp), _ptr(dweight), _ptr(dbias), _ptr(dout), _ptr(inp),
                                       _ptr(weight), _ptr(pre_act), _ptr(inp_pre_act), BT, C, OC, act,
                                       int(accumulate), dweight_dtype,
                                       _stream() if stream is None else stream))


def nb_reduce_dbias(dbias, dout, BT, OC, accumulate) -> None:
    lib().nb_set_stream(_stream())
    _check(lib().nb_reduce_dbias(_ptr(dbias), _ptr(dout), BT, OC, int(accumulate)))


def nb_workspace_reserve(nbytes: int) -> None:
    _check(lib().nb_workspace_reserve(nbytes))


def nb_release() -> None:
    _check(lib().nb_release())


def nb_check_status() -> None:
    """Synchronise and raise NbError(NB_ERR_TIMEOUT / NB_ERR_CUDA) if a kernel reported a failure."""
    _check(lib().nb_check_status())


NOALLOC_MAX_ELEMS = 4194304


def nb_gelu_dbias_noalloc(dbias, dout, pre_act, BT, OC, accumulate, stream=None) -> None:
    """dbias (+)= column sums of dout * gelu'(pre_act), using only the scratch array built into
    the library: for callers that may not allocate device memory. BT*OC <= NOALLOC_MAX_ELEMS."""
    _check(lib().nb_gelu_dbias_noalloc(_ptr(dbias), _ptr(dout), _ptr(pre_act), BT, OC,
                                       int(accumulate), _stream() if stream is None else stream))


def nb_lora_linear_forward(out, t, inp, weight, bias, lora_a, lora_b, scale, BT, C, OC, r, stream=None) -> None:
    """out = inp @ W.T (+ bias) + t @ B.T with t = bf16(scale * inp @ A.T), the adapter term fused in."""
    _check(lib().nb_lora_linear_forward(_ptr(out), _ptr(t), _ptr(inp), _ptr(weight), _ptr(bias),
                                        _ptr(lora_a), _ptr(lora_b), scale, BT, C, OC, r,
                                        _stream() if stream is None else stream))


def nb_lora_linear_backward(dinp, dlora_a, dlora_b, u, dout, inp, weight, lora_a, lora_b, t, scale, BT, C,
                            OC, r, accumulate, stream=None) -> None:
    """Gradients of the adapter layer with the base weight frozen (dinp, dA, dB)."""
    _check(lib().nb_lora_linear_backward(_ptr(dinp), _ptr(dlora_a), _ptr(dlora_b), _ptr(u), _ptr(dout),
                                         _ptr(inp), _ptr(weight), _ptr(lora_a), _ptr(lora_b), _ptr(t),
                                         scale, BT, C, OC, r, int(accumulate),
                                         _stream() if stream is None else stream))


def nb_lora_down_stacked(t_stack, inp, a_stack, scale, BT, C, R, stream=None) -> None:
    """t_stack = bf16(scale * inp @ a_stack.T): the down-projections of all adapters of a group at once."""
    _check(lib().nb_lora_down_stacked(_ptr(t_stack), _ptr(inp), _ptr(a_stack), scale, BT, C, R,
                                      _stream() if stream is None else stream))


def nb_lora_linear_forward_stacked(out, inp, weight, bias, t_stack, lora_b, BT, C, OC, r, R, off,
                                   stream=None) -> None:
    """out = inp @ W.T (+ bias) + t_stack[:, off:off+r] @ B.T, the adapter term fused in."""
    _check(lib().nb_lora_linear_forward_stacked(_ptr(out), _ptr(inp), _ptr(weight), _ptr(bias), _ptr(t_stack),
                                                _ptr(lora_b), BT, C, OC, r, R, off,
                                                _stream() if stream is None else stream))


def nb_lora_linear_backward_stacked(dinp, dlora_b, u_stack, dout, weight, lora_a, lora_b, t_stack, scale, BT, C,
                                    OC, r, R, off, accumulate, stream=None) -> None:
    """u slice, dinp and dB of one adapted projection of a stacked group (dA comes from nb_lora_da_stacked)."""
    _check(lib().nb_lora_linear_backward_stacked(_ptr(dinp), _ptr(dlora_b), _ptr(u_stack), _ptr(dout),
                                                 _ptr(weight), _ptr(lora_a), _ptr(lora_b), _ptr(t_stack), scale,
                                                 BT, C, OC, r, R, off, int(accumulate),
                                                 _stream() if stream is None else stream))


def nb_lora_da_stacked(da_stack, u_stack, inp, BT, C, R, accumulate, stream=None) -> None:
    """da_stack (+)= u_stack.T @ inp: the A gradients of all adapters of a group at once."""
    _check(lib().nb_lora_da_stacked(_ptr(da_stack), _ptr(u_stack), _ptr(inp), BT, C, R, int(accumulate),
                                    _stream() if stream is None else stream))


def nb_lm_head_ce_forward(logits, loss, lse, inp, weight, targets, BT, C, Vp, V, stream=None) -> None:
    """Head GEMM with the softmax statistics of the first V columns fused in: logits, loss, lse."""
    _check(lib().nb_lm_head_ce_forward(_ptr(logits), _ptr(loss), _ptr(lse), _ptr(inp), _ptr(weight),
                                       _ptr(targets), BT, C, Vp, V,
                                       _stream() if stream is None else stream))


def nb_ce_backward(dlogits, logits, lse, targets, gscale, BT, Vp, V, stream=None) -> None:
    """dlogits = gscale * (softmax - onehot) on the first V columns, 0 on the padding."""
    _check(lib().nb_ce_backward(_ptr(dlogits), _ptr(logits), _ptr(lse), _ptr(targets), gscale, BT, Vp, V,
                                _stream() if stream is None else stream))


def nb_cast_f32_to_bf16(dst, src, n, stream=None) -> None:
    """Master-weight cast: dst (bf16) = src (fp32), round to nearest even."""
    _check(lib().nb_cast_f32_to_bf16(_ptr(dst), _ptr(src), n, _stream() if stream is None else stream))


def nb_debug_split_plan(M: int, N: int, K: int, slots: int, tile_m: int):
    """(row tiles, column tiles, split-K factor, k-blocks per split, k-blocks) of a wgrad."""
    out = (_int * 5)()
    _check(lib().nb_debug_split_plan(M, N, K, slots, tile_m, out))
    return tuple(out)


def nb_debug_layer_bwd_plan(BT: int, C: int, OC: int, pairs: int, gelu_grad: bool):
    """(header of eight ints, list of (pair, is_dweight, row tile, column tile, kb0, kb1)) of the
    one-launch layer backward; raises NbError for shapes its schedule does not cover."""
    cap = 8 + 6 * (4 * pairs + 64 + 2 * (-(-BT // 256)) * (-(-C // 256))
                   + 2 * (-(-OC // 256)) * (-(-C // 256)) * max(1, BT // 1024))
    out = (_int * cap)()
    n = lib().nb_debug_layer_bwd_plan(BT, C, OC, pairs, int(bool(gelu_grad)), out, cap)
    if n < 0:
        raise NbError(-n, lib().nb_last_error().decode())
    recs = [tuple(out[8 + 6 * i: 14 + 6 * i]) for i in range(n)]
    return tuple(out[:8]), recs


def nb_kernel_launches() -> int:
    return int(lib().nb_kernel_launches())


def nb_debug_gemm_timeout(out, inp, weight, limit_us: int) -> None:
    """One-tile forward GEMM whose producer stops half way: exercises the kernel's time-out exit."""
    lib().nb_set_stream(_stream())
    _check(lib().nb_debug_gemm_timeout(_ptr(out), _ptr(inp), _ptr(weight), limit_us))


def nb_debug_wait_timeout(limit_us: int) -> None:
    lib().nb_set_stream(_stream())
    _check(lib().nb_debug_wait_timeout(limit_us))


# ------------------------------------------------------------------ conveniences (allocation only)

def linear_forward(inp, weight, bias=None, act=ACT_NONE):
    """Allocate the outputs and call nb_linear_forward_ex. Returns (out, pre_act or None)."""
    BT, C = inp.shape
    OC = weight.shape[0]
    ocols = OC // 2 if act == ACT_SWIGLU else OC
    out = torch.empty((BT, ocols), dtype=torch.bfloat16, device=inp.device)
    pre = torch.empty((BT, OC), dtype=torch.bfloat16, device=inp.device) if act != ACT_NONE else None
    nb_linear_forward_ex(out, pre, inp, weight, bias, BT, C, OC, act)
    return out, pre


def linear_backward(dout, inp, weight, pre_act=None, inp_pre_act=None, act=ACT_NONE, dweight=None,
                    dbias=None, accumulate=False, need_dinp=True, need_dweight=True,
                    need_dbias=True):
    """Allocate missing outputs and call nb_linear_backward_ex. Returns (dinp, dweight, dbias)."""
    BT = dout.shape[0]
    OC, C = weight.shape
    dev = dout.device
    dinp = torch.empty((BT, C), dtype=torch.bfloat16, device=dev) if need_dinp else None
    if need_dweight and dweight is None:
        dweight = torch.empty((OC, C), dtype=torch.float32, device=dev)
    if need_dbias and dbias is None:
        dbias = torch.empty((OC,), dtype=torch.float32, device=dev)
    nb_linear_backward_ex(dinp, dweight if need_dweight else None, dbias if need_dbias else None,
                          dout, inp, weight, pre_act, inp_pre_act, BT, C, OC, act, accumulate)
    return dinp, dweight, dbias
