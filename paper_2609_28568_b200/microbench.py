"""Time one kind of library call on one shape (also the small case used for ncu captures).

    python -m paper_2609_28568_b200.microbench KIND BT C OC [REPS] [energy]

KIND: fwd, fwd_nobias, fwd_gelu, fwd_swiglu, dgrad, dgrad_fused (dgrad with the producer's GELU
backward in the epilogue), wgrad (accumulating), wgrad_bias (wgrad with the fused bias gradient),
dbias (stand-alone column reduction), bwd (dinp + dweight + dbias in one call), bwd_nobias (dinp +
dweight), bwd_fused (bwd with the producer's GELU backward in the dinp epilogue), cast (fp32 -> bf16
master-weight cast of OC*C elements; reports GB/s), head_ce (head forward with the fused softmax
statistics, vocabulary OC with the last 47 columns as padding), ce_bwd (dlogits from logits, GB/s),
lora_fwd / lora_bwd (rank-16 adapter beside a frozen weight; TFLOP/s counts base + adapter flops).
Prints microseconds per call and TFLOP/s from CUDA events around REPS back-to-back calls.

With the word `energy` after REPS (GEMM kinds only) the call is instead replayed from a CUDA graph for
about 2.5 seconds over rotating sets of buffers (inputs come from DRAM, as inside a training step, and the
part settles at its power cap), and the GPU's energy counter (NVML, read-only) is read around the loop:
microseconds, TFLOP/s, millijoules per call, picojoules per flop and average watts.
"""
from __future__ import annotations

import sys

import torch

from . import binding as nb
from . import synth


def sustained_energy(kind: str, BT: int, C: int, OC: int) -> int:
    """Energy per call under sustained load: see the module docstring."""
    import time

    import pynvml
    pynvml.nvmlInit()
    h = pynvml.nvmlDeviceGetHandleByIndex(torch.cuda.current_device())
    dev, bf, f32 = "cuda", torch.bfloat16, torch.float32
    nbuf = 2 if BT * OC > (1 << 28) else 6
    inp = [synth.normal(1 + i, (BT, C), 1.0, dev) for i in range(nbuf)]
    w, b = synth.normal(2, (OC, C), 0.02, dev), synth.normal(3, (OC,), 0.02, dev)
    dout = [synth.normal(40 + i, (BT, OC), 1e-3, dev) for i in range(nbuf)]
    ipre = [synth.normal(50 + i, (BT, C), 1.0, dev) for i in range(nbuf)]
    out = [torch.empty((BT, OC), dtype=bf, device=dev) for _ in range(nbuf)]
    pre = [torch.empty((BT, OC), dtype=bf, device=dev) for _ in range(nbuf)]
    dinp = [torch.empty((BT, C), dtype=bf, device=dev) for _ in range(nbuf)]
    dw, db = torch.zeros((OC, C), dtype=f32, device=dev), torch.zeros((OC,), dtype=f32, device=dev)
    calls = {
        "fwd": lambda i: nb.nb_linear_forward_ex(out[i], None, inp[i], w, b, BT, C, OC, nb.ACT_NONE),
        "fwd_nobias": lambda i: nb.nb_linear_forward_ex(out[i], None, inp[i], w, None, BT, C, OC, nb.ACT_NONE),
        "fwd_gelu": lambda i: nb.nb_linear_forward_ex(out[i], pre[i], inp[i], w, b, BT, C, OC, nb.ACT_GELU),
        "dgrad": lambda i: nb.nb_linear_backward_ex(dinp[i], None, None, dout[i], None, w, None, None, BT, C, OC, 0, 0),
        "dgrad_fused": lambda i: nb.nb_linear_backward_ex(dinp[i], None, None, dout[i], None, w, None, ipre[i], BT,
                                                          C, OC, 0, 0),
        "wgrad": lambda i: nb.nb_linear_backward_ex(None, dw, None, dout[i], inp[i], None, None, None, BT, C, OC, 0, 1),
        "wgrad_bias": lambda i: nb.nb_linear_backward_ex(None, dw, db, dout[i], inp[i], None, None, None, BT, C, OC,
                                                         0, 1),
        "bwd": lambda i: nb.nb_linear_backward_ex(dinp[i], dw, db, dout[i], inp[i], w, None, None, BT, C, OC, 0, 1),
        "bwd_nobias": lambda i: nb.nb_linear_backward_ex(dinp[i], dw, None, dout[i], inp[i], w, None, None, BT, C,
                                                         OC, 0, 1),
        "bwd_fused": lambda i: nb.nb_linear_backward_ex(dinp[i], dw, db, dout[i], inp[i], w, None, ipre[i], BT, C,
                                                        OC, 0, 1),
    }
    if kind not in calls:
        print(__doc__)
        return 2
    call = calls[kind]
    flops = 2 * BT * C * OC * (2 if kind.startswith("bwd") else 1)
    for i in range(nbuf):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(20):
        call(i % nbuf)
    e1.record()
    torch.cuda.synchronize()
    per_graph = nbuf * 4
    reps = max(2, int(2500.0 / (e0.elapsed_time(e1) / 20)) // per_graph)
    g, cap = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        with torch.cuda.graph(g, stream=cap):
            for i in range(per_graph):
                call(i % nbuf)
    torch.cuda.current_stream().wait_stream(cap)
    g.replay()
    torch.cuda.synchronize()
    j0, t0 = pynvml.nvmlDeviceGetTotalEnergyConsumption(h), time.time()
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    j1, t1 = pynvml.nvmlDeviceGetTotalEnergyConsumption(h), time.time()
    nb.nb_check_status()
    n = reps * per_graph
    us, joule = e0.elapsed_time(e1) * 1e3 / n, (j1 - j0) / 1e3 / n
    print(f"{kind} BT={BT} C={C} OC={OC} sustained: {us:.1f} us/call  {flops / us / 1e6:.0f} TFLOP/s  "
          f"{joule * 1e3:.2f} mJ/call  {joule / flops * 1e12:.3f} pJ/flop  {(j1 - j0) / 1e3 / (t1 - t0):.0f} W")
    return 0


def main(argv) -> int:
    if len(argv) < 5:
        print(__doc__)
        return 2
    kind, BT, C, OC = argv[1], int(argv[2]), int(argv[3]), int(argv[4])
    reps = int(argv[5]) if len(argv) > 5 else 20
    if len(argv) > 6 and argv[6] == "energy":
        return sustained_energy(kind, BT, C, OC)
    dev = "cuda"
    bf, f32 = torch.bfloat16, torch.float32
    inp = synth.normal(1, (BT, C), 1.0, dev)
    w = synth.normal(2, (OC, C), 0.02, dev)
    b = synth.normal(3, (OC,), 0.02, dev)
    dout = synth.normal(4, (BT, OC), 1e-3, dev)
    ipre = synth.normal(5, (BT, C), 1.0, dev)
    out = torch.empty((BT, OC), dtype=bf, device=dev)
    pre = torch.empty((BT, OC), dtype=bf, device=dev)
    dinp = torch.empty((BT, C), dtype=bf, device=dev)
    dw = torch.zeros((OC, C), dtype=f32, device=dev)
    db = torch.zeros((OC,), dtype=f32, device=dev)
    calls = {
        "fwd": lambda: nb.nb_linear_forward_ex(out, None, inp, w, b, BT, C, OC, nb.ACT_NONE),
        "fwd_nobias": lambda: nb.nb_linear_forward_ex(out, None, inp, w, None, BT, C, OC, nb.ACT_NONE),
        "fwd_gelu": lambda: nb.nb_linear_forward_ex(out, pre, inp, w, b, BT, C, OC, nb.ACT_GELU),
        "fwd_swiglu": lambda: nb.nb_linear_forward_ex(out, pre, inp, w, None, BT, C, OC, nb.ACT_SWIGLU),
        "dgrad": lambda: nb.nb_linear_backward_ex(dinp, None, None, dout, None, w, None, None, BT, C, OC, 0, 0),
        "dgrad_fused": lambda: nb.nb_linear_backward_ex(dinp, None, None, dout, None, w, None, ipre, BT, C,
                                                        OC, 0, 0),
        "wgrad": lambda: nb.nb_linear_backward_ex(None, dw, None, dout, inp, None, None, None, BT, C, OC, 0, 1),
        "wgrad_bias": lambda: nb.nb_linear_backward_ex(None, dw, db, dout, inp, None, None, None, BT, C, OC,
                                                       0, 1),
        "dbias": lambda: nb.nb_reduce_dbias(db, dout, BT, OC, 1),
        "bwd": lambda: nb.nb_linear_backward_ex(dinp, dw, db, dout, inp, w, None, None, BT, C, OC, 0, 1),
        "bwd_nobias": lambda: nb.nb_linear_backward_ex(dinp, dw, None, dout, inp, w, None, None, BT, C, OC, 0, 1),
        "bwd_fused": lambda: nb.nb_linear_backward_ex(dinp, dw, db, dout, inp, w, None, ipre, BT, C, OC, 0, 1),
    }
    if kind == "cast":
        n = OC * C
        src = torch.randn(n, dtype=f32, device=dev)
        dst = torch.empty(n, dtype=bf, device=dev)
        calls["cast"] = lambda: nb.nb_cast_f32_to_bf16(dst, src, n)
    if kind in ("head_ce", "ce_bwd"):
        V = OC - 47 if OC > 47 else OC
        tg = torch.randint(0, V, (BT,), dtype=torch.int32, device=dev)
        loss = torch.empty(BT, dtype=f32, device=dev)
        lse = torch.empty(BT, dtype=f32, device=dev)
        calls["head_ce"] = lambda: nb.nb_lm_head_ce_forward(out, loss, lse, inp, w, tg, BT, C, OC, V)
        if kind == "ce_bwd":
            calls["head_ce"]()
            calls["ce_bwd"] = lambda: nb.nb_ce_backward(pre, out, lse, tg, 1.0 / BT, BT, OC, V)
    if kind in ("lora_fwd", "lora_bwd"):
        r, scale = 16, 8.0
        la = synth.normal(6, (r, C), 0.02, dev)
        lb = synth.normal(7, (OC, r), 0.02, dev)
        t = torch.empty((BT, r), dtype=bf, device=dev)
        u = torch.empty((BT, r), dtype=bf, device=dev)
        dla = torch.zeros((r, C), dtype=f32, device=dev)
        dlb = torch.zeros((OC, r), dtype=f32, device=dev)
        calls["lora_fwd"] = lambda: nb.nb_lora_linear_forward(out, t, inp, w, None, la, lb, scale, BT, C, OC, r)
        calls["lora_fwd"]()
        calls["lora_bwd"] = lambda: nb.nb_lora_linear_backward(dinp, dla, dlb, u, dout, inp, w, la, lb, t,
                                                               scale, BT, C, OC, r, 1)
    if kind not in calls:
        print(__doc__)
        return 2
    call = calls[kind]
    for _ in range(2):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        call()
    e1.record()
    torch.cuda.synchronize()
    nb.nb_check_status()
    ms = e0.elapsed_time(e1) / reps
    if kind == "cast":
        print(f"cast n={OC * C}: {ms * 1e3:.1f} us/call  {OC * C * 6 / ms / 1e6:.1f} GB/s")
        return 0
    if kind == "ce_bwd":
        print(f"ce_bwd BT={BT} Vp={OC}: {ms * 1e3:.1f} us/call  {BT * OC * 4 / ms / 1e6:.1f} GB/s")
        return 0
    flops = 2 * BT * C * OC * (2 if kind.startswith("bwd") else 1)
    if kind == "lora_fwd":
        flops += 2 * BT * 16 * (C + OC)
    if kind == "lora_bwd":
        flops += 4 * BT * 16 * (C + OC)
    print(f"{kind} BT={BT} C={C} OC={OC}: {ms * 1e3:.1f} us/call  {flops / ms / 1e9:.1f} TFLOP/s")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
