"""Replay a captured training step many times and check that the results do not move.

    python -m paper_2609_28568_b200.soak [WORKLOAD] [REPLAYS] [CHECK_EVERY]

WORKLOAD is `gpt2` (the GPT-2 124M stack, 4 micro-steps at BT = 16384; default) or `qwen3_lora` (the
adapter stage). One step is captured into a CUDA graph and replayed REPLAYS times (default 1000). Every
CHECK_EVERY replays (default 100) the bf16 results of every layer (out, pre-activation, dinp) must be
bit-identical to the first replay's — none of them is summed across CTAs — and the fp32 gradients, whose
partial sums meet in memory in varying order, equal to rounding; the library's status word must be clean.
A stage handed back too early, a barrier phase off by one or a missing dependency between launches shows
up here as a rare mismatch. Exit code 0 when everything held.
"""
from __future__ import annotations

import sys
import time

import torch

from . import binding as nb
from .stack import LinearStack, LoraStack


def _digest(tensors) -> list[int]:
    # exact and cheap: the bit patterns of a bf16 tensor summed as integers
    return [int(t.view(torch.int16).to(torch.int64).sum().item()) for t in tensors]


def soak(workload: str = "gpt2", replays: int = 1000, every: int = 100, device: int = 0) -> float:
    dev = torch.device("cuda", device)
    torch.cuda.set_device(dev)
    if workload == "gpt2":
        stack = LinearStack("gpt2", 16384, 4, device=dev, config_id=4)
    elif workload == "qwen3_lora":
        stack = LoraStack(16384, 1, device=dev, config_id=6, fused=True)
    else:
        raise ValueError("workload must be gpt2 or qwen3_lora")
    for _ in range(3):
        stack.step()
    torch.cuda.synchronize()
    cap = torch.cuda.Stream(device=dev)
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=cap):
            stack.step()
    torch.cuda.current_stream().wait_stream(cap)
    bf16 = [t for L in stack.layers for t in (getattr(L, "out", None), getattr(L, "pre", None),
                                              getattr(L, "dinp", None)) if t is not None]
    grads = stack.gradient_tensors()
    graph.replay()
    torch.cuda.synchronize()
    ref_digest, ref_grads = _digest(bf16), [g.clone() for g in grads]
    worst = 0.0
    for i in range(replays):
        graph.replay()
        if (i + 1) % every == 0 or i + 1 == replays:
            torch.cuda.synchronize()
            d = _digest(bf16)
            if d != ref_digest:
                moved = [k for k in range(len(d)) if d[k] != ref_digest[k]]
                raise AssertionError(f"replay {i}: bf16 results changed (tensors {moved[:8]})")
            for g, r in zip(grads, ref_grads):
                worst = max(worst, float((g.double() - r.double()).norm() / (r.double().norm() + 1e-30)))
            if worst > 1e-4:
                raise AssertionError(f"replay {i}: fp32 gradients drifted by {worst:.3e}")
            nb.nb_check_status()
    return worst


def main(argv) -> int:
    workload = argv[1] if len(argv) > 1 else "gpt2"
    replays = int(argv[2]) if len(argv) > 2 else 1000
    every = int(argv[3]) if len(argv) > 3 else 100
    t0 = time.time()
    worst = soak(workload, replays, every)
    print(f"{workload}: {replays} replays, bf16 results bit-identical, worst fp32 gradient drift {worst:.2e}, "
          f"{time.time() - t0:.1f} s")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
