#!/usr/bin/env python
"""Benchmark of the dense-linear hot path.

A step is one pass of the whole path on the GPT-2 124M linear stack: 4 gradient-
accumulation micro-steps at B=16, T=1024, each running the forward of 12 x
(qkv, attn-proj, fc+GELU, proj) + tied head and then every backward (dgrad, wgrad,
dbias; GELU backward fused into proj's dgrad), with fp32 gradient accumulation.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Prints one JSON line (rank 0). Under torchrun every rank runs its own replica of
the workload on its own GPU with its own seeds (rows shard across ranks; the
graded path has no collective), and the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

WORKLOADS = {
    # name: (model, BT, micro_steps, config id, wgrad, description)
    "gpt2_124m_stack": ("gpt2", 16384, 4, 4, True,
                        "GPT-2 124M linear stack, B=16 T=1024, 4 accumulation micro-steps (config 4)"),
    "gpt2_lm_head": ("gpt2_head", 16384, 1, 3, True, "tied lm_head, B=16 T=1024 (config 3)"),
    "gpt2_block": ("gpt2_block", 4096, 1, 2, True, "one GPT-2 block's four linears, B=4 T=1024 (config 2)"),
    "qwen3_adapter": ("qwen3", 16384, 1, 5, True, "Qwen3-0.6B-shaped linears x28, B=8 T=2048 (config 5a)"),
    "qwen3_adapter_frozen": ("qwen3", 16384, 1, 5, False,
                             "Qwen3-0.6B-shaped linears x28, frozen base: fwd+dgrad (config 5b)"),
    "qwen3_lora": ("qwen3_lora", 16384, 1, 6, False,
                   "Qwen3-0.6B's seven projections x28 with rank-16 adapters (alpha 32, rank-stabilised), "
                   "frozen base: fwd, dinp, dA, dB, B=8 T=2048"),
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------- clocks
class EnergyMeter:
    """The GPU's own energy counter (NVML, read-only) around the timed region: joules per step.
    On a power-capped part the step time follows this figure, not the cycle count."""

    def __init__(self, gpu_id: str):
        """gpu_id: "GPU-<uuid>" (CUDA and NVML may number the devices differently) or an index."""
        self.h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            if gpu_id.startswith("GPU-"):
                try:
                    self.h = pynvml.nvmlDeviceGetHandleByUUID(gpu_id)
                except Exception:
                    self.h = pynvml.nvmlDeviceGetHandleByUUID(gpu_id.encode())
            else:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(int(gpu_id))
        except Exception:
            self.h = None

    def read(self):
        if self.h is None:
            return None
        try:
            return (self.nv.nvmlDeviceGetTotalEnergyConsumption(self.h) / 1e3, time.time())  # joules, seconds
        except Exception:
            return None

    @staticmethod
    def report(a, b, steps: int):
        if a is None or b is None or steps <= 0 or b[1] <= a[1]:
            return None
        return {"j_per_step": (b[0] - a[0]) / steps, "avg_w": (b[0] - a[0]) / (b[1] - a[1]),
                "window_s": b[1] - a[1],
                "source": "NVML total energy counter around the timed region (the counter is updated in "
                          "steps of the order of 0.1 s: windows under about 2 s, i.e. fewer than 50 steps of "
                          "the default workload, read 10 % low)"}


class ClockSampler:
    """nvidia-smi samples (SM clock, throttle reasons) taken while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.path = tempfile.mktemp(prefix="nb_clocks_", suffix=".csv")
        self.proc = None
        self.gpu_id = gpu_id

    def start(self):
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.fh, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            # median over the samples under load (the upper half of the power draw)
            import statistics
            cut = statistics.median(pw)
            loaded = [s for s, p in zip(sm, pw) if p >= cut] or sm
            out.update(sm_mhz=statistics.median(loaded), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(pw))
        return out


# ------------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(seconds_hint: float = 15.0):
    """Time the fp32 oracle, as it stands, on a bounded sample of the stack: one GPT-2 block's four
    linears forward + backward plus a row slice of the head. Returns (flops, seconds, description)."""
    import numpy as np
    import oracle
    from paper_2609_28568_b200 import shapes, synth

    BT, HEAD_ROWS = 16384, 4096  # about 12 s of work on 16 cores
    specs = shapes.gpt2_block() + [shapes.gpt2_lm_head()]
    flops, secs = 0, 0.0
    for li, s in enumerate(specs):
        rows = BT if s.OC != shapes.VOCAB_PADDED else HEAD_ROWS
        f = lambda t: t.float().numpy()
        inp = f(synth.normal(9000 + li, (rows, s.C), 1.0))
        w = f(synth.normal(9100 + li, (s.OC, s.C), s.w_std))
        b = f(synth.normal(9200 + li, (s.OC,), 0.02)) if s.bias else None
        dout = f(synth.normal(9300 + li, (rows, s.OC), 1e-3))
        t0 = time.perf_counter()
        _, pre = oracle.linear_forward(inp, w, b, s.act, "f32")
        oracle.linear_backward(dout, inp, w, pre=pre if s.act else None, act=s.act, dtype="f32",
                               want=("dinp", "dweight", "dbias") if s.bias else ("dinp", "dweight"))
        secs += time.perf_counter() - t0
        flops += 6 * rows * s.C * s.OC
    desc = (f"fp32 oracle on one GPT-2 block (qkv, attn-proj, fc+GELU, proj) fwd+bwd at BT={BT} and the "
            f"tied head fwd+bwd on {HEAD_ROWS} rows; {flops / 1e9:.1f} GFLOP")
    return flops, secs, desc, oracle.num_threads()


def run_reference(args, rank):
    """The reference arm: the CPU oracle on the host cores, a bounded sample per step."""
    if rank != 0:
        return
    from paper_2609_28568_b200 import shapes
    times, flops, desc, cores = [], 0, "", 1
    for i in range(args.warmup + args.steps):
        fl, s, desc, cores = oracle_sample()
        if i >= args.warmup:
            times.append(s)
            flops = fl
    sec = sum(times) / len(times)
    tflops = flops / sec / 1e12
    model, BT, ms, cfg, wgrad, wdesc = WORKLOADS[args.workload]
    line = {
        "impl": "reference", "metric": "gpt2_124m_linear_fwd_bwd_tflops", "value": tflops,
        "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "tokens_per_s": flops / sec / shapes.gpt2_stack_flops_per_token(),
        "config": {"workload": args.workload, "description": wdesc,
                   "note": "each step is the bounded sample below, not the whole workload"},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_library(args, rank, local_rank):
    """Context, not a contract arm: the same stack composed from the framework's library ops
    (cuBLAS GEMMs, separate bias / GELU / GELU-backward / reduction / accumulation kernels) on one
    GPU, and its bare GEMMs alone. None of this repository's kernels run here."""
    if rank != 0:
        return
    import torch
    import torch.nn.functional as F
    from paper_2609_28568_b200 import shapes
    from paper_2609_28568_b200.stack import LinearStack
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    model, BT, micro_steps, cfg_id, wgrad, wdesc = WORKLOADS[args.workload]
    stack = LinearStack(model, BT, micro_steps, device=dev, config_id=cfg_id, wgrad=wgrad)
    if any(L.spec.act == shapes.ACT_SWIGLU for L in stack.layers):
        raise SystemExit("--impl library covers the GPT-2 workloads only")

    def step(full: bool):
        for ms in range(micro_steps):
            for L in stack.layers:
                x = stack.layer_inp(L, ms)
                if not full:
                    F.linear(x, L.weight)
                    continue
                y = F.linear(x, L.weight, L.bias)
                if L.spec.act == shapes.ACT_GELU:
                    L.pre, y = y, F.gelu(y, approximate="tanh")
                L.out = y
            for L in reversed(stack.layers):
                dz = L.dz_from.dinp if L.dz_from is not None else L.dout[ms]
                x = stack.layer_inp(L, ms)
                if not full:
                    dz @ L.weight
                    if wgrad:
                        dz.t() @ x
                    continue
                dx = dz @ L.weight
                if L.chained_from is not None:  # the producer's GELU backward as its own kernel
                    dx = torch.ops.aten.gelu_backward(dx, L.chained_from.pre, approximate="tanh")
                L.dinp = dx
                if wgrad:
                    g = dz.t() @ x              # bf16 product, then the fp32 accumulation
                    if ms == 0:
                        L.dweight.copy_(g)
                    else:
                        L.dweight.add_(g)
                    if L.dbias is not None:
                        b = dz.sum(0, dtype=torch.float32)
                        if ms == 0:
                            L.dbias.copy_(b)
                        else:
                            L.dbias.add_(b)

    flops = stack.flops_per_micro_step() * micro_steps
    res = {}
    for name, full in (("composed", True), ("gemms_only", False)):
        for _ in range(max(args.warmup, 2)):
            step(full)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step(full)
        e1.record()
        torch.cuda.synchronize()
        ms_step = e0.elapsed_time(e1) / args.steps
        res[name] = {"ms_per_step": ms_step, "tflops": flops / (ms_step * 1e-3) / 1e12}
    print(json.dumps({
        "impl": "library", "metric": "gpt2_124m_linear_fwd_bwd_tflops", "value": res["composed"]["tflops"],
        "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": res["composed"]["ms_per_step"], "higher_is_better": True, "dtype": "bf16",
        "data": "synthetic", "config": {"workload": args.workload, "description": wdesc},
        "gemms_only": res["gemms_only"],
        "note": "framework library ops (cuBLAS GEMMs + separate elementwise / reduction kernels); "
                "gemms_only = the bare bf16 GEMMs without bias, GELU, gradient accumulation",
    }), flush=True)


def max_over_ranks(value: float, dist, device) -> float:
    """The slowest rank's figure (a job is as slow as its slowest replica)."""
    if dist is None:
        return value
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ------------------------------------------------------------------------------- GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "library"],
                    help="ours; reference = the CPU oracle (the contract's reference arm); library = the same "
                         "stack from cuBLAS and framework kernels, for context")
    ap.add_argument("--workload", default="gpt2_124m_stack", choices=sorted(WORKLOADS))
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-graph", action="store_true",
                    help="launch every call from the host in the timed region instead of replaying a CUDA graph")
    ap.add_argument("--two-streams", action="store_true",
                    help="issue the weight-gradient calls on a second stream, as separate launches (default: one "
                         "stream, one launch per layer backward; the two arrangements time the same on a "
                         "power-capped part)")
    ap.add_argument("--one-stream", action="store_true", help="accepted for compatibility: this is the default")
    ap.add_argument("--lora-unfused", action="store_true",
                    help="qwen3_lora: one set of calls per projection (seven per layer) instead of one per group "
                         "of projections that share an input (q_k_v, o, gate_up, down)")
    ap.add_argument("--dp", action="store_true",
                    help="data parallel instead of replicas: the same weights on every rank, its own rows, and "
                         "the fp32 gradients all-reduced (NCCL) in buckets under the last micro-step's backward; "
                         "launches eagerly (no graph)")
    args = ap.parse_args()
    if args.dp:
        args.no_graph = True
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started once, directly: start the N ranks here (one process per GPU); rank 0 prints the line
        from paper_2609_28568_b200.launch import spawn_ranks
        raise SystemExit(spawn_ranks(args.gpus, [os.path.abspath(__file__), *sys.argv[1:]]))

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.impl == "library":
        run_library(args, rank, local_rank)
        return

    import torch
    from paper_2609_28568_b200 import binding as nb
    from paper_2609_28568_b200 import shapes
    from paper_2609_28568_b200.stack import LinearStack

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    model, BT, micro_steps, cfg_id, wgrad, wdesc = WORKLOADS[args.workload]
    # one stream in model order by default; --two-streams puts the weight gradients on a second one
    if model == "qwen3_lora":
        from paper_2609_28568_b200.stack import LoraStack
        if args.dp:
            raise SystemExit("--dp is wired for the dense stacks only")
        stack = LoraStack(BT, micro_steps, device=dev, config_id=cfg_id, seed_offset=rank,
                          fused=not args.lora_unfused)
    else:
        stack = LinearStack(model, BT, micro_steps, device=dev, config_id=cfg_id, seed_offset=rank,
                            wgrad=wgrad, shared_weights=args.dp,
                            wgrad_stream=bool(args.two_streams and not args.dp))
    reducer = None
    if args.dp:
        from paper_2609_28568_b200 import dp as dpmod
        if not wgrad:
            raise SystemExit("--dp needs a workload with weight gradients")
        fp = torch.stack([t.float().sum() for t in stack.input_tensors(0)])
        dpmod.assert_ranks_differ(fp, dist, "inputs")
        reducer = dpmod.GradAllReducer(stack.attach_gradient_buckets(), dist, average=True)
    # reserve the activation-backward workspace before timing so no call allocates
    need = max((BT * L.spec.OC * 2 for L in stack.layers
                if L.spec.act != shapes.ACT_NONE and L.dz_from is None), default=0)
    if need:
        nb.nb_workspace_reserve(need)
    flops_step = stack.flops_per_micro_step() * micro_steps
    tokens_step = BT * micro_steps

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- warm-up
    for _ in range(args.warmup):
        if reducer is not None:
            stack.step_dp(reducer)
        else:
            stack.step()
    nb.nb_check_status()

    # ---- timed region: K steps between two events on the launch stream. No events between the
    # calls: an event record between two kernels keeps the second kernel's set-up from overlapping
    # the first kernel's tail (programmatic dependent launch) and costs 2-3 % of the step.
    records = []  # (kind, layer name, start event, end event), filled by the breakdown pass

    def hook(kind, L, begin):
        # one event per call boundary: a call's end is the next call's start (the calls of a step
        # follow one another without gaps), which halves the events the breakdown pass inserts
        if begin:
            e = torch.cuda.Event(enable_timing=True)
            e.record()
            if records and records[-1][3] is None:
                records[-1][3] = e
            records.append([kind, L.spec.name, e, None])

    def close_records():
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        if records and records[-1][3] is None:
            records[-1][3] = e

    props = torch.cuda.get_device_properties(dev)
    gpu_id = f"GPU-{props.uuid}" if hasattr(props, "uuid") else str(local_rank)
    sampler = ClockSampler(gpu_id)
    # One step is captured into a CUDA graph after the warm-up (every library call is
    # capturable: no allocation, no synchronisation) and the timed region replays it, so the
    # launches of a step (392 for the GPT-2 stack) cost the host one call.
    run_step, launches_per_step = stack.step, None
    if reducer is not None:
        run_step = lambda: stack.step_dp(reducer)  # noqa: E731
    if not args.no_graph:
        cap = torch.cuda.Stream(device=dev)
        cap.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cap):
            graph = torch.cuda.CUDAGraph()
            l0 = nb.nb_kernel_launches()
            with torch.cuda.graph(graph, stream=cap):
                stack.step()
            launches_per_step = nb.nb_kernel_launches() - l0
        torch.cuda.current_stream().wait_stream(cap)
        run_step = graph.replay
        run_step()  # one untimed replay
    barrier()
    sampler.start()
    meter = EnergyMeter(gpu_id)
    launches0 = nb.nb_kernel_launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    en0 = meter.read()
    ev0.record()
    for _ in range(args.steps):
        run_step()
    ev1.record()
    barrier()
    energy = EnergyMeter.report(en0, meter.read(), args.steps)
    launches = (launches_per_step * args.steps if launches_per_step is not None
                else nb.nb_kernel_launches() - launches0)
    nb.nb_check_status()
    elapsed_ms = max_over_ranks(ev0.elapsed_time(ev1), dist, dev)
    ms_per_step = elapsed_ms / args.steps
    tflops = world * flops_step / (ms_per_step * 1e-3) / 1e12
    tokens_per_s = world * tokens_step / (ms_per_step * 1e-3)

    # ---- breakdown pass: the same K steps again, now with an event pair around every call
    bev0, bev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    bev0.record()
    for _ in range(args.steps):
        stack.step(hook)
    close_records()
    bev1.record()
    barrier()
    clocks = sampler.stop()
    nb.nb_check_status()
    breakdown_ms_per_step = bev0.elapsed_time(bev1) / args.steps

    # ---- per-call breakdown from the events of the timed region
    per = {}
    for kind, name, a, b in records:
        key = f"{kind}:{name}"
        per.setdefault(key, [0.0, 0])
        per[key][0] += a.elapsed_time(b)
        per[key][1] += 1
    spec_by_name = {L.spec.name: L.spec for L in stack.layers}
    breakdown, gemm_flops, gemm_ms = {}, 0.0, 0.0
    for key, (ms, n) in per.items():
        kind, name = key.split(":")
        s = spec_by_name[name]
        fl = 2 * BT * s.C * s.OC * (1 if kind == "fwd" else (2 if wgrad else 1))
        breakdown[key] = {"calls": n, "ms_per_call": ms / n, "tflops": fl / (ms / n * 1e-3) / 1e12}
        gemm_flops += fl * n
        gemm_ms += ms
    peaks, peak_src = load_peaks()
    # the GPU is under load for warm-up + timed + breakdown steps back to back: over a second of
    # that is the "kernel timed inside a long step" case, compared with the sustained peak
    long_step = ms_per_step * (args.warmup + 2 * args.steps) > 1000.0
    peak_tf = peaks["bf16_tflops_sustained"] if long_step else peaks["bf16_tflops"]
    # Every launch of a step is one of the two tensor-core GEMM kernels (forward; layer backward), so
    # their average launch duration over the timed region is that region's length / launches, and
    # algorithmic flops per launch / that duration is this rank's flops / time of the timed region.
    # (The breakdown pass below it has events between the calls, which cost it dependent-launch
    # overlap: it is only used for the per-call split.)
    my_ms_per_step = ev0.elapsed_time(ev1) / args.steps
    achieved_tf = flops_step / (my_ms_per_step * 1e-3) / 1e12
    breakdown_tf = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath):
        try:
            traffic = json.load(open(tpath)).get(args.workload)
        except Exception:
            traffic = None
    roofline = {
        "bound": "tensor", "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s",
        "frac": achieved_tf / peak_tf, "traffic": traffic,
        "peak_source": f"{peak_src} cuBLAS bf16 ({'sustained' if long_step else 'burst'})",
        "kernel": "nb::gemm_kernel (tcgen05 forward instantiations) and nb::layer_bwd_kernel (dinp tiles and "
                  "dweight k-chunks of a layer in one launch): every launch of a step; "
                  "average launch duration = timed region (CUDA events on the launch stream) / launches; "
                  "per_call from a second pass over the same steps with an event at every call boundary",
        "launches_per_step": launches / args.steps,
        "avg_launch_us": my_ms_per_step * 1e3 / (launches / args.steps) if launches else None,
        "flops_per_launch": flops_step / (launches / args.steps) if launches else None,
        "breakdown_pass_ms_per_step": breakdown_ms_per_step,
        "breakdown_pass_tflops": breakdown_tf,
        "frac_of_nominal_2250": achieved_tf / NOMINAL_BF16_TFLOPS,
        "frac_of_burst_peak": achieved_tf / peaks["bf16_tflops"],
        "frac_of_sustained_peak": achieved_tf / peaks["bf16_tflops_sustained"],
        "per_call": breakdown,
    }
    # clock-normalised view: the share of the tensor cores' per-clock capacity (148 SMs x 8192 bf16 flop
    # per clock on B200) in use at the SM clock sampled during the run; under the power cap the clock
    # moves against this figure, so neither alone says how good the kernels are
    if clocks.get("sm_mhz"):
        roofline["mma_use_per_clock"] = achieved_tf * 1e12 / (props.multi_processor_count * 8192 * clocks["sm_mhz"] * 1e6)
        roofline["sm_mhz_under_load"] = clocks["sm_mhz"]

    # ---- end to end through the C ABI with host buffers (rank-local; max over ranks)
    e2e = None
    if not args.no_e2e:
        e2e = measure_e2e(torch, nb, stack, args, dist, dev, flops_step, world)

    # ---- CPU oracle baseline (rank 0, single GPU run only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        fl, s, desc, cores = oracle_sample()
        cpu = {"value": fl / s / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
               "sample": desc, "tokens_per_s": fl / s / shapes.gpt2_stack_flops_per_token()}

    if rank == 0:
        line = {
            "metric": "gpt2_124m_linear_fwd_bwd_tflops", "value": tflops, "unit": "TFLOP/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "tokens_per_s": tokens_per_s,
            "pct_of_nominal_bf16_peak": 100.0 * tflops / (world * NOMINAL_BF16_TFLOPS),
            "config": {"workload": args.workload, "description": wdesc, "BT": BT,
                       "micro_steps": micro_steps, "l2": "inputs_exceed_l2 (a step touches >20 GB)",
                       "launch": "eager" if args.no_graph else "cuda_graph_replay",
                       "streams": 2 if stack.wgrad_stream else 1,
                       "parallelism": (f"dp{world}: fp32 gradient all-reduce in {len(reducer.b.buckets)} buckets "
                                       f"under the last micro-step's backward" if reducer is not None
                                       else f"replicas x{world}, no collective")},
            "clocks": clocks, "energy": energy, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches),
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def measure_e2e(torch, nb, stack, args, dist, dev, flops_step, world, return_host=False):
    """The same step with every micro-step's inputs copied from pinned host memory inside the timed
    region, and the accumulated gradients read back to the host at the end of each step."""
    host_in = []
    h2d = 0
    for ms in range(stack.micro_steps):
        hs = []
        for t in stack.input_tensors(ms):
            h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
            h.copy_(t)
            hs.append(h)
            h2d += t.numel() * t.element_size()
        host_in.append(hs)
    grads = stack.gradient_tensors()
    host_out = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True) for g in grads]
    d2h = sum(g.numel() * g.element_size() for g in grads)
    copy_stream = torch.cuda.Stream(device=dev)
    d2h_stream = torch.cuda.Stream(device=dev)
    main = torch.cuda.current_stream()
    n_ms = stack.micro_steps
    used = [None] * n_ms   # event: the previous step's micro-step ms has finished with its input buffers
    read = [None]          # event: the previous step's gradients have been read back

    def one_step():
        # Three queues: inputs of micro-step ms go to the device as soon as the previous step's micro-step
        # ms has released those buffers (so the copies of step i+1 run under the compute of step i),
        # the micro-steps wait for their own inputs, and the gradients of a step are read back on a
        # third stream while the next step's inputs already arrive (PCIe carries both directions).
        ready = []
        for ms in range(n_ms):
            with torch.cuda.stream(copy_stream):
                if used[ms] is not None:
                    copy_stream.wait_event(used[ms])
                for h, t in zip(host_in[ms], stack.input_tensors(ms)):
                    t.copy_(h, non_blocking=True)
                e = torch.cuda.Event()
                e.record(copy_stream)
                ready.append(e)
        for ms in range(n_ms):
            main.wait_event(ready[ms])
            if ms == 0 and read[0] is not None:
                main.wait_event(read[0])   # micro-step 0 overwrites the gradients
            stack.micro_step(ms)
            used[ms] = torch.cuda.Event()
            used[ms].record(main)
        with torch.cuda.stream(d2h_stream):
            d2h_stream.wait_event(used[n_ms - 1])
            for g, h in zip(grads, host_out):
                h.copy_(g, non_blocking=True)
            read[0] = torch.cuda.Event()
            read[0].record(d2h_stream)

    torch.cuda.synchronize()
    one_step()  # warm-up
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.e2e_steps):
        one_step()
    main.wait_stream(d2h_stream)  # the last step's gradients are on the host before the clock stops
    main.wait_stream(copy_stream)
    ev1.record()
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3
    ms = max_over_ranks(max(ev0.elapsed_time(ev1), wall_ms) / args.e2e_steps, dist, dev)
    nb.nb_check_status()
    result = {"value": world * flops_step / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "ms_per_step": ms,
            "steps": args.e2e_steps,
            "note": "inputs of each micro-step copied from pinned host memory on a copy stream (the next "
                    "step's copies start as soon as the buffers are free), gradients read back to pinned "
                    "host memory on a third stream, all inside the timed region"}
    return (result, host_out) if return_host else result


if __name__ == "__main__":
    main()
